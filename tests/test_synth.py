"""The synthetic input recipe: parameter-set sizes, policies as data, and the statistics of
the gradient streams (per-tensor scale, share of the signal common to the workers)."""
import math

import numpy as np
import pytest
import torch

from paper_2202_06009_b200 import synth


def test_layout_sizes():
    # BERT-Base / BERT-Large with the pre-training heads, GPT-2 with 48 layers of width 1600.
    assert synth.bert_base().n == 110_106_428
    assert synth.bert_large().n == 336_226_108
    assert synth.gpt2_xl().n == 1_557_611_200
    assert synth.tiny().n == 1 << 20
    # one encoder layer of BERT-Base: 4 projections, 2 LayerNorms, the feed-forward pair
    h, f = 768, 3072
    per_layer = 4 * (h * h + h) + 2 * 2 * h + h * f + f + f * h + h
    base = synth._bert_tensors(12, h, f)
    more = synth._bert_tensors(13, h, f)
    assert sum(more) - sum(base) == per_layer


@pytest.mark.parametrize("make, n_sync, n_var", [(synth.tiny, 40, 6), (synth.bert_base, 114, 9),
                                                 (synth.bert_large, 82, 8), (synth.gpt2_xl, 25, 7)])
def test_policy_counts(make, n_sync, n_var):
    wl = make()
    assert sum(wl.in_T_u(t) for t in range(wl.steps)) == n_sync
    assert sum(wl.in_T_v(t) for t in range(wl.steps)) == n_var
    # every variance step is also a sync step, so v never changes inside a local interval
    assert all(wl.in_T_u(t) for t in range(wl.steps) if wl.in_T_v(t))


def test_scaled_keeps_structure():
    wl = synth.scaled(synth.bert_large(), 64)
    base = synth.bert_large()
    assert len(wl.tensors) == len(base.tensors) and (wl.W, wl.chunk) == (base.W, base.chunk)
    assert abs(wl.n - base.n / 64) < len(base.tensors)
    assert wl.n % wl.chunk != 0          # still ends in a ragged chunk


def _corr(a, b):
    a, b = a.double(), b.double()
    return float((a * b).mean() / math.sqrt(float((a * a).mean()) * float((b * b).mean())))


def test_tiny_stream_statistics():
    wl = synth.tiny(n=1 << 18)
    g = synth.GradientStream(wl, "cpu").fill(0)
    assert len(g) == wl.W and all(b.shape == (wl.n,) and b.dtype == torch.float32 for b in g)
    # g = s + 0.5 n_i: variance 1.25, correlation between two workers 1 / 1.25
    for b in g:
        assert abs(float(b.double().var()) - 1.25) < 0.02
        assert abs(float(b.double().mean())) < 0.01
    assert abs(_corr(g[0], g[1]) - 0.8) < 0.01
    assert abs(_corr(g[1], g[3]) - 0.8) < 0.01


def test_bert_stream_statistics():
    wl = synth.scaled(synth.bert_base(), 32)
    stream = synth.GradientStream(wl, "cpu")
    g = [b.clone() for b in stream.fill(3)]
    scales = synth.tensor_scales(wl)
    assert len(scales) == len(wl.tensors) and min(scales) > 0
    # per tensor: standard deviation sigma_T, 70 % of the variance shared between workers
    off, checked = 0, 0
    for size, sigma in zip(wl.tensors, scales):
        if size >= 50_000:
            a, b = g[0][off:off + size], g[5][off:off + size]
            assert abs(float(a.double().std()) / sigma - 1.0) < 0.03
            assert abs(_corr(a, b) - 0.7) < 0.03
            checked += 1
        off += size
    assert checked >= 3
    # log of the scales is standard normal: loosely, its spread over ~200 tensors
    logs = np.log(np.array(scales))
    assert abs(logs.mean()) < 0.3 and 0.7 < logs.std() < 1.3


def test_gpt2_stream_is_heavy_tailed():
    wl = synth.scaled(synth.gpt2_xl(), 4096)
    g = synth.GradientStream(wl, "cpu").fill(0)
    scales = synth.tensor_scales(wl)
    size, sigma = wl.tensors[0], scales[0]          # the token embedding
    a = (g[0][:size] / sigma).double()
    b = (g[2][:size] / sigma).double()
    # Student-t noise: far more mass beyond 6 standard deviations than a Gaussian's 2e-9
    assert float((a.abs() > 6).double().mean()) > 1e-5
    # the shared part still dominates: robust (rank) correlation well above one half
    ra, rb = a.argsort().argsort().double(), b.argsort().argsort().double()
    ra, rb = ra - ra.mean(), rb - rb.mean()
    assert 0.6 < _corr(ra, rb) < 0.85


def test_streams_are_reproducible_and_distinct():
    wl = synth.tiny(n=4096)
    a = [b.clone() for b in synth.GradientStream(wl, "cpu").fill(7)]
    b = [b.clone() for b in synth.GradientStream(wl, "cpu").fill(7)]
    c = [b.clone() for b in synth.GradientStream(wl, "cpu").fill(8)]
    d = [b.clone() for b in synth.GradientStream(wl, "cpu", seed=1).fill(7)]
    assert all(torch.equal(x, y) for x, y in zip(a, b))
    assert not torch.equal(a[0], c[0]) and not torch.equal(a[0], d[0]) and not torch.equal(a[0], a[1])
    x0 = synth.initial_params(wl, "cpu")
    assert abs(float(x0.std()) - wl.x0_std) < 0.002 and torch.equal(x0, synth.initial_params(wl, "cpu"))
