"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times.  The method is chunk-local (every reduction stays inside one chunk), so
the oracle runs on a sample of chunks - the first, the ragged last, chunks that
straddle tensor boundaries, random ones - gathered into one short vector, and is
compared with the same chunks of the full-size GPU state."""
import numpy as np
import pytest
import torch

from helpers import assert_close
from oracle import zoa_oracle as zo
from paper_2202_06009_b200 import Zoa, synth

pytestmark = pytest.mark.gpu


def _sample_chunks(wl, count, seed):
    n_chunks = -(-wl.n // wl.chunk)
    picks = {0, 1, n_chunks - 2}
    off = 0
    for size in wl.tensors[:40]:                      # chunks that straddle a tensor boundary
        off += size
        picks.add(min(off // wl.chunk, n_chunks - 2))
    rng = np.random.default_rng(seed)
    while len(picks) < count - 1:
        picks.add(int(rng.integers(0, n_chunks - 1)))
    return sorted(picks)[:count - 1] + [n_chunks - 1]    # the ragged last chunk stays last


def _run(wl, steps, check_at, n_sample=40, algorithm="alg1", grad_dtype=torch.float32):
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    need = (5 * wl.W + 6) * wl.n * 4
    if free < need * 1.03:
        pytest.skip(f"needs {need / 1e9:.0f} GB of device memory, {free / 1e9:.0f} GB free")
    chunks = _sample_chunks(wl, n_sample, 7)
    spans = [(c * wl.chunk, min((c + 1) * wl.chunk, wl.n)) for c in chunks]
    idx = torch.cat([torch.arange(a, b, device="cuda") for a, b in spans])
    d = idx.numel()
    stream = synth.GradientStream(wl, "cuda")
    x0 = synth.initial_params(wl, "cuda")
    cpu = zo.Oracle(d, wl.W, wl.chunk, wl.beta1, wl.beta2, wl.eps, dtype=np.float32)
    cpu.set_params(x0[idx].cpu().numpy())
    gpu = Zoa(wl.n, wl.W, wl.beta1, wl.beta2, wl.eps, wl.chunk)
    try:
        gpu.set_params(x0)
        del x0
        gpu.set_policies(wl.var_steps, wl.sync_boundaries, wl.sync_intervals)
        gpu.set_grad_dtype(grad_dtype)
        g16 = None if grad_dtype == torch.float32 else [torch.empty(wl.n, device="cuda", dtype=grad_dtype) for _ in range(wl.W)]

        def gather(name, worker=0):
            return np.concatenate([gpu.read(name, worker, a, b - a) for a, b in spans])

        for t in range(steps):
            bufs = stream.fill(t)
            if g16 is not None:                       # the oracle gets the binary32 values of the 16-bit numbers
                for dst, src in zip(g16, bufs):
                    dst.copy_(src)
                bufs = g16
            g = np.stack([b[idx].float().cpu().numpy() for b in bufs])
            if algorithm == "alg2":
                gpu.alg2_step(bufs, wl.lr_at(t), t)
                cpu.alg2_step(g, np.float32(wl.lr_at(t)), wl.in_T_v(t))
            else:
                if algorithm == "two_call":
                    gpu.step(bufs, wl.lr_at(t), t)
                    if wl.in_T_u(t):
                        gpu.onebit_reduce()
                else:
                    gpu.step_auto(bufs, wl.lr_at(t), t)
                assert cpu.step(g, np.float32(wl.lr_at(t)), t, wl.in_T_u(t), wl.in_T_v(t)) == 0
            if t in check_at:
                torch.cuda.synchronize()
                for i in range(wl.W):
                    assert_close(gather("x", i), cpu.x[i], f"t={t} x[{i}]")
                    assert_close(gather("m", i), cpu.m[i], f"t={t} m[{i}]")
                    assert_close(gather("u", i), cpu.u[i], f"t={t} u[{i}]")
                    assert_close(gather("delta_w", i), cpu.delta[i], f"t={t} delta_w[{i}]")
                assert_close(gather("v"), cpu.v, f"t={t} v")
                assert_close(gather("delta_s"), cpu.delta_bar, f"t={t} delta_s")
                assert_close(gather("x_sync"), cpu.x_sync, f"t={t} x_sync")
                if wl.in_T_u(t) and algorithm != "alg2":
                    # packed words, bit-exact: oracle word k of sampled chunk j <-> GPU word (start_j/32 + k)
                    per = wl.chunk // 32
                    for j, (a, b) in enumerate(spans):
                        nw = -(-(b - a) // 32)
                        for i in (0, wl.W - 1):
                            assert np.array_equal(gpu.read("words_w", i, a // 32, nw),
                                                  cpu.words_worker[i][j * per:j * per + nw]), (t, j, i)
                        assert np.array_equal(gpu.read("words_s", 0, a // 32, nw),
                                              cpu.words_server[j * per:j * per + nw]), (t, j)
                    got = np.array([gpu.read("scales_s", 0, c, 1)[0] for c in chunks])
                    assert_close(got, cpu.scales_server, f"t={t} scales_s")
        gpu.check_device()
    finally:
        gpu.close()
        del stream
        torch.cuda.empty_cache()


def test_bert_large_full_size_sampled_chunks():
    """336,226,108 parameters, W = 16, chunk 4096, all 100 steps of the schedule."""
    _run(synth.bert_large(), 100, {0, 1, 2, 5, 17, 33, 63, 64, 65, 66, 67, 99})


def test_gpt2_full_size_sampled_chunks():
    """1,557,611,200 parameters, W = 4, chunk 8192, Student-t noise; all 50 steps of the schedule."""
    _run(synth.gpt2_xl(), 50, {0, 3, 15, 16, 17, 19, 20, 21, 32, 33, 36, 47, 48, 49}, n_sample=24)


def test_bert_base_full_size_sampled_chunks():
    """110,106,428 parameters, W = 8, chunk 4096, all 200 steps of the schedule (sync every step,
    every second, every fourth)."""
    _run(synth.bert_base(), 200, {0, 1, 2, 31, 63, 64, 65, 66, 127, 128, 129, 130, 131, 132, 199})


def test_bert_large_full_size_algorithm_2():
    """The configuration `bench.py --algorithm alg2` times: full-precision steps on T_v, compressed
    gradients through the ring kernel otherwise; first 20 steps."""
    _run(synth.bert_large(), 20, {0, 1, 2, 3, 4, 5, 8, 9, 16, 17, 19}, n_sample=24, algorithm="alg2")


def test_bert_large_full_size_bfloat16_gradients():
    """The configuration `bench.py --grad-dtype bf16` times; first 12 steps and two local steps."""
    wl = synth.bert_large()
    wl.sync_boundaries, wl.sync_intervals = (0, 8), (1, 2)
    _run(wl, 12, {0, 1, 2, 7, 8, 9, 10, 11}, n_sample=24, grad_dtype=torch.bfloat16)


def test_bert_large_full_size_two_call_path():
    """The configuration `bench.py --two-call` times: zoa_step, then zoa_onebit_reduce on sync steps."""
    wl = synth.bert_large()
    wl.sync_boundaries, wl.sync_intervals = (0, 4), (1, 2)
    _run(wl, 8, {0, 1, 3, 4, 5, 6, 7}, n_sample=24, algorithm="two_call")


def test_bert_large_full_size_whole_vector_properties():
    """What must hold for every coordinate after a sync step, checked over the whole vector with
    plain torch operations (no sampling): all workers hold the same model, equal to x_sync; the
    buffer is zero; the momentum is +-(server magnitude of the chunk) / (sum of learning rates)
    with the sign the server's packed word carries; rows end in zero padding."""
    wl = synth.bert_large()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < (5 * wl.W + 8) * wl.n * 4 * 1.03:
        pytest.skip("not enough device memory")
    stream = synth.GradientStream(wl, "cuda")
    gpu = Zoa(wl.n, wl.W, wl.beta1, wl.beta2, wl.eps, wl.chunk)
    try:
        gpu.set_params(synth.initial_params(wl, "cuda"))
        gpu.set_policies(wl.var_steps, (0, 2), (1, 2))
        lrs = [1e-3, 5e-4, 2.5e-4, 1e-3, 7e-4]
        for t in range(5):                                      # sync at 0, 1, 2, 4; local at 3: the last sync spans two steps
            gpu.step_auto(stream.fill(t), lrs[t], t)
        torch.cuda.synchronize()
        n, chunk = wl.n, wl.chunk
        gamma_sum = np.float32(np.float64(np.float32(lrs[3])) + np.float64(np.float32(lrs[4])))
        x_sync = gpu.device_view("x_sync")
        words = gpu.device_view("words_s")
        scales = gpu.device_view("scales_s")
        n_chunks = -(-n // chunk)
        m_mag = scales[:n_chunks] / torch.tensor(gamma_sum, device="cuda")          # one IEEE division per chunk
        for i in range(wl.W):
            assert torch.equal(gpu.device_view("x", i), x_sync), f"x[{i}] differs from x_sync"
            assert not gpu.device_view("u", i).any(), f"u[{i}] is not zero"
        shifts = torch.arange(32, device="cuda", dtype=torch.int32)
        span = 1 << 24                                          # coordinates per slice, a multiple of the chunk size
        for lo in range(0, n, span):
            hi = min(lo + span, n)
            w = words[lo // 32:(hi + 31) // 32]
            bits = ((w[:, None] >> shifts[None, :]) & 1).reshape(-1)[:hi - lo].bool()
            mag = m_mag[lo // chunk:(hi + chunk - 1) // chunk].repeat_interleave(chunk)[:hi - lo]
            want = torch.where(bits, mag, -mag)
            for i in (0, wl.W // 2, wl.W - 1):
                assert torch.equal(gpu.device_view("m", i)[lo:hi], want), f"m[{i}] in [{lo}, {hi})"
        pad = (-n) % 128
        if pad:
            for name in ("x", "m", "u", "delta_w"):
                assert not gpu.device_view(name, wl.W - 1)[n:n + pad].any()
        gpu.check_device()
    finally:
        gpu.close()
        del stream
        torch.cuda.empty_cache()


def _unpack(words, count):
    shifts = torch.arange(32, device=words.device, dtype=torch.int32)
    return ((words[:, None] >> shifts[None, :]) & 1).reshape(-1)[:count].bool()


def _every_coordinate_against_torch_arithmetic(wl):
    """Four sync steps and a local step (the last sync spans two learning rates), every coordinate
    of every worker:
    the step is worked out again from the state before it with plain torch operations (one IEEE
    binary32 operation each, binary64 for the three reductions) and compared exactly; only the
    per-chunk magnitudes get one unit in the last place, since a binary64 sum taken in another
    order may round to the neighbouring binary32 value."""
    n, W, chunk = wl.n, wl.W, wl.chunk
    n_chunks, n_full = -(-n // chunk), n // chunk
    f32 = lambda v: float(np.float32(v))
    b1, b2, eps = f32(wl.beta1), f32(wl.beta2), f32(wl.eps)
    ob1, ob2 = f32(np.float32(1) - np.float32(wl.beta1)), f32(np.float32(1) - np.float32(wl.beta2))
    stream = synth.GradientStream(wl, "cuda")
    gpu = Zoa(n, W, wl.beta1, wl.beta2, wl.eps, chunk)

    def chunk_l1_scale(z):
        """Eq. 3 magnitudes of a whole row: binary64 sums per chunk, one rounding."""
        a = z[:n].abs().double()
        s = a[:n_full * chunk].view(n_full, chunk).sum(1) / chunk
        if n_chunks > n_full:
            s = torch.cat([s, (a[n_full * chunk:].sum() / (n - n_full * chunk)).reshape(1)])
        return s.float()

    def per_coordinate(scales):
        return scales.repeat_interleave(chunk)[:n]

    def close_to_one_ulp(got, want, what):
        bad = ~torch.isclose(got, want, rtol=1.3e-7, atol=0.0)
        assert not bad.any(), f"{what}: {int(bad.sum())} magnitudes differ by more than one unit in the last place"

    try:
        gpu.set_params(synth.initial_params(wl, "cuda"))
        gpu.set_policies((0, 1), (0, 2), (1, 2))                  # sync at t = 0, 1, 2, 4; t = 3 is a local step
        lrs = [1e-3, 5e-4, 2e-3, 7e-4, 1e-3]
        for t, lr in enumerate(lrs):
            gamma = f32(lr)
            before = {k: [gpu.device_view(k, i).clone() for i in range(W)] for k in ("m", "u", "delta_w")}
            ds_old, xs_old = gpu.device_view("delta_s").clone(), gpu.device_view("x_sync").clone()
            v_old = gpu.device_view("v").clone()
            x_old = [gpu.device_view("x", i).clone() for i in range(W)] if t == 3 else None
            g = stream.fill(t)
            gpu.step_auto(g, lr, t)
            torch.cuda.synchronize()

            if t == 3:                                                # local step: momentum, model and buffer updates
                den = (v_old[:n] + eps).sqrt()
                for i in range(W):
                    m_half = before["m"][i][:n] * b1 + g[i] * ob1
                    step = m_half * gamma
                    assert torch.equal(gpu.device_view("m", i)[:n], m_half), f"t={t} m[{i}]"
                    assert torch.equal(gpu.device_view("x", i)[:n], x_old[i][:n] - step / den), f"t={t} x[{i}]"
                    assert torch.equal(gpu.device_view("u", i)[:n], before["u"][i][:n] + step), f"t={t} u[{i}]"
                    assert torch.equal(gpu.device_view("delta_w", i), before["delta_w"][i]), f"t={t} delta_w[{i}]"
                assert torch.equal(gpu.device_view("delta_s"), ds_old) and torch.equal(gpu.device_view("x_sync"), xs_old)
                assert torch.equal(gpu.device_view("v"), v_old)
                del before, x_old, den
                continue
            # sum of the learning rates since the last sync: binary64 sum of the binary32 values, rounded once
            gamma_sum = f32(np.float64(np.float32(lrs[3])) + np.float64(np.float32(lrs[4]))) if t == 4 else gamma

            A = torch.zeros(n, dtype=torch.float64, device="cuda")
            for i in range(W):
                m_half = before["m"][i][:n] * b1 + g[i] * ob1                      # momentum update
                z = (before["u"][i][:n] + m_half * gamma) + before["delta_w"][i][:n]
                s_gpu = gpu.device_view("scales_w", i)[:n_chunks]
                close_to_one_ulp(s_gpu, chunk_l1_scale(z), f"t={t} scales_w[{i}]")
                bits = z >= 0
                assert torch.equal(_unpack(gpu.device_view("words_w", i), n), bits), f"t={t} words_w[{i}]"
                s = per_coordinate(s_gpu)
                z_hat = torch.where(bits, s, -s)
                assert torch.equal(gpu.device_view("delta_w", i)[:n], z - z_hat), f"t={t} delta_w[{i}]"
                A += z_hat.double()                                                 # worker order; exact in binary64
                del m_half, z, bits, s, z_hat
            a = (A / torch.tensor(float(W), dtype=torch.float64, device="cuda") + ds_old[:n].double()).float()
            del A
            s_gpu = gpu.device_view("scales_s")[:n_chunks]
            close_to_one_ulp(s_gpu, chunk_l1_scale(a), f"t={t} scales_s")
            bits = a >= 0
            assert torch.equal(_unpack(gpu.device_view("words_s"), n), bits), f"t={t} words_s"
            s = per_coordinate(s_gpu)
            z_bar = torch.where(bits, s, -s)
            assert torch.equal(gpu.device_view("delta_s")[:n], a - z_bar), f"t={t} delta_s"
            x_new = xs_old[:n] - z_bar / (v_old[:n] + eps).sqrt()                    # model sync, with v_t
            # momentum approximation; a tensor divisor, because torch
            # turns division by a Python scalar into a multiplication by its reciprocal
            m_new = z_bar / torch.tensor(gamma_sum, device="cuda")
            assert torch.equal(gpu.device_view("x_sync")[:n], x_new), f"t={t} x_sync"
            for i in range(W):
                assert torch.equal(gpu.device_view("x", i)[:n], x_new), f"t={t} x[{i}]"
                assert torch.equal(gpu.device_view("m", i)[:n], m_new), f"t={t} m[{i}]"
                assert not gpu.device_view("u", i).any(), f"t={t} u[{i}]"
            if t in (0, 1):                                                           # variance update, effective from the next step
                G = torch.zeros(n, dtype=torch.float64, device="cuda")
                for i in range(W):
                    G += g[i].double()
                g_bar = (G / torch.tensor(float(W), dtype=torch.float64, device="cuda")).float()
                assert torch.equal(gpu.device_view("v")[:n], v_old[:n] * b2 + (g_bar * g_bar) * ob2), f"t={t} v"
            else:
                assert torch.equal(gpu.device_view("v"), v_old), f"t={t} v changed outside T_v"
            del before, a, bits, s, z_bar, x_new, m_new
        gpu.check_device()
    finally:
        gpu.close()
        del stream
        torch.cuda.empty_cache()


def test_bert_base_full_size_every_coordinate_against_torch_arithmetic():
    _every_coordinate_against_torch_arithmetic(synth.bert_base())


def test_gpt2_shaped_every_coordinate_against_torch_arithmetic():
    """The GPT-2-shaped layout shrunk 8x (194,701,400 parameters, W = 4, chunk 8192, Student-t noise):
    the four-tile ring kernel, with and without the fused variance update."""
    _every_coordinate_against_torch_arithmetic(synth.scaled(synth.gpt2_xl(), 8))


def test_bert_base_full_size_algorithm_2_every_coordinate_against_torch_arithmetic():
    """Algorithm 2 on the BERT-Base-shaped configuration: two full-precision steps (T_v) and two
    compressed ones, every coordinate of every worker worked out again with plain torch operations."""
    wl = synth.bert_base()
    n, W, chunk = wl.n, wl.W, wl.chunk
    n_chunks, n_full = -(-n // chunk), n // chunk
    f32 = lambda v: float(np.float32(v))
    b1, b2, eps = f32(wl.beta1), f32(wl.beta2), f32(wl.eps)
    ob1, ob2 = f32(np.float32(1) - np.float32(wl.beta1)), f32(np.float32(1) - np.float32(wl.beta2))
    W64 = torch.tensor(float(W), dtype=torch.float64, device="cuda")
    stream = synth.GradientStream(wl, "cuda")
    gpu = Zoa(n, W, wl.beta1, wl.beta2, wl.eps, chunk)

    def chunk_l1_scale(z):
        a = z[:n].abs().double()
        s = a[:n_full * chunk].view(n_full, chunk).sum(1) / chunk
        if n_chunks > n_full:
            s = torch.cat([s, (a[n_full * chunk:].sum() / (n - n_full * chunk)).reshape(1)])
        return s.float()

    def one_ulp(got, want, what):
        bad = ~torch.isclose(got, want, rtol=1.3e-7, atol=0.0)
        assert not bad.any(), f"{what}: {int(bad.sum())} magnitudes differ by more than one unit in the last place"

    try:
        gpu.set_params(synth.initial_params(wl, "cuda"))
        gpu.set_policies((0, 1), (0,), (1,))
        for t, lr in enumerate([1e-3, 5e-4, 2e-3, 1e-3]):
            gamma = f32(lr)
            m_old = [gpu.device_view("m", i).clone() for i in range(W)]
            x_old = [gpu.device_view("x", i).clone() for i in range(W)]
            d_old = [gpu.device_view("delta_w", i).clone() for i in range(W)]
            ds_old, v_old = gpu.device_view("delta_s").clone(), gpu.device_view("v").clone()
            g = stream.fill(t)
            gpu.alg2_step(g, lr, t)
            torch.cuda.synchronize()
            den = (v_old[:n] + eps).sqrt()
            if t < 2:                                      # full-precision exchange, then the variance
                G = torch.zeros(n, dtype=torch.float64, device="cuda")
                for i in range(W):
                    G += g[i].double()
                g_bar = (G / W64).float()
                assert torch.equal(gpu.device_view("v")[:n], v_old[:n] * b2 + (g_bar * g_bar) * ob2), f"t={t} v"
                for i in range(W):
                    assert torch.equal(gpu.device_view("delta_w", i), d_old[i]), f"t={t} delta_w[{i}]"
                assert torch.equal(gpu.device_view("delta_s"), ds_old), f"t={t} delta_s"
            else:                                          # gradients through the 1-bit AllReduce
                A = torch.zeros(n, dtype=torch.float64, device="cuda")
                for i in range(W):
                    z = g[i] + d_old[i][:n]
                    s_gpu = gpu.device_view("scales_w", i)[:n_chunks]
                    one_ulp(s_gpu, chunk_l1_scale(z), f"t={t} scales_w[{i}]")
                    bits = z >= 0
                    assert torch.equal(_unpack(gpu.device_view("words_w", i), n), bits), f"t={t} words_w[{i}]"
                    s = s_gpu.repeat_interleave(chunk)[:n]
                    z_hat = torch.where(bits, s, -s)
                    assert torch.equal(gpu.device_view("delta_w", i)[:n], z - z_hat), f"t={t} delta_w[{i}]"
                    A += z_hat.double()
                    del z, bits, s, z_hat
                a = (A / W64 + ds_old[:n].double()).float()
                s_gpu = gpu.device_view("scales_s")[:n_chunks]
                one_ulp(s_gpu, chunk_l1_scale(a), f"t={t} scales_s")
                bits = a >= 0
                assert torch.equal(_unpack(gpu.device_view("words_s"), n), bits), f"t={t} words_s"
                s = s_gpu.repeat_interleave(chunk)[:n]
                g_bar = torch.where(bits, s, -s)
                assert torch.equal(gpu.device_view("delta_s")[:n], a - g_bar), f"t={t} delta_s"
                assert torch.equal(gpu.device_view("v"), v_old), f"t={t} v changed outside T_v"
                del A, a, bits, s
            for i in range(W):
                m_new = m_old[i][:n] * b1 + g_bar * ob1
                assert torch.equal(gpu.device_view("m", i)[:n], m_new), f"t={t} m[{i}]"
                assert torch.equal(gpu.device_view("x", i)[:n], x_old[i][:n] - (m_new * gamma) / den), f"t={t} x[{i}]"
            del m_old, x_old, d_old, g_bar, den
        gpu.check_device()
    finally:
        gpu.close()
        del stream
        torch.cuda.empty_cache()
