"""Pins for the CPU oracle: each test checks it against something the paper or
the mathematics fixes by another route (hand-worked values, closed forms,
invariants, library routines, brute force), never against a re-typing of the
oracle's own loops."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import zoa_oracle as zo

DTYPES = [np.float32, np.float64]


def _load(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return json.load(f)


# --------------------------------------------------------------------------
# Eq. 3: the compressor
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", DTYPES)
def test_compress_hand_worked(golden_dir, dtype):
    fx = _load(golden_dir, "compress_worked.json")
    a = np.array(fx["a"], dtype)
    a_hat, words, scales = zo.compress(a, fx["chunk"])
    assert np.array_equal(a_hat, np.array(fx["a_hat"], dtype))
    assert np.array_equal(a - a_hat, np.array(fx["error"], dtype))
    assert np.array_equal(scales, np.array(fx["scales"], dtype))
    assert words.tolist() == fx["words"]


@pytest.mark.parametrize("d,chunk", [(1, 32), (31, 32), (33, 32), (4096, 1024), (5000, 2048), (777, 4096)])
def test_compress_invariants(d, chunk):
    rng = np.random.default_rng(d * 7 + chunk)
    a = rng.standard_normal(d)
    a[rng.random(d) < 0.01] *= 100.0
    a_hat, words, scales = zo.compress(a, chunk)
    err = a - a_hat
    # what was sent plus what was kept is the input
    np.testing.assert_allclose(a_hat + err, a, rtol=0, atol=1e-15 * np.abs(a).max())
    # compression keeps the sign pattern
    assert np.array_equal(a_hat >= 0, a >= 0)
    for c, c0 in enumerate(range(0, d, chunk)):
        sl = slice(c0, min(c0 + chunk, d))
        ln = sl.stop - sl.start
        # one magnitude per chunk, and it preserves the chunk's l1 norm (tail uses its true length)
        assert np.all(np.abs(a_hat[sl]) == scales[c])
        assert math.isclose(np.abs(a_hat[sl]).sum(), math.fsum(np.abs(a[sl])), rel_tol=1e-12)
        # closed form of the error energy: |a|_2^2 - |a|_1^2 / len
        closed = math.fsum(a[sl] ** 2) - math.fsum(np.abs(a[sl])) ** 2 / ln
        assert math.isclose(math.fsum(err[sl] ** 2), closed, rel_tol=1e-9, abs_tol=1e-12)
    # wire layout equals numpy's little-endian bit packing of (a >= 0)
    packed = np.packbits((a >= 0).astype(np.uint8), bitorder="little")
    packed = np.concatenate([packed, np.zeros((-packed.size) % 4, np.uint8)]).view("<u4")
    assert np.array_equal(words, packed)


def test_compress_scale_minimises_l2_error_brute_force():
    """Among all a_hat = s * sign(a) the mean |a| is the least-squares magnitude:
    scan s on a fine grid and check nothing beats the oracle's scale."""
    rng = np.random.default_rng(5)
    for _ in range(20):
        a = rng.standard_normal(16) * rng.lognormal()
        a_hat, _, scales = zo.compress(a, 16)
        best = ((a - a_hat) ** 2).sum()
        sgn = np.where(a >= 0, 1.0, -1.0)
        grid = np.linspace(0.0, 2.5 * np.abs(a).max(), 20001)
        errs = ((a[None, :] - grid[:, None] * sgn[None, :]) ** 2).sum(axis=1)
        assert best <= errs.min() + 1e-12
        assert abs(grid[errs.argmin()] - scales[0]) <= grid[1] - grid[0]


def test_compress_gaussian_error_ratio():
    """For i.i.d. N(0,1) input, |C[a] - a|^2 / |a|^2 -> 1 - 2/pi (E|a| = sqrt(2/pi))."""
    a = np.random.default_rng(11).standard_normal(1 << 20)
    a_hat, _, _ = zo.compress(a, 4096)
    ratio = ((a - a_hat) ** 2).sum() / (a ** 2).sum()
    assert abs(ratio - (1 - 2 / math.pi)) < 3e-3


def test_compress_whole_vector_when_chunk_covers_it():
    a = np.random.default_rng(3).standard_normal(1000)
    a_hat, _, scales = zo.compress(a, 4096)
    assert scales.size == 1
    assert math.isclose(scales[0], np.linalg.norm(a, 1) / a.size, rel_tol=1e-14)
    assert np.array_equal(np.sign(a_hat), np.sign(a))


@pytest.mark.parametrize("dtype", DTYPES)
def test_compress_special_values(dtype):
    a = np.array([0.0, -0.0, np.nan, -1.0] + [1.0] * 28, dtype)
    with np.errstate(invalid="ignore"):
        a_hat, words, _ = zo.compress(a, 32)
    assert words[0] & 0xF == 0b0011          # +0 and -0 -> 1, NaN and negatives -> 0
    zeros = np.zeros(64, dtype)
    a_hat, words, scales = zo.compress(zeros, 32)
    assert scales.tolist() == [0.0, 0.0] and words.tolist() == [0xFFFFFFFF] * 2
    assert np.all(a_hat == 0)


def test_allreduce_is_the_mean():
    g = np.random.default_rng(2).standard_normal((5, 1000))
    np.testing.assert_allclose(zo.allreduce(g), g.mean(axis=0), rtol=1e-15, atol=1e-16)
    g32 = g.astype(np.float32)
    np.testing.assert_array_equal(zo.allreduce(g32), g32.astype(np.float64).mean(axis=0).astype(np.float32))


# --------------------------------------------------------------------------
# Algorithm 3: error-feedback 1-bit AllReduce
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", DTYPES)
def test_onebit_allreduce_hand_worked(golden_dir, dtype):
    fx = _load(golden_dir, "onebit_allreduce_worked.json")
    z = np.array(fx["z"], dtype)
    o = zo.Oracle(d=z.shape[1], n=z.shape[0], chunk=fx["chunk"], dtype=dtype)
    for r in fx["rounds"]:
        z_bar = o.onebit_allreduce(z)
        assert np.array_equal(z_bar, np.array(r["z_bar"], dtype))
        assert np.array_equal(o.delta, np.array(r["delta"], dtype))
        assert np.array_equal(o.delta_bar, np.array(r["delta_bar"], dtype))
        assert o.scales_worker[:, 0].tolist() == r["scales_worker"]
        assert o.words_worker[:, 0].tolist() == r["words_worker"]
        assert o.scales_server[0] == r["scale_server"] and o.words_server[0] == r["word_server"]


def test_onebit_allreduce_telescopes():
    """Error feedback delays mass, it never loses it: over any number of rounds
    sum_r z_bar_r = sum_r mean_i z_r^(i) - (mean_i delta^(i) + delta_bar) at the end."""
    rng = np.random.default_rng(8)
    n, d, chunk = 3, 700, 256
    o = zo.Oracle(d, n, chunk, dtype=np.float64)
    sent, received = np.zeros(d), np.zeros(d)
    for r in range(12):
        z = rng.standard_normal((n, d)) * (1 + r % 3)
        d_before = o.delta.mean(axis=0) + o.delta_bar
        z_bar = o.onebit_allreduce(z)
        d_after = o.delta.mean(axis=0) + o.delta_bar
        # per round: z_bar = mean z + (errors before) - (errors after)
        np.testing.assert_allclose(z_bar, z.mean(axis=0) + d_before - d_after, rtol=0, atol=1e-13)
        sent += z.mean(axis=0)
        received += z_bar
    np.testing.assert_allclose(received, sent - (o.delta.mean(axis=0) + o.delta_bar), rtol=0, atol=1e-12)
    # the errors stay bounded by a few scales (no drift)
    assert np.abs(o.delta).max() < 50 and np.abs(o.delta_bar).max() < 50


def test_onebit_allreduce_worker_permutation():
    rng = np.random.default_rng(9)
    n, d = 4, 300
    z = rng.standard_normal((n, d)).astype(np.float32)
    perm = np.array([2, 0, 3, 1])
    a, b = zo.Oracle(d, n, 128), zo.Oracle(d, n, 128)
    for _ in range(3):
        za = a.onebit_allreduce(z)
        zb = b.onebit_allreduce(z[perm])
        assert np.array_equal(za, zb)
        assert np.array_equal(a.delta[perm], b.delta)
        assert np.array_equal(a.delta_bar, b.delta_bar)


# --------------------------------------------------------------------------
# Algorithm 1
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", DTYPES)
def test_alg1_hand_worked(golden_dir, dtype):
    fx = _load(golden_dir, "alg1_worked.json")
    o = zo.Oracle(d=4, n=2, chunk=fx["chunk"], beta1=fx["beta1"], beta2=fx["beta2"], eps=fx["eps"], dtype=dtype)
    o.set_params(fx["x0"])
    tol = dict(rtol=0, atol=5e-7 if dtype == np.float32 else 1e-15)

    def check(want):
        for key, val in want.items():
            if key in ("x", "m", "u", "delta", "delta_bar", "v"):
                np.testing.assert_allclose(getattr(o, key), np.array(val, dtype), err_msg=key, **tol)
        if "scales_worker" in want:
            assert o.scales_worker[:, 0].tolist() == want["scales_worker"]
            assert o.words_worker[:, 0].tolist() == want["words_worker"]
            assert o.scales_server[0] == want["scale_server"] and o.words_server[0] == want["word_server"]

    for s in fx["steps"]:
        g = np.array(s["g"], dtype)
        if "half" in s:   # split form, to see the half-step values
            o.half_step(g, s["gamma"])
            check(s["half"])
            if s["in_T_u"]:
                assert o.sync(s["t"]) == 0
            if s["in_T_v"]:
                o.variance(g)
        else:
            assert o.step(g, s["gamma"], s["t"], s["in_T_u"], s["in_T_v"]) == 0
        check(s["end"])


def _adam_closed_form(g_bar, gammas, beta1, beta2, eps, x0):
    """Unrolled Adam recurrences (Eq. 2 in its distributed form, stale v, no bias
    correction): m_{t+1} = (1-b1) sum_k b1^(t-k) g_k, v likewise with squares,
    x_T = x_0 - sum_t gamma_t m_{t+1} / sqrt(v_t + eps)."""
    T = len(gammas)
    k = np.arange(T)
    lower = np.tril(np.ones((T, T)))
    w1 = (1 - beta1) * beta1 ** np.clip(k[:, None] - k[None, :], 0, None) * lower
    w2 = (1 - beta2) * beta2 ** np.clip(k[:, None] - k[None, :], 0, None) * lower
    m_after = w1 @ g_bar                      # row t: m_{t+1}
    v_after = w2 @ g_bar ** 2                 # row t: v_{t+1}
    v_used = np.vstack([np.zeros_like(g_bar[:1]), v_after[:-1]])   # row t: v_t
    x = x0 - (np.asarray(gammas)[:, None] * m_after / np.sqrt(v_used + eps)).sum(axis=0)
    return x, m_after[-1], v_after[-1]


def test_alg1_reduces_to_adam():
    """T_u = T_v = every step with the identity compressor is distributed Adam."""
    rng = np.random.default_rng(21)
    n, d, T = 3, 40, 25
    beta1, beta2, eps = 0.9, 0.999, 1e-8
    g = rng.standard_normal((T, n, d))
    gammas = 1e-3 * (1 + 0.1 * np.arange(T))
    x0 = rng.standard_normal(d) * 0.02
    o = zo.Oracle(d, n, 16, beta1, beta2, eps, dtype=np.float64, compressor=zo.IDENTITY)
    o.set_params(x0)
    for t in range(T):
        assert o.step(g[t], gammas[t], t, True, True) == 0
    x, m, v = _adam_closed_form(g.mean(axis=1), gammas, beta1, beta2, eps, x0)
    for i in range(n):
        np.testing.assert_allclose(o.x[i], x, rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(o.m[i], m, rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(o.v, v, rtol=1e-11)
    # the float build follows the same trajectory to float accuracy
    o32 = zo.Oracle(d, n, 16, beta1, beta2, eps, dtype=np.float32, compressor=zo.IDENTITY)
    o32.set_params(x0)
    for t in range(T):
        o32.step(g[t].astype(np.float32), gammas[t], t, True, True)
    np.testing.assert_allclose(o32.x[0], x, rtol=2e-4, atol=2e-5)
    np.testing.assert_allclose(o32.v, v, rtol=1e-4)


def test_alg1_identical_workers_equal_one_worker():
    rng = np.random.default_rng(22)
    d, T = 200, 9
    g = rng.standard_normal((T, 1, d)).astype(np.float32)
    x0 = rng.standard_normal(d).astype(np.float32)
    one, four = zo.Oracle(d, 1, 64), zo.Oracle(d, 4, 64)
    one.set_params(x0), four.set_params(x0)
    for t in range(T):
        one.step(g[t], 1e-3, t, t % 2 == 0, t < 4)
        four.step(np.repeat(g[t], 4, axis=0), 1e-3, t, t % 2 == 0, t < 4)
    for i in range(4):
        assert np.array_equal(four.x[i], one.x[0]) and np.array_equal(four.m[i], one.m[0])
    assert np.array_equal(four.v, one.v)


def test_alg1_frozen_variance_is_momentum_sgd():
    """With T_v empty the denominator is the constant sqrt(eps): the method is
    momentum SGD with dampening, which torch.optim.SGD implements."""
    rng = np.random.default_rng(23)
    n, d, T = 2, 30, 12
    beta1, eps, gamma = 0.9, 1e-4, 1e-3
    g = rng.standard_normal((T, n, d))
    g[0] = 0.0        # torch seeds its momentum buffer with the first gradient undamped
    x0 = rng.standard_normal(d)
    o = zo.Oracle(d, n, 16, beta1, 0.999, eps, dtype=np.float64, compressor=zo.IDENTITY)
    o.set_params(x0)
    p = torch.tensor(x0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=gamma / math.sqrt(eps), momentum=beta1, dampening=beta1)
    for t in range(T):
        o.step(g[t], gamma, t, True, False)
        p.grad = torch.tensor(g[t].mean(axis=0))
        opt.step()
    np.testing.assert_allclose(o.x[0], p.detach().numpy(), rtol=1e-11, atol=1e-13)
    assert np.all(o.v == 0)


def test_alg1_local_steps_are_linear_in_u():
    """Between two syncs with v frozen, x^(i) = x_{t'} - u^(i) / sqrt(v + eps)."""
    rng = np.random.default_rng(24)
    n, d = 3, 500
    o = zo.Oracle(d, n, 128, dtype=np.float64)
    o.set_params(rng.standard_normal(d) * 0.02)
    t = 0
    for t in range(4):
        o.step(rng.standard_normal((n, d)), 1e-3, t, True, True)
    x_sync = o.x[0].copy()
    gammas = []
    for t in range(4, 9):
        gammas.append(1e-3 * (t - 2))
        o.step(rng.standard_normal((n, d)), gammas[-1], t, False, False)
        for i in range(n):
            np.testing.assert_allclose(o.x[i], x_sync - o.u[i] / np.sqrt(o.v + 1e-8), rtol=1e-9, atol=1e-12)
    assert math.isclose(o.gamma_sum, sum(gammas), rel_tol=1e-15)
    assert o.t_sync == 3
    # after the next sync every worker agrees, u is cleared, and per chunk m takes two values +-scale/sum(gamma)
    total = o.gamma_sum + 2e-3
    o.step(rng.standard_normal((n, d)), 2e-3, 9, True, False)
    assert np.all(o.u == 0) and o.gamma_sum == 0 and o.t_sync == 9
    for i in range(1, n):
        assert np.array_equal(o.x[i], o.x[0]) and np.array_equal(o.m[i], o.m[0])
    assert np.array_equal(o.x_sync, o.x[0])
    for c in range(o.n_chunks):
        sl = slice(c * 128, min((c + 1) * 128, d))
        np.testing.assert_allclose(np.abs(o.m[0][sl]), o.scales_server[c] / total, rtol=1e-14)
        np.testing.assert_allclose(x_sync[sl] - o.x[0][sl], o.u_bar[sl] / np.sqrt(o.v[sl] + 1e-8), rtol=1e-9, atol=1e-15)


def test_alg1_printed_momentum_index_is_degenerate():
    """Taking m_t (from before the momentum update) in the model and buffer updates, as printed, with a sync at every
    step: the gradient never reaches the model.  This is why m_{t+1/2} is used."""
    rng = np.random.default_rng(25)
    o = zo.Oracle(64, 2, 32, dtype=np.float64, compressor=zo.IDENTITY, literal_momentum=True)
    x0 = rng.standard_normal(64)
    o.set_params(x0)
    for t in range(6):
        o.step(rng.standard_normal((2, 64)), 1e-3, t, True, True)
    assert np.array_equal(o.x[0], x0) and np.all(o.m == 0)


def test_alg1_sync_without_accumulation_is_refused():
    o = zo.Oracle(64, 2, 32)
    assert o.sync(0) == -1


@pytest.mark.parametrize("dtype", DTYPES)
def test_alg1_symmetries(dtype):
    """g -> -g, x0 -> -x0 negates every state; g -> 4g with eps -> 16 eps scales
    m, u, the errors by 4 and v by 16 and leaves x untouched (exact in binary)."""
    rng = np.random.default_rng(26)
    n, d, T, chunk = 3, 300, 10, 64
    g = rng.standard_normal((T, n, d)).astype(dtype)
    x0 = (rng.standard_normal(d) * 0.02).astype(dtype)
    T_u = [True, True, False, True, False, False, True, True, False, True]
    T_v = [True, True, False, True, False, False, False, False, False, False]

    def run(scale, sign, eps):
        o = zo.Oracle(d, n, chunk, eps=eps, dtype=dtype)
        o.set_params(sign * x0)
        for t in range(T):
            o.step(sign * scale * g[t], 1e-3, t, T_u[t], T_v[t])
        return o

    base, neg, big = run(1, 1, 2.0 ** -27), run(1, -1, 2.0 ** -27), run(4, 1, 2.0 ** -23)
    for key in ("x", "m", "u", "delta", "delta_bar"):
        assert np.array_equal(getattr(neg, key), -getattr(base, key)), key
    assert np.array_equal(neg.v, base.v)
    assert np.array_equal(big.x, base.x)
    for key in ("m", "u", "delta", "delta_bar"):
        assert np.array_equal(getattr(big, key), 4 * getattr(base, key)), key
    assert np.array_equal(big.v, 16 * base.v)


def test_alg1_variance_bounds():
    """0 <= v <= max g_bar^2, v moves only on T_v steps, and the sync of a step in
    both sets still used the old v (checked through x)."""
    rng = np.random.default_rng(27)
    n, d = 2, 100
    o = zo.Oracle(d, n, 32, dtype=np.float64, compressor=zo.IDENTITY)
    o.set_params(np.zeros(d))
    g_max = 0.0
    for t in range(8):
        g = rng.standard_normal((n, d))
        v_before, x_before = o.v.copy(), o.x[0].copy()
        in_v = t in (0, 1, 2, 4)
        o.step(g, 1e-3, t, True, in_v)
        g_max = max(g_max, (g.mean(axis=0) ** 2).max())
        assert (np.array_equal(o.v, v_before)) != in_v
        assert np.all(o.v >= 0) and o.v.max() <= g_max
        np.testing.assert_allclose(x_before - o.x[0], 1e-3 * o.m[0] / np.sqrt(v_before + 1e-8), rtol=1e-9, atol=1e-15)


# --------------------------------------------------------------------------
# Algorithm 2 (frozen-variance 1-bit framework; 1-bit Adam as a special case)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", DTYPES)
def test_alg2_hand_worked(golden_dir, dtype):
    fx = _load(golden_dir, "alg2_worked.json")
    o = zo.Oracle(d=4, n=2, chunk=fx["chunk"], beta1=fx["beta1"], beta2=fx["beta2"], eps=fx["eps"], dtype=dtype)
    o.set_params(fx["x0"])
    tol = dict(rtol=0, atol=5e-7 if dtype == np.float32 else 1e-15)
    for s in fx["steps"]:
        o.alg2_step(np.array(s["g"], dtype), s["gamma"], s["in_T_v"])
        for i in range(2):
            np.testing.assert_allclose(o.m[i], np.array(s["m"], dtype), **tol)
            np.testing.assert_allclose(o.x[i], np.array(s["x"], dtype), **tol)
        np.testing.assert_allclose(o.v, np.array(s["v"], dtype), **tol)
        np.testing.assert_allclose(o.delta, np.array(s["delta"], dtype), **tol)
        np.testing.assert_allclose(o.delta_bar, np.array(s["delta_bar"], dtype), **tol)


def test_alg2_identity_compressor_is_adam_and_equals_alg1_without_local_steps():
    rng = np.random.default_rng(31)
    n, d, T = 3, 50, 20
    beta1, beta2, eps = 0.9, 0.999, 1e-8
    g = rng.standard_normal((T, n, d))
    gammas = 1e-3 * (1 + 0.05 * np.arange(T))
    x0 = rng.standard_normal(d) * 0.02
    two = zo.Oracle(d, n, 16, beta1, beta2, eps, dtype=np.float64, compressor=zo.IDENTITY)
    one = zo.Oracle(d, n, 16, beta1, beta2, eps, dtype=np.float64, compressor=zo.IDENTITY)
    two.set_params(x0), one.set_params(x0)
    for t in range(T):
        two.alg2_step(g[t], gammas[t], True)
        one.step(g[t], gammas[t], t, True, True)
    x, m, v = _adam_closed_form(g.mean(axis=1), gammas, beta1, beta2, eps, x0)
    np.testing.assert_allclose(two.x[0], x, rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(two.m[0], m, rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(two.v, v, rtol=1e-11)
    np.testing.assert_allclose(two.x, one.x, rtol=1e-9, atol=1e-13)     # Algorithm 1 with a sync at every step
    np.testing.assert_allclose(two.m, one.m, rtol=1e-9, atol=1e-13)


def test_alg2_one_bit_adam_special_case():
    """T_v = the first T0 steps: plain Adam for T0 steps, then the variance is
    frozen, the workers agree, and the received gradients telescope: their sum
    is the sum of the true means minus the errors still held back."""
    rng = np.random.default_rng(32)
    n, d, T0, T = 4, 300, 5, 14
    o = zo.Oracle(d, n, 64, dtype=np.float64)
    x0 = rng.standard_normal(d) * 0.02
    o.set_params(x0)
    g = rng.standard_normal((T, n, d))
    for t in range(T0):
        o.alg2_step(g[t], 1e-3, True)
    x, m, v = _adam_closed_form(g[:T0].mean(axis=1), [1e-3] * T0, 0.9, 0.999, 1e-8, x0)
    np.testing.assert_allclose(o.x[0], x, rtol=1e-10, atol=1e-13)
    assert np.all(o.delta == 0) and np.all(o.delta_bar == 0)
    v_frozen, m_before = o.v.copy(), o.m[0].copy()
    received = np.zeros(d)
    for t in range(T0, T):
        m_prev = o.m[0].copy()
        o.alg2_step(g[t], 1e-3, False)
        assert np.array_equal(o.v, v_frozen)
        received += (o.m[0] - 0.9 * m_prev) / (1 - 0.9)             # the g_bar this step used
        for i in range(1, n):
            assert np.array_equal(o.x[i], o.x[0]) and np.array_equal(o.m[i], o.m[0])
    np.testing.assert_allclose(received, g[T0:].mean(axis=1).sum(axis=0) - (o.delta.mean(axis=0) + o.delta_bar),
                               rtol=0, atol=1e-11)


def test_alg1_minimises_a_noisy_quadratic():
    """Sanity of signs and scales end to end: on f(x) = |x|^2 / 2 with noisy gradients, 0/1 Adam
    with 1-bit syncs and local steps drives the loss down about as far as Adam does (the paper's
    claim is the same convergence rate as Adam)."""
    rng = np.random.default_rng(41)
    n, d, T = 4, 512, 400
    x0 = rng.standard_normal(d)

    def run(compressor, sync_every, var_until):
        # eps = 1 keeps the very first steps, which divide by sqrt(v_0 + eps) with v_0 = 0, well scaled
        o = zo.Oracle(d, n, 128, eps=1.0, dtype=np.float64, compressor=compressor)
        o.set_params(x0)
        for t in range(T):
            g = o.x + 0.3 * rng.standard_normal((n, d))        # gradient of |x|^2/2 at each worker's model, plus noise
            o.step(g, 0.02, t, t % sync_every == 0, t < var_until)
        return 0.5 * float((o.x.mean(axis=0) ** 2).sum())

    f0 = 0.5 * float((x0 ** 2).sum())
    adam = run(zo.IDENTITY, 1, T)
    zero_one = run(zo.ONEBIT, 4, 100)
    assert adam < 0.02 * f0
    assert zero_one < 0.05 * f0
