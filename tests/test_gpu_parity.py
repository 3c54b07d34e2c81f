"""Parity of the CUDA path (through the C ABI) with the CPU oracle on identical
seeded float32 inputs: packed sign words bit-exact, every float32 state within
1e-5 relative (1e-7 absolute near zero), after every step."""
import numpy as np
import pytest
import torch

from helpers import ATOL, RTOL, Pair, assert_close
from oracle import zoa_oracle as zo
from paper_2202_06009_b200 import Zoa, ZoaError, binding as B, synth

pytestmark = pytest.mark.gpu


def _grads(rng, W, n, scale=1.0, outliers=True):
    g = rng.standard_normal((W, n)).astype(np.float32) * np.float32(scale)
    if outliers:
        g[rng.random((W, n)) < 0.01] *= np.float32(100.0)
    return g


SIZES = [1, 31, 32, 33, 127, 128, 129, 2047, 2048, 2049, 3 * 2048 + 17]


@pytest.mark.parametrize("mode", ["fused", "two_call"])
@pytest.mark.parametrize("n", SIZES)
def test_ragged_sizes(n, mode):
    """Sizes around word, tile and chunk boundaries; six steps mixing local, sync and variance steps."""
    rng = np.random.default_rng(n)
    W, chunk = 3, 2048
    p = Pair(n, W, chunk, var_steps=(0, 1, 3), sync=((0, 2), (1, 2)), x0=rng.standard_normal(n) * 0.02)
    try:
        for t in range(6):
            p.step(_grads(rng, W, n), 1e-3 * (1 + t), t, mode)
            p.compare(f"n={n} t={t}")
        p.padding_is_zero()
    finally:
        p.close()


@pytest.mark.parametrize("W,chunk,n", [(1, 32, 1000), (1, 2048, 2048 * 6 + 5), (1, 8192, 8192 * 3), (2, 64, 4096 + 5), (5, 96, 96 * 7 + 3), (4, 1024, 20000),
                                       (8, 4096, 3 * 4096 + 1852), (16, 4096, 2 * 4096 + 77), (4, 8192, 8192 * 2 + 704),
                                       (2, 16384, 16384 * 2 + 100), (64, 256, 1500), (3, 4000, 9000)])
@pytest.mark.parametrize("mode", ["fused", "two_call"])
def test_worker_and_chunk_shapes(W, chunk, n, mode):
    rng = np.random.default_rng(W * 131 + chunk)
    p = Pair(n, W, chunk, var_steps=(0, 2), sync=((0, 3), (1, 2)), x0=rng.standard_normal(n) * 0.02)
    try:
        for t in range(6):
            p.step(_grads(rng, W, n), 1e-3, t, mode)
            p.compare(f"W={W} chunk={chunk} t={t}")
        p.padding_is_zero()
    finally:
        p.close()


def test_fused_equals_two_call_bit_for_bit():
    rng = np.random.default_rng(77)
    n, W, chunk = 5 * 1024 + 333, 4, 1024
    x0 = torch.from_numpy((rng.standard_normal(n) * 0.02).astype(np.float32))
    a, b = Zoa(n, W, chunk=chunk), Zoa(n, W, chunk=chunk)
    try:
        for z in (a, b):
            z.set_params(x0)
            z.set_policies((0, 1, 4), (0, 3), (1, 2))
        for t in range(8):
            g = list(torch.from_numpy(_grads(rng, W, n)).cuda())
            a.step_auto(g, 2e-3, t)
            b.step(g, 2e-3, t)
            if b.sync_due(t):
                b.onebit_reduce()
            torch.cuda.synchronize()
            for name in ("x", "m", "u", "delta_w", "words_w", "scales_w"):
                for i in range(W):
                    assert np.array_equal(a.read(name, i), b.read(name, i)), (name, i, t)
            for name in ("v", "delta_s", "x_sync", "words_s", "scales_s"):
                assert np.array_equal(a.read(name), b.read(name)), (name, t)
        assert a.stats()["n_syncs"] == b.stats()["n_syncs"] == 6
    finally:
        a.close(), b.close()


@pytest.mark.parametrize("W,chunk,n_chunks,tail", [(5, 4096, 301, 1852), (3, 2048, 700, 0), (4, 8192, 160, 704),
                                                   (16, 4096, 40, 5), (64, 2048, 20, 33), (33, 8192, 9, 0),
                                                   (4, 16384, 150, 9000), (3, 1024, 1400, 1500), (5, 512, 2600, 700),
                                                   (2, 256, 5000, 300), (7, 128, 9000, 131), (64, 1024, 41, 0)])
def test_pipelined_kernel_equals_chunk_per_block_kernel(W, chunk, n_chunks, tail):
    """The bulk-copy ring kernel and the chunk-per-block kernel give the same bits,
    over enough chunks that every block wraps its ring many times; steps with and
    without the fused variance update.  Chunks of 2048, 4096 and 8192 coordinates are units of one,
    two and four tiles; chunks of 128 ... 1024 share a tile, and the whole chunks that do not fill
    the last tile go to the chunk-per-block kernel with the ragged tail.  (Chunk 16384 has no ring
    variant: both handles run the chunk-per-block kernel.)"""
    rng = np.random.default_rng(W + chunk)
    n = n_chunks * chunk + tail
    x0 = torch.from_numpy((rng.standard_normal(n) * 0.02).astype(np.float32))
    a, b = Zoa(n, W, chunk=chunk), Zoa(n, W, chunk=chunk)
    try:
        a.set_pipeline("force")
        b.set_pipeline(False)
        for z in (a, b):
            z.set_params(x0)
            z.set_policies((0, 2), (0,), (1,))
        g = torch.empty(W, n, device="cuda")
        for t in range(4):
            g.normal_(generator=torch.Generator("cuda").manual_seed(t + 5))
            a.step_sync(list(g), 1e-3, t)
            b.step_sync(list(g), 1e-3, t)
            torch.cuda.synchronize()
            a.check_device()
            for name in ("x", "m", "u", "delta_w", "words_w", "scales_w"):
                for i in (0, W // 2, W - 1):
                    assert np.array_equal(a.read(name, i), b.read(name, i)), (name, i, t)
            for name in ("v", "delta_s", "x_sync", "words_s", "scales_s"):
                assert np.array_equal(a.read(name), b.read(name)), (name, t)
        if chunk <= 8192 and W <= 16 and not tail and n_chunks % max(1, 2048 // chunk) == 0:      # the variance update rides along in the ring kernel
            assert a.stats()["n_launches"] < b.stats()["n_launches"]
    finally:
        a.close(), b.close()


@pytest.mark.parametrize("W,chunk,n_units,tail", [(5, 4096, 301, 1852), (3, 2048, 700, 0), (4, 8192, 160, 704), (16, 16384, 40, 5),
                                                  (2, 1024, 700, 1500), (7, 512, 650, 700), (3, 256, 620, 100), (64, 128, 610, 3),
                                                  (33, 4096, 20, 0), (64, 2048, 30, 33), (1, 1024, 1300, 1024)])
def test_two_call_ring_kernels_equal_chunk_per_block_kernels(W, chunk, n_units, tail):
    """zoa_step + zoa_onebit_reduce with the compress / server ring kernels (chunks of 128 ... 16384,
    several chunks per tile below 2048, several tiles per chunk above) against the same calls with
    one block or cluster per chunk: same bits, and both within tolerance of the oracle.  The tail
    holds whole chunks that do not fill a unit and a ragged last chunk."""
    rng = np.random.default_rng(W + chunk)
    n = n_units * max(chunk, 2048) + tail
    x0 = (rng.standard_normal(n) * 0.02).astype(np.float32)
    p = Pair(n, W, chunk, var_steps=(0, 2), x0=x0)          # ring kernels forced on
    b = Zoa(n, W, chunk=chunk)
    try:
        b.set_pipeline(False)
        b.set_params(torch.from_numpy(x0))
        b.set_policies((0, 2), (0,), (1,))
        for t in range(3):
            g = (rng.standard_normal((W, n)) * 10.0 ** rng.integers(-2, 2)).astype(np.float32)
            p.step(g, 1e-3, t, "two_call")
            b.step(list(torch.from_numpy(g).cuda()), 1e-3, t)
            b.onebit_reduce()
            torch.cuda.synchronize()
            p.gpu.check_device()
            for name in ("x", "m", "u", "delta_w", "words_w", "scales_w"):
                for i in (0, W // 2, W - 1):
                    assert np.array_equal(p.gpu.read(name, i), b.read(name, i)), (name, i, t)
            for name in ("v", "delta_s", "x_sync", "words_s", "scales_s"):
                assert np.array_equal(p.gpu.read(name), b.read(name)), (name, t)
            p.compare(f"t={t}")
        p.padding_is_zero()
        assert p.gpu.stats()["n_launches"] > b.stats()["n_launches"] or tail == 0      # ring + tail kernels
    finally:
        p.close(), b.close()


@pytest.mark.parametrize("mode", ["fused", "two_call"])
def test_special_values(mode):
    """Signed zeros, subnormals, an all-zero chunk, a chunk of one sign, a lone outlier."""
    W, chunk, n = 2, 64, 64 * 6
    g = np.zeros((W, n), np.float32)
    g[:, 0:64] = 0.0                                   # all-zero chunk: scale 0, every bit 1
    g[0, 64:128] = np.float32(-0.0)
    g[1, 64:128] = np.float32(1e-42)                   # subnormal gradients
    g[:, 128:192] = np.float32(3.0)                    # constant sign
    g[0, 192:256] = np.float32(1e-3); g[0, 200] = np.float32(1e6)   # one outlier dominates the l1 norm
    g[1, 192:256] = np.float32(-1e-3)
    rng = np.random.default_rng(4)
    g[:, 256:] = rng.standard_normal((W, n - 256)).astype(np.float32) * np.float32(1e-20)  # tiny values
    p = Pair(n, W, chunk, var_steps=(0,), x0=np.zeros(n))
    try:
        for t in range(3):
            p.step(g, 1e-3, t, mode)
            p.compare(f"t={t}")
        words = p.gpu.read("words_w", 0)
        assert words[0] == 0xFFFFFFFF and words[1] == 0xFFFFFFFF
    finally:
        p.close()


@pytest.mark.parametrize("seed", [synth.DEFAULT_SEED, 7, 123456789])
def test_tiny_config_full_run(seed):
    """The small configuration in full: 2^20 parameters, W = 4, chunk 2048, 64 steps,
    T_v = {0,1,2,4,8,16}, sync every step until 16 then every other step; every
    state compared after every step; three seeds."""
    wl = synth.tiny()
    stream = synth.GradientStream(wl, "cuda", seed)
    x0 = synth.initial_params(wl, "cuda", seed)
    p = Pair(wl.n, wl.W, wl.chunk, wl.beta1, wl.beta2, wl.eps, wl.var_steps,
             (wl.sync_boundaries, wl.sync_intervals), x0=x0.cpu().numpy())
    try:
        n_sync = 0
        for t in range(wl.steps):
            bufs = stream.fill(t)
            g = torch.stack(bufs).cpu().numpy()
            sync, var = wl.in_T_u(t), wl.in_T_v(t)
            assert p.gpu.sync_due(t) == sync and p.gpu.var_due(t) == var
            p.gpu.step_auto(bufs, wl.lr_at(t), t)
            torch.cuda.synchronize()
            assert p.cpu.step(g, np.float32(wl.lr_at(t)), t, sync, var) == 0
            n_sync += sync
            p.compare(f"t={t}", wire=sync)
        assert n_sync == 40 and p.gpu.stats()["n_syncs"] == 40 and p.gpu.stats()["n_var_updates"] == 6
    finally:
        p.close()


@pytest.mark.parametrize("name,divisor", [("bert_base", 64), ("gpt2_1p5b", 1024)])
def test_shaped_workloads_scaled_down(name, divisor):
    """BERT- and GPT-2-shaped layouts shrunk per tensor (per-tensor lognormal scales,
    Student-t noise for GPT-2), their own policies, first 24 steps."""
    wl = synth.scaled(synth.WORKLOADS[name](), divisor, steps=24)
    stream = synth.GradientStream(wl, "cuda")
    x0 = synth.initial_params(wl, "cuda")
    p = Pair(wl.n, wl.W, wl.chunk, wl.beta1, wl.beta2, wl.eps, wl.var_steps,
             (wl.sync_boundaries, wl.sync_intervals), x0=x0.cpu().numpy())
    try:
        for t in range(wl.steps):
            bufs = stream.fill(t)
            g = torch.stack(bufs).cpu().numpy()
            p.gpu.step_auto(bufs, wl.lr, t)
            torch.cuda.synchronize()
            p.cpu.step(g, np.float32(wl.lr), t, wl.in_T_u(t), wl.in_T_v(t))
            if t % 4 == 3 or t < 3:
                p.compare(f"{name} t={t}", wire=wl.in_T_u(t))
    finally:
        p.close()


@pytest.mark.parametrize("W,chunk", [(2, 1024), (16, 1024), (4, 4096), (8, 16384), (16, 16384)])
def test_sweep_recipe_compress_then_average(W, chunk):
    """The kernel sweep's recipe (N(0,1) with 1 % of the elements x100), through the two
    halves of zoa_onebit_reduce called separately, two rounds so that the second sees
    non-zero errors."""
    rng = np.random.default_rng(W * chunk)
    n = (1 << 20) // 8 + 77
    p = Pair(n, W, chunk, x0=np.zeros(n))
    try:
        for r in range(2):
            z = rng.standard_normal((W, n)).astype(np.float32)
            z[rng.random((W, n)) < 0.01] *= np.float32(100.0)
            for i in range(W):
                p.gpu.write("u", z[i], i)
                p.cpu.u[i] = z[i]
            B.zoa_set_scalars(p.gpu.h, 1e-3, 0, r)
            p.cpu._st.gamma_sum = 1e-3
            p.gpu.onebit_compress()
            p.gpu.onebit_average()
            torch.cuda.synchronize()
            assert p.cpu.sync(r) == 0
            p.compare(f"round {r}")
    finally:
        p.close()


def test_unaligned_gradient_pointers():
    rng = np.random.default_rng(5)
    n, W, chunk = 3000, 2, 1024
    p = Pair(n, W, chunk, var_steps=(0,), sync=((0,), (2,)), x0=rng.standard_normal(n) * 0.02)
    try:
        for t in range(4):
            g = _grads(rng, W, n)
            backing = torch.zeros(W, n + 8, device="cuda")
            views = [backing[i, 1 + i:1 + i + n] for i in range(W)]     # 4- and 8-byte offsets
            for i in range(W):
                views[i].copy_(torch.from_numpy(g[i]))
            assert any(v.data_ptr() % 16 for v in views)
            p.gpu.step_auto(views, 1e-3, t)
            torch.cuda.synchronize()
            p.cpu.step(g, np.float32(1e-3), t, p.gpu.sync_due(t), p.gpu.var_due(t))
            p.compare(f"t={t}", wire=False)
    finally:
        p.close()


@pytest.mark.parametrize("light", [True, False])
@pytest.mark.parametrize("n,W,chunk,offset", [(3 * 1024 + 77, 4, 1024, 0), (5000, 3, 256, 0), (4096 + 9, 2, 4096, 1),
                                              (2 * 16384 + 100, 5, 16384, 0), (40, 1, 32, 3), (7 * 8192, 64, 8192, 0)])
def test_onebit_allreduce_on_caller_buffers(n, W, chunk, offset, light):
    """zoa_onebit_allreduce (Algorithm 3 by itself) against the oracle's zo_onebit_allreduce over three
    rounds, so that non-zero worker and server errors enter; on a handle that holds only Algorithm 3's
    state and on a full one; `offset` shifts the caller's buffers off 16-byte alignment."""
    rng = np.random.default_rng(n + W)
    cpu = zo.Oracle(n, W, chunk, dtype=np.float32)
    gpu = Zoa(n, W, chunk=chunk, allreduce_only=light)
    try:
        for r in range(3):
            z = (rng.standard_normal((W, n)) * 10.0 ** rng.integers(-2, 2)).astype(np.float32)
            z[rng.random((W, n)) < 0.01] *= np.float32(100.0)
            z_dev = [torch.zeros(n + offset, device="cuda")[offset:].copy_(torch.from_numpy(z[i])) for i in range(W)]
            z_bar = torch.full((n + offset + 8,), 7.0, device="cuda")[offset:offset + n]
            if r == 1:          # the two halves separately
                gpu.allreduce_compress(z_dev)
                gpu.allreduce_average(z_bar)
            else:
                gpu.onebit_allreduce(z_dev, z_bar)
            torch.cuda.synchronize()
            want = cpu.onebit_allreduce(z)
            assert_close(z_bar.cpu().numpy(), want, f"z_bar, round {r}")
            assert np.array_equal(gpu.read("words_s"), cpu.words_server), f"words_s, round {r}"
            assert_close(gpu.read("scales_s"), cpu.scales_server, f"scales_s, round {r}")
            assert_close(gpu.read("delta_s"), cpu.delta_bar, f"delta_s, round {r}")
            for i in range(W):
                assert np.array_equal(gpu.read("words_w", i), cpu.words_worker[i]), f"words_w[{i}], round {r}"
                assert_close(gpu.read("scales_w", i), cpu.scales_worker[i], f"scales_w[{i}], round {r}")
                assert_close(gpu.read("delta_w", i), cpu.delta[i], f"delta_w[{i}], round {r}")
                assert np.array_equal(z_dev[i].cpu().numpy(), z[i]), "the input was written"
        gpu.check_device()
        if light:
            g = list(torch.zeros(W, n, device="cuda"))
            for call in (lambda: gpu.step(g, 1e-3, 0), lambda: gpu.step_sync(g, 1e-3, 0), lambda: gpu.alg2_step(g, 1e-3, 0),
                         gpu.onebit_reduce, gpu.export_state, lambda: gpu.read("x")):
                with pytest.raises(ZoaError) as e:
                    call()
                assert e.value.status in (B.ERR_STATE, B.ERR_ARG)
            assert B.zoa_check_finite(gpu.h) == 0
    finally:
        gpu.close()


@pytest.mark.parametrize("W,chunk,n_units,tail", [(5, 4096, 301, 1852), (16, 8192, 160, 704), (4, 16384, 150, 9000), (2, 2048, 600, 2048 + 33),
                                                  (7, 1024, 650, 1500), (3, 512, 620, 0), (64, 256, 610, 3), (33, 4096, 20, 0),
                                                  (1, 1024, 600, 1024), (16, 128, 300, 0)])
def test_server_prefetch_kernel_equals_plain_kernel(W, chunk, n_units, tail):
    """zoa_allreduce_average through the kernel that prefetches a chunk's inputs into shared memory
    against the same call through the plain one-block-per-chunk kernel: same bits in everything it
    writes, over rounds with non-zero errors, with and without a result buffer.  A ragged last chunk
    goes to the plain kernel in both; chunk 128 has no prefetching variant.  A smaller case of the
    same shape is also compared with the oracle."""
    rng = np.random.default_rng(W * chunk + 1)
    n = n_units * max(chunk, 4096) + tail
    a, b = Zoa(n, W, chunk=chunk, allreduce_only=True), Zoa(n, W, chunk=chunk, allreduce_only=True)
    try:
        a.set_pipeline("force")
        b.set_pipeline(False)
        za, zb = torch.empty(n, device="cuda"), torch.empty(n, device="cuda")
        for r in range(3):
            z = [torch.randn(n, device="cuda", generator=torch.Generator("cuda").manual_seed(100 * r + i)) * 10.0 ** (r - 1) for i in range(W)]
            for h, out in ((a, za), (b, zb)):
                h.allreduce_compress(z)
                h.allreduce_average(out if r != 1 else None)
            torch.cuda.synchronize()
            a.check_device()
            if r != 1:
                assert torch.equal(za, zb), f"z_bar, round {r}"
            for name in ("delta_s", "words_s", "scales_s"):
                assert np.array_equal(a.read(name), b.read(name)), (name, r)
        if chunk % 256 == 0 and n % chunk != 0:
            assert a.stats()["n_launches"] > b.stats()["n_launches"]      # prefetching kernel + the ragged chunk's
    finally:
        a.close(), b.close()
    # the same shape, small, against the oracle
    n = 3 * max(chunk, 4096) + (tail % (2 * chunk))
    cpu = zo.Oracle(n, W, chunk, dtype=np.float32)
    gpu = Zoa(n, W, chunk=chunk, allreduce_only=True)
    try:
        gpu.set_pipeline("force")
        for r in range(2):
            z = (rng.standard_normal((W, n)) * 10.0 ** rng.integers(-2, 2, size=(W, 1))).astype(np.float32)
            z_bar = torch.empty(n, device="cuda")
            gpu.onebit_allreduce([torch.from_numpy(z[i]).cuda() for i in range(W)], z_bar)
            torch.cuda.synchronize()
            want = cpu.onebit_allreduce(z)
            assert np.array_equal(gpu.read("words_s"), cpu.words_server), f"words_s, round {r}"
            assert_close(z_bar.cpu().numpy(), want, f"z_bar, round {r}")
            assert_close(gpu.read("scales_s"), cpu.scales_server, f"scales_s, round {r}")
            assert_close(gpu.read("delta_s"), cpu.delta_bar, f"delta_s, round {r}")
        gpu.check_device()
    finally:
        gpu.close()


@pytest.mark.parametrize("prefetch", [False, True])
@pytest.mark.parametrize("W,chunk", [(6, 1024), (16, 4096), (64, 256), (3, 1024)])
def test_onebit_allreduce_worker_magnitudes_far_apart(W, chunk, prefetch):
    """The server kernels add table entries for groups of four workers, which gives the bits of the
    worker-by-worker binary64 sum only while every partial sum is exact; a chunk whose workers'
    magnitudes are too far apart for that must take the worker-by-worker loop.  Here the chunks
    alternate between magnitudes of one size, magnitudes spread over 2^100 (partial sums round), a
    spread just inside and just outside the limit, and workers whose buffers are all zero; through the
    plain one-block-per-chunk kernel and through the prefetching kernel."""
    rng = np.random.default_rng(W * chunk)
    n = 9 * chunk + 77
    cpu = zo.Oracle(n, W, chunk, dtype=np.float32)
    gpu = Zoa(n, W, chunk=chunk, allreduce_only=True)
    gpu.set_pipeline("force" if prefetch else False)
    limit = 29 - int(np.ceil(np.log2(W)))                  # largest exponent gap with exact partial sums
    try:
        for r in range(3):
            z = rng.standard_normal((W, n)).astype(np.float32)
            for c in range((n + chunk - 1) // chunk):
                sl = slice(c * chunk, min((c + 1) * chunk, n))
                for i in range(W):
                    if c % 5 == 1:
                        z[i, sl] *= np.float32(2.0 ** (-50 + (100 * i) // max(W - 1, 1)))
                    elif c % 5 == 2:
                        z[i, sl] *= np.float32(2.0 ** ((limit - 2) * (i % 2)))
                    elif c % 5 == 3:
                        z[i, sl] *= np.float32(2.0 ** ((limit + 3) * (i % 2)))
                    elif c % 5 == 4 and i % 3 == 0:
                        z[i, sl] = 0.0
            z_dev = [torch.from_numpy(z[i]).cuda() for i in range(W)]
            z_bar = torch.empty(n, device="cuda")
            gpu.onebit_allreduce(z_dev, z_bar)
            torch.cuda.synchronize()
            want = cpu.onebit_allreduce(z)
            assert np.array_equal(gpu.read("words_s"), cpu.words_server), f"words_s, round {r}"
            assert_close(z_bar.cpu().numpy(), want, f"z_bar, round {r}")
            assert_close(gpu.read("scales_s"), cpu.scales_server, f"scales_s, round {r}")
            assert_close(gpu.read("delta_s"), cpu.delta_bar, f"delta_s, round {r}")
        gpu.check_device()
    finally:
        gpu.close()


@pytest.mark.parametrize("where", ["pending_variance", "after_sync", "mid_interval"])
def test_checkpoint_round_trip(where):
    """zoa_export_state / zoa_import_state through the C ABI: run, export, import into a fresh handle,
    continue on both; the two handles stay bit-identical and both match the oracle.  In the
    "pending_variance" case the export falls between zoa_step on a step in T_u and T_v and
    zoa_onebit_reduce, when the handle holds v_t (which the model sync still needs) and v_{t+1}."""
    rng = np.random.default_rng(6)
    n, W, chunk = 5000, 3, 512
    var_steps, sync = (0, 1, 5), ((0, 2), (1, 3))        # T_u = {0, 1, 2, 5, 8, ...}
    cut = {"pending_variance": 5, "after_sync": 3, "mid_interval": 4}[where]
    gs = [_grads(rng, W, n) for _ in range(10)]
    x0 = rng.standard_normal(n) * 0.02
    p = Pair(n, W, chunk, var_steps=var_steps, sync=sync, x0=x0)
    b = Zoa(n, W, chunk=chunk, beta1=0.5, beta2=0.5, eps=1e-3)      # everything, hyper-parameters included, comes from the blob
    try:
        a = p.gpu
        for t in range(cut):
            p.step(gs[t], 1e-3, t, "two_call")
        if where == "pending_variance":
            # first half of step `cut`: zoa_step on a T_u and T_v step, export before the reduce
            a.step(list(torch.from_numpy(gs[cut]).cuda()), 1e-3, cut)
        size = B.zoa_state_size(a.h)
        blob = a.export_state()
        assert blob.size == size
        with pytest.raises(ZoaError):                    # a truncated blob changes nothing
            B.zoa_import_state(b.h, blob.ctypes.data, size - 4)
        other = Zoa(n + 1, W, chunk=chunk)
        try:
            with pytest.raises(ZoaError):                # another shape
                other.import_state(blob)
        finally:
            other.close()
        b.import_state(blob)
        assert b.stats() == {**a.stats(), "n_launches": b.stats()["n_launches"]}
        assert b.sync_due(4) == a.sync_due(4) and b.var_due(5) and not b.var_due(4)
        if where == "pending_variance":
            a.onebit_reduce(), b.onebit_reduce()
            torch.cuda.synchronize()
            assert p.cpu.step(gs[cut], np.float32(1e-3), cut, True, True) == 0
            p.compare(f"{where} t={cut}")
            cut += 1
        for t in range(cut, 10):
            g = list(torch.from_numpy(gs[t]).cuda())
            b.step_auto(g, 1e-3, t)
            p.step(gs[t], 1e-3, t, "fused")
            p.compare(f"{where} t={t}", wire=a.sync_due(t))
            for name in ("x", "m", "u", "delta_w"):
                for i in range(W):
                    assert np.array_equal(a.read(name, i), b.read(name, i)), (name, i, t)
            for name in ("v", "delta_s", "x_sync"):
                assert np.array_equal(a.read(name), b.read(name)), (name, t)
        assert a.stats()["gamma_sum"] == b.stats()["gamma_sum"] and a.stats()["t_sync"] == b.stats()["t_sync"]
        b.check_device()
    finally:
        p.close(), b.close()


def test_host_gradient_entry_point():
    rng = np.random.default_rng(8)
    n, W, chunk = 4096 + 100, 2, 1024
    a, b = Zoa(n, W, chunk=chunk), Zoa(n, W, chunk=chunk)
    try:
        for t in range(3):
            g = torch.from_numpy(_grads(rng, W, n)).pin_memory()
            out = torch.empty(n).pin_memory()
            a.step_host(list(g), 1e-3, t, out)
            b.step_auto(list(g.cuda()), 1e-3, t)
            torch.cuda.synchronize()
            assert np.array_equal(out.numpy(), b.read("x", 0))
            assert np.array_equal(a.read("m", 1), b.read("m", 1))
    finally:
        a.close(), b.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_host_entry_point_in_overlapped_segments(dtype):
    """Large enough to be cut into eight chunk ranges with the copies overlapping the kernels:
    every state must equal the plain device path, over sync, local and variance steps."""
    rng = np.random.default_rng(21)
    n, W, chunk = 700 * 1024 + 100, 3, 1024
    a, b = Zoa(n, W, chunk=chunk), Zoa(n, W, chunk=chunk)
    try:
        for z in (a, b):
            z.set_pipeline("force")
            z.set_policies((0, 1, 4), (0, 2), (1, 3))
            z.set_grad_dtype(dtype)
        out = torch.empty(n).pin_memory()
        for t in range(7):
            g = torch.from_numpy(_grads(rng, W, n)).to(dtype).pin_memory()
            a.step_host(list(g), 1e-3, t, out)
            b.step_auto(list(g.cuda()), 1e-3, t)
            torch.cuda.synchronize()
            assert np.array_equal(out.numpy(), b.read("x", 0)), t
            for name in ("x", "m", "u", "delta_w"):
                for i in range(W):
                    assert np.array_equal(a.read(name, i), b.read(name, i)), (name, i, t)
            for name in ("v", "delta_s", "x_sync", "words_s", "scales_s"):
                assert np.array_equal(a.read(name), b.read(name)), (name, t)
        assert a.stats()["n_syncs"] == b.stats()["n_syncs"] and a.stats()["t_sync"] == b.stats()["t_sync"]
        a.check_device()
    finally:
        a.close(), b.close()


def test_argument_and_state_errors():
    with pytest.raises(ZoaError) as e:
        Zoa(100, 0)
    assert e.value.status == B.ERR_ARG
    for kw in (dict(chunk=48), dict(chunk=16), dict(chunk=(1 << 30) + 32), dict(beta1=1.0), dict(eps=0.0)):
        with pytest.raises(ZoaError):
            Zoa(100, 2, **kw)
    z = Zoa(100, 2, chunk=32)
    try:
        with pytest.raises(ZoaError) as e:
            z.onebit_reduce()                       # nothing accumulated: the momentum approximation would divide by zero
        assert e.value.status == B.ERR_STATE
        g = list(torch.zeros(2, 100, device="cuda"))
        z.step(g, 1e-3, 5)
        with pytest.raises(ZoaError) as e:
            z.step(g, 1e-3, 5)                      # t must increase
        assert e.value.status == B.ERR_STATE
        with pytest.raises(ZoaError):
            z.step(g, float("nan"), 6)
        with pytest.raises(ZoaError) as e:
            z.step_sync(g, -1.0, 7)                 # the sum of learning rates would not be positive
        assert e.value.status == B.ERR_STATE
        z.onebit_reduce()
        with pytest.raises(ZoaError):
            z.onebit_reduce()
        with pytest.raises(ZoaError):
            z.read("x", worker=2)
        z.check_device()
        assert B.zoa_check_finite(z.h) == 0
        s = z.stats()
        assert s["n_steps"] == 1 and s["n_syncs"] == 1 and s["n_launches"] == 3
        assert s["bits_per_worker"] == 100 + 32 * 4
    finally:
        z.close()


def test_policies_match_the_workload_tables():
    for make in synth.WORKLOADS.values():
        wl = synth.scaled(make(), 1 << 14)
        z = Zoa(wl.n, wl.W, chunk=wl.chunk)
        try:
            z.set_policies(wl.var_steps, wl.sync_boundaries, wl.sync_intervals)
            for t in range(wl.steps):
                assert z.sync_due(t) == wl.in_T_u(t) and z.var_due(t) == wl.in_T_v(t)
        finally:
            z.close()
    z = Zoa(64, 1, chunk=32)
    try:
        B.zoa_set_var_policy_doubling(z.h, 2, 40)   # gaps 1,1,2,2,4,4,8,8,...
        got = [t for t in range(60) if z.var_due(t)]
        assert got == [0, 1, 2, 4, 6, 10, 14, 22, 30]
    finally:
        z.close()


@pytest.mark.parametrize("algorithm", ["alg1", "alg2", "two_call", "allreduce", "alg1_chunk_1024", "alg1_chunk_8192"])
def test_device_wait_runs_out_and_is_reported(algorithm):
    """Error path of the ring kernels without any fault: the copy-issuing lane of every block
    stops after three tiles (test hook), the other threads' bounded waits run out after
    100 ms, the kernel ends by itself, zoa_check_device reports ZOA_ERR_DEVICE, and the
    context and the handle stay usable.  Covers the fused kernel (one, two and four tiles per
    unit), Algorithm 2's, the server kernel of the two-call path with its store-issuing warp, and the
    prefetching server kernel of Algorithm 3 alone (whose copies are then never started)."""
    import time
    chunk = 1024 if algorithm.endswith("1024") else 8192 if algorithm.endswith("8192") else 4096
    n, W = 300 * max(chunk, 2048), 4
    z = Zoa(n, W, chunk=chunk)
    try:
        g = list(torch.randn(W, n, device="cuda"))
        z.set_pipeline("force")

        def two_call(g, lr, t):
            z.step(g, lr, t)
            z.onebit_reduce()
        z_bar = torch.empty(n, device="cuda")

        def allreduce(g, lr, t):
            z.onebit_allreduce(g, z_bar)
        step = {"alg2": z.alg2_step, "two_call": two_call, "allreduce": allreduce}.get(algorithm, z.step_sync)
        step(g, 1e-3, 0)
        z.check_device()                                  # the normal path works
        B.zoa_set_option(z.h, B.OPT_WAIT_LIMIT_MS, 100)
        B.zoa_set_option(z.h, B.OPT_TEST_STOP_AFTER_TILES, 3)
        t0 = time.perf_counter()
        step(g, 1e-3, 1)
        torch.cuda.synchronize()                          # the kernel has ended by itself
        assert time.perf_counter() - t0 < 5.0             # bounded: a few wait limits, not a hang
        with pytest.raises(ZoaError) as e:                # the next step call itself refuses, without any check call
            step(g, 1e-3, 2)
        assert e.value.status == B.ERR_DEVICE
        with pytest.raises(ZoaError) as e:
            z.onebit_reduce()
        assert e.value.status == B.ERR_DEVICE
        with pytest.raises(ZoaError) as e:
            z.check_device()
        assert e.value.status == B.ERR_DEVICE
        B.zoa_set_option(z.h, B.OPT_TEST_STOP_AFTER_TILES, 0)
        B.zoa_set_option(z.h, B.OPT_WAIT_LIMIT_MS, 2000)
        step(g, 1e-3, 2)
        z.check_device()                                  # flag cleared, chunk counter rearmed
    finally:
        z.close()


# --------------------------------------------------------------------------
# Algorithm 2 (gradients through the 1-bit AllReduce; 1-bit Adam special case)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("W,chunk,n", [(3, 2048, 1), (3, 2048, 33), (3, 2048, 2049), (2, 64, 4096 + 5), (5, 96, 96 * 7 + 3),
                                       (8, 4096, 3 * 4096 + 1852), (4, 8192, 8192 * 2 + 704), (2, 16384, 16384 * 2 + 100),
                                       (64, 256, 1500), (16, 4096, 40 * 4096 + 77)])
def test_alg2_parity(W, chunk, n):
    """Ten steps of Algorithm 2: a full-precision stage (T_v = {0,1,2}) then compressed steps,
    i.e. the 1-bit Adam special case; every state after every step."""
    rng = np.random.default_rng(W + chunk + n)
    p = Pair(n, W, chunk, var_steps=(0, 1, 2), x0=rng.standard_normal(n) * 0.02)
    try:
        for t in range(10):
            g = _grads(rng, W, n)
            p.gpu.alg2_step(list(torch.from_numpy(g).cuda()), 1e-3 * (1 + t % 3), t)
            torch.cuda.synchronize()
            p.cpu.alg2_step(g, np.float32(1e-3 * (1 + t % 3)), t in (0, 1, 2))
            p.compare(f"t={t}", wire=t > 2)
        p.padding_is_zero()
        s = p.gpu.stats()
        assert s["n_var_updates"] == 3 and s["n_syncs"] == 7 and s["n_steps"] == 10
    finally:
        p.close()


def test_alg2_unaligned_and_interleaved_variance_steps():
    rng = np.random.default_rng(55)
    n, W, chunk = 5000, 3, 1024
    p = Pair(n, W, chunk, var_steps=(0, 3, 4), x0=rng.standard_normal(n) * 0.02)
    try:
        for t in range(7):
            g = _grads(rng, W, n)
            backing = torch.zeros(W, n + 8, device="cuda")
            views = [backing[i, 1:1 + n] for i in range(W)]
            for i in range(W):
                views[i].copy_(torch.from_numpy(g[i]))
            p.gpu.alg2_step(views, 2e-3, t)
            torch.cuda.synchronize()
            p.cpu.alg2_step(g, np.float32(2e-3), t in (0, 3, 4))
            p.compare(f"t={t}", wire=False)
    finally:
        p.close()


# --------------------------------------------------------------------------
# Chunks larger than one block can hold, up to the whole vector (Eq. 3 as printed)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("mode", ["fused", "two_call", "alg2"])
@pytest.mark.parametrize("W,chunk,n", [(3, 32768, 2 * 32768 + 5000), (4, 1 << 20, 300001), (2, 20000 * 32, 20000 * 32),
                                       (5, 16384 + 32, 3 * (16384 + 32) + 17), (16, 1 << 22, 70000)])
def test_large_chunks_and_whole_vector_scale(W, chunk, n, mode):
    """chunk > 16384 goes through the multi-pass kernels; chunk >= n is the paper's compressor
    with one magnitude for the whole vector."""
    rng = np.random.default_rng(W + n)
    p = Pair(n, W, chunk, var_steps=(0, 2), sync=((0, 3), (1, 2)), x0=rng.standard_normal(n) * 0.02)
    try:
        for t in range(6):
            g = _grads(rng, W, n)
            if mode == "alg2":
                p.gpu.alg2_step(list(torch.from_numpy(g).cuda()), 1e-3, t)
                torch.cuda.synchronize()
                p.cpu.alg2_step(g, np.float32(1e-3), t in (0, 2))
                p.compare(f"t={t}", wire=t not in (0, 2))
            else:
                p.step(g, 1e-3, t, mode)
                p.compare(f"t={t}", wire=p.gpu.sync_due(t))
        p.padding_is_zero()
        if chunk >= n:
            assert p.gpu.read("scales_s").size == 1
    finally:
        p.close()


@pytest.mark.parametrize("mode", ["fused", "two_call", "alg2"])
@pytest.mark.parametrize("W,chunk,n", [(3, 32768, 2 * 32768 + 5000), (5, 1 << 22, 70000)])
def test_large_chunks_worker_magnitudes_far_apart(W, chunk, n, mode):
    """The large-chunk server pass also looks the sum over the workers up in tables; with the workers'
    gradients 2^25 apart from one another the partial sums round and it must add worker by worker."""
    rng = np.random.default_rng(W * n)
    p = Pair(n, W, chunk, var_steps=(0,), sync=((0,), (1,)), x0=rng.standard_normal(n) * 0.02)
    factor = (2.0 ** (25.0 * np.arange(W) - 40.0)).astype(np.float32)[:, None]
    try:
        for t in range(4):
            g = _grads(rng, W, n) * factor
            if mode == "alg2":
                p.gpu.alg2_step(list(torch.from_numpy(g).cuda()), 1e-3, t)
                torch.cuda.synchronize()
                p.cpu.alg2_step(g, np.float32(1e-3), t == 0)
                p.compare(f"t={t}", wire=t != 0)
            else:
                p.step(g, 1e-3, t, mode)
                p.compare(f"t={t}", wire=True)
    finally:
        p.close()


def test_paper_schedules_on_a_handle():
    z = Zoa(64, 1, chunk=32)
    try:
        B.zoa_set_var_policy_doubling(z.h, 2, 1000)
        B.zoa_set_sync_policy_doubling(z.h, 10, 5, 4, True)      # interval 1 until step 15, 2 until 20, then 4
        assert [t for t in range(30) if z.sync_due(t)] == list(range(15)) + [15, 17, 19] + [20, 24, 28]
        assert [t for t in range(40) if z.var_due(t)] == [0, 1, 2, 4, 6, 10, 14]     # nothing from step 15 on
    finally:
        z.close()


# --------------------------------------------------------------------------
# 16-bit gradients (the paper trains in FP16): converted exactly on load
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("mode", ["fused", "two_call", "alg2"])
@pytest.mark.parametrize("W,chunk,n,offset", [(4, 2048, 9 * 2048 + 77, 0), (3, 4096, 5 * 4096 + 1852, 0), (2, 8192, 3 * 8192, 0),
                                              (3, 1024, 5000, 0), (2, 4096, 3 * 4096 + 5, 1), (2, 32768, 70000, 0)])
def test_sixteen_bit_gradients(dtype, mode, W, chunk, n, offset):
    """The oracle is given the binary32 values of the very same 16-bit numbers; the GPU reads
    the 16-bit buffers.  `offset` shifts the buffers by one element (unaligned path)."""
    rng = np.random.default_rng(W * chunk + n)
    p = Pair(n, W, chunk, var_steps=(0, 2), sync=((0, 3), (1, 2)), x0=rng.standard_normal(n) * 0.02)
    try:
        p.gpu.set_grad_dtype(dtype)
        for t in range(5):
            backing = torch.from_numpy(_grads(rng, W, n + offset)).cuda().to(dtype)
            g16 = [backing[i, offset:offset + n] for i in range(W)]
            if offset == 0:
                g16 = [g.clone() for g in g16]
            g32 = torch.stack([g.float() for g in g16]).cpu().numpy()
            sync, var = p.gpu.sync_due(t), p.gpu.var_due(t)
            if mode == "alg2":
                p.gpu.alg2_step(g16, 1e-3, t)
                p.cpu.alg2_step(g32, np.float32(1e-3), var)
            else:
                if mode == "fused":
                    p.gpu.step_auto(g16, 1e-3, t)
                else:
                    p.gpu.step(g16, 1e-3, t)
                    if sync:
                        p.gpu.onebit_reduce()
                p.cpu.step(g32, np.float32(1e-3), t, sync, var)
            torch.cuda.synchronize()
            p.compare(f"t={t}", wire=False)
        p.gpu.check_device()
    finally:
        p.close()


def test_sixteen_bit_host_gradients():
    rng = np.random.default_rng(9)
    n, W, chunk = 3 * 2048 + 100, 2, 2048
    a, b = Zoa(n, W, chunk=chunk), Zoa(n, W, chunk=chunk)
    try:
        a.set_grad_dtype(torch.bfloat16), b.set_grad_dtype(torch.bfloat16)
        for t in range(3):
            g = torch.from_numpy(_grads(rng, W, n)).to(torch.bfloat16).pin_memory()
            out = torch.empty(n).pin_memory()
            a.step_host(list(g), 1e-3, t, out)
            b.step_auto(list(g.cuda()), 1e-3, t)
            torch.cuda.synchronize()
            assert np.array_equal(out.numpy(), b.read("x", 0))
    finally:
        a.close(), b.close()


def test_create_destroy_returns_device_memory():
    torch.cuda.empty_cache()
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(20):
        z = Zoa(1 << 22, 4, chunk=4096)            # ~340 MB of state each
        z.step_sync(list(torch.zeros(4, 1 << 22, device="cuda")), 1e-3, 0)
        z.close()
    torch.cuda.empty_cache()
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free0 - free1 < 64 << 20, f"{(free0 - free1) >> 20} MiB did not come back"


@pytest.mark.parametrize("W,chunk,n_chunks,tail,dtype", [(5, 4096, 301, 1852, torch.float32), (3, 2048, 700, 0, torch.float32),
                                                         (4, 8192, 160, 704, torch.bfloat16), (16, 4096, 40, 5, torch.float16),
                                                         (64, 2048, 20, 33, torch.float32)])
def test_alg2_ring_kernel_equals_block_kernel(W, chunk, n_chunks, tail, dtype):
    rng = np.random.default_rng(W + chunk)
    n = n_chunks * chunk + tail
    x0 = torch.from_numpy((rng.standard_normal(n) * 0.02).astype(np.float32))
    a, b = Zoa(n, W, chunk=chunk), Zoa(n, W, chunk=chunk)
    try:
        a.set_pipeline("force")
        b.set_pipeline(False)
        for z in (a, b):
            z.set_params(x0)
            z.set_policies((0,), (0,), (1,))
            z.set_grad_dtype(dtype)
        g = torch.empty(W, n, device="cuda")
        for t in range(4):
            g.normal_(generator=torch.Generator("cuda").manual_seed(t + 5))
            gg = list(g.to(dtype))
            a.alg2_step(gg, 1e-3, t)
            b.alg2_step(gg, 1e-3, t)
            torch.cuda.synchronize()
            a.check_device()
            for name in ("x", "m", "delta_w", "words_w", "scales_w"):
                for i in (0, W // 2, W - 1):
                    assert np.array_equal(a.read(name, i), b.read(name, i)), (name, i, t)
            for name in ("v", "delta_s", "words_s", "scales_s"):
                assert np.array_equal(a.read(name), b.read(name)), (name, t)
    finally:
        a.close(), b.close()


@pytest.mark.parametrize("mode", ["fused", "two_call"])
def test_nonfinite_gradients_propagate_like_the_oracle(mode):
    """NaN and infinities do not trap or hang: the affected chunks turn NaN on both sides in the
    same places, the others stay exact."""
    rng = np.random.default_rng(13)
    W, chunk, n = 3, 2048, 5 * 2048 + 9
    p = Pair(n, W, chunk, var_steps=(0,), x0=rng.standard_normal(n) * 0.02)
    try:
        for t in range(3):
            g = _grads(rng, W, n)
            if t == 1:
                g[0, 5] = np.nan                # chunk 0 of worker 0
                g[1, 2 * 2048 + 7] = np.inf     # chunk 2 of worker 1
                g[2, n - 1] = -np.inf           # the ragged last chunk
            with np.errstate(invalid="ignore", over="ignore"):
                p.step(g, 1e-3, t, mode)
            p.compare(f"t={t}", wire=False)
            for i in range(W):
                assert np.array_equal(p.gpu.read("words_w", i), p.cpu.words_worker[i]), (t, i)
        assert B.zoa_check_finite(p.gpu.h) > 0
        assert np.isnan(p.gpu.read("delta_w", 0)[:2048]).all()
        assert np.isfinite(p.gpu.read("x", 0)[2048:2 * 2048]).all()      # an untouched chunk
    finally:
        p.close()


def test_zero_learning_rate_steps():
    rng = np.random.default_rng(14)
    W, chunk, n = 2, 1024, 3000
    p = Pair(n, W, chunk, var_steps=(0,), sync=((0,), (3,)), x0=rng.standard_normal(n) * 0.02)
    try:
        for t, lr in enumerate([1e-3, 0.0, 0.0, 2e-3, 0.0, 1e-3, 1e-3]):
            p.step(_grads(rng, W, n), lr, t, "fused")
            p.compare(f"t={t}", wire=False)
    finally:
        p.close()


@pytest.mark.parametrize("W,chunk,n_chunks", [(64, 8192, 3), (64, 4096, 5), (48, 8192, 4)])
def test_many_workers_ring_or_fallback(W, chunk, n_chunks):
    """W = 64 with chunk 8192 does not leave room for the ring in shared memory and takes the
    block kernel; chunk 4096 does fit.  Either way the oracle decides."""
    rng = np.random.default_rng(W + chunk)
    n = n_chunks * chunk + 100
    p = Pair(n, W, chunk, var_steps=(0,), x0=rng.standard_normal(n) * 0.02)
    try:
        for t in range(2):
            p.step(_grads(rng, W, n), 1e-3, t, "fused")
            p.compare(f"t={t}")
    finally:
        p.close()


def test_allocation_failure_is_reported_and_leaves_the_context_usable():
    with pytest.raises(ZoaError) as e:
        Zoa(1 << 36, 64, chunk=4096)                  # 70 TB of state
    assert e.value.status == B.ERR_ALLOC
    z = Zoa(4096, 2, chunk=1024)                      # the device still works
    try:
        z.step_sync(list(torch.ones(2, 4096, device="cuda")), 1e-3, 0)
        z.check_device()
    finally:
        z.close()


def test_work_is_ordered_on_the_callers_stream():
    """Gradients are produced late on a non-blocking side stream and consumed by the steps
    enqueued behind them on the same stream; nothing synchronises in between, so a kernel
    launched on any other stream would read the stale buffers."""
    n, W, chunk = 6 * 4096 + 100, 3, 4096
    rng = np.random.default_rng(77)
    p = Pair(n, W, chunk, var_steps=(0, 2), sync=((0,), (2,)), x0=rng.standard_normal(n) * 0.02)
    side = torch.cuda.Stream()
    gdev = torch.zeros((W, n), device="cuda")
    staged = [torch.from_numpy(rng.standard_normal((W, n)).astype(np.float32)).cuda() for _ in range(4)]
    torch.cuda.synchronize()
    try:
        with torch.cuda.stream(side):
            for t in range(4):
                torch.cuda._sleep(20_000_000)            # ~10 ms: the copy below lands well after the host has moved on
                gdev.copy_(staged[t], non_blocking=True)
                if t >= 2:
                    p.gpu.step_auto(list(gdev), 1e-3, t)
                else:
                    p.gpu.step(list(gdev), 1e-3, t)
                    if p.gpu.sync_due(t):
                        p.gpu.onebit_reduce()
        side.synchronize()
        for t in range(4):
            assert p.cpu.step(staged[t].cpu().numpy(), np.float32(1e-3), t, p.gpu.sync_due(t), p.gpu.var_due(t)) == 0
        p.compare("side stream")
    finally:
        p.close()
