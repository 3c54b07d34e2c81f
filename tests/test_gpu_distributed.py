"""One worker per GPU, checked on one GPU: the ranks are emulated as separate handles in one
process (each with a single worker and its own server range), the collectives by plain copies
between their buffers; the result must equal the CPU oracle of Algorithm 1 / Algorithm 3 (worker
side on every rank, server side on the range each rank serves) within the parity tolerance with
bit-exact packed words, and the single handle that holds all W workers bit for bit.  A second
test runs the real driver, collectives included, as a one-rank NCCL job."""
import os

import numpy as np
import pytest
import torch

from helpers import assert_close
from oracle import zoa_oracle as zo
from paper_2202_06009_b200 import Zoa
from paper_2202_06009_b200.distributed import PeerTable, WorkerPerGpu

pytestmark = pytest.mark.gpu


def _one_rank_process_group():
    """A one-rank NCCL group on a port nobody holds (each test makes and destroys its own)."""
    import socket
    import torch.distributed as dist
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    return dist


def _compare_ranks_with_oracle(ranks, cpu, chunk, n, t, synced, worker_wire=True):
    """Every rank against the oracle that holds all the workers: rank r is worker r of Algorithm 1
    and the server of Algorithm 3 for its own chunk range."""
    for r, w in enumerate(ranks):
        what = f"rank {r} t={t}"
        assert_close(w.opt.read("x", 0), cpu.x[r], f"{what} x")
        assert_close(w.opt.read("m", 0), cpu.m[r], f"{what} m")
        assert_close(w.opt.read("u", 0), cpu.u[r], f"{what} u")
        assert_close(w.opt.read("delta_w", 0), cpu.delta[r], f"{what} delta_w")
        assert_close(w.opt.read("v"), cpu.v, f"{what} v")
        assert_close(w.opt.read("x_sync"), cpu.x_sync, f"{what} x_sync")
        cr = w.plan.chunks[r]
        lo, hi = cr.start * chunk, min(cr.stop * chunk, n)
        if hi > lo:
            assert_close(w.opt.read("delta_s", 0, lo, hi - lo), cpu.delta_bar[lo:hi], f"{what} delta_s of the served range")
        if synced:
            if worker_wire:
                assert np.array_equal(w.opt.read("words_w", 0), cpu.words_worker[r]), f"{what} words_w"
                assert_close(w.opt.read("scales_w", 0), cpu.scales_worker[r], f"{what} scales_w")
            assert np.array_equal(w.opt.read("words_s"), cpu.words_server), f"{what} words_s"
            assert_close(w.opt.read("scales_s"), cpu.scales_server, f"{what} scales_s")


@pytest.mark.parametrize("W,chunk,n", [(3, 1024, 7 * 1024 + 100), (4, 4096, 9 * 4096), (5, 256, 3 * 256 + 7), (2, 2048, 2048 * 5 + 33)])
def test_emulated_ranks_equal_the_single_handle(W, chunk, n):
    rng = np.random.default_rng(W * n)
    var_steps, sync = (0, 1, 3), ((0, 3), (1, 2))
    x0 = torch.from_numpy((rng.standard_normal(n) * 0.02).astype(np.float32))
    ref = Zoa(n, W, chunk=chunk)
    cpu = zo.Oracle(n, W, chunk, dtype=np.float32)
    ranks = [WorkerPerGpu(n, chunk, r, W, var_steps, *sync) for r in range(W)]
    try:
        ref.set_params(x0)
        ref.set_policies(var_steps, *sync)
        cpu.set_params(x0.numpy())
        for w in ranks:
            w.opt.set_params(x0)
        for t in range(7):
            g = torch.from_numpy(rng.standard_normal((W, n)).astype(np.float32)).cuda()
            ref.step_auto(list(g), 1e-3, t)
            assert cpu.step(g.cpu().numpy(), np.float32(1e-3), t, ref.sync_due(t), t in var_steps) == 0
            for r, w in enumerate(ranks):
                w.opt.step([g[r]], 1e-3, t)
            if t in var_steps:                       # stands in for the all-reduce: the same worker-order binary64 mean
                acc = g[0].double()
                for i in range(1, W):
                    acc = acc + g[i].double()
                g_bar = (acc / W).float()
                for w in ranks:
                    w.variance(g_bar)
            if ref.sync_due(t):
                packs = [w.pack() for w in ranks]
                torch.cuda.synchronize()
                served = []
                for r, w in enumerate(ranks):        # stands in for the all-to-all
                    wr, cr = w.plan.words[r], w.plan.chunks[r]
                    recv_words = torch.stack([p[0][wr.start:wr.stop] for p in packs]).contiguous()
                    recv_scales = torch.stack([p[1][cr.start:cr.stop] for p in packs]).contiguous()
                    served.append(w.serve(recv_words, recv_scales))
                torch.cuda.synchronize()
                for r, w in enumerate(ranks):        # stands in for the all-gather
                    wr, cr = w.plan.words[r], w.plan.chunks[r]
                    for q, other in enumerate(ranks):
                        if q != r:
                            served[q][0][wr.start:wr.stop] = served[r][0][wr.start:wr.stop]
                            served[q][1][cr.start:cr.stop] = served[r][1][cr.start:cr.stop]
                for w in ranks:
                    w.apply()
            torch.cuda.synchronize()
            _compare_ranks_with_oracle(ranks, cpu, chunk, n, t, ref.sync_due(t))
            for r, w in enumerate(ranks):
                for name in ("x", "m", "u", "delta_w"):
                    assert np.array_equal(w.opt.read(name, 0), ref.read(name, r)), (name, r, t)
                assert np.array_equal(w.opt.read("v"), ref.read("v")), ("v", r, t)
                assert np.array_equal(w.opt.read("x_sync"), ref.read("x_sync")), ("x_sync", r, t)
                cr = w.plan.chunks[r]
                lo, hi = cr.start * chunk, min(cr.stop * chunk, n)
                if hi > lo:
                    assert np.array_equal(w.opt.read("delta_s", 0, lo, hi - lo), ref.read("delta_s", 0, lo, hi - lo)), ("delta_s", r, t)
                if ref.sync_due(t):
                    assert np.array_equal(w.opt.read("words_s"), ref.read("words_s")), ("words_s", r, t)
                    assert np.array_equal(w.opt.read("scales_s"), ref.read("scales_s")), ("scales_s", r, t)
    finally:
        ref.close()
        for w in ranks:
            w.close()


def _compare_ranks_with_single_handle(ranks, ref, chunk, n, t, synced):
    for r, w in enumerate(ranks):
        for name in ("x", "m", "u", "delta_w"):
            assert np.array_equal(w.opt.read(name, 0), ref.read(name, r)), (name, r, t)
        assert np.array_equal(w.opt.read("v"), ref.read("v")), ("v", r, t)
        assert np.array_equal(w.opt.read("x_sync"), ref.read("x_sync")), ("x_sync", r, t)
        cr = w.plan.chunks[r]
        lo, hi = cr.start * chunk, min(cr.stop * chunk, n)
        if hi > lo:
            assert np.array_equal(w.opt.read("delta_s", 0, lo, hi - lo), ref.read("delta_s", 0, lo, hi - lo)), ("delta_s", r, t)
        if synced:
            assert np.array_equal(w.opt.read("words_w", 0), ref.read("words_w", r)), ("words_w", r, t)
            assert np.array_equal(w.opt.read("scales_w", 0), ref.read("scales_w", r)), ("scales_w", r, t)
            assert np.array_equal(w.opt.read("words_s"), ref.read("words_s")), ("words_s", r, t)
            assert np.array_equal(w.opt.read("scales_s"), ref.read("scales_s")), ("scales_s", r, t)


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("W,chunk,n", [(3, 1024, 7 * 1024 + 100), (4, 4096, 9 * 4096), (5, 256, 3 * 256 + 7),
                                       (2, 2048, 2048 * 5 + 33), (8, 16384, 3 * 16384 + 5000), (1, 512, 2000)])
def test_exchange_by_peer_stores_equals_the_single_handle(W, chunk, n, fused):
    """The ranks (one handle each, all on this GPU) store their packed buffers straight into one
    another's memory; stream order stands in for the two barriers.  fused: sync steps go through
    zoa_dist_step_pack_push, which never writes the half-step m, x, u."""
    rng = np.random.default_rng(W * n + fused)
    var_steps, sync = (0, 1, 3), ((0, 3), (1, 2))
    x0 = torch.from_numpy((rng.standard_normal(n) * 0.02).astype(np.float32))
    ref = Zoa(n, W, chunk=chunk)
    cpu = zo.Oracle(n, W, chunk, dtype=np.float32)
    ranks = [WorkerPerGpu(n, chunk, r, W, var_steps, *sync) for r in range(W)]
    try:
        ref.set_params(x0)
        ref.set_policies(var_steps, *sync)
        cpu.set_params(x0.numpy())
        for w in ranks:
            w.opt.set_params(x0)
        peers = PeerTable.local(ranks)
        for t in range(7):
            g = torch.from_numpy(rng.standard_normal((W, n)).astype(np.float32)).cuda()
            ref.step_auto(list(g), 1e-3, t)
            synced = ref.sync_due(t)
            assert cpu.step(g.cpu().numpy(), np.float32(1e-3), t, synced, t in var_steps) == 0
            for r, w in enumerate(ranks):
                if synced and fused:
                    w.push_pack(peers, g[r], 1e-3, t)
                else:
                    w.opt.step([g[r]], 1e-3, t)
            if t in var_steps:
                acc = g[0].double()
                for i in range(1, W):
                    acc = acc + g[i].double()
                g_bar = (acc / W).float()
                for w in ranks:
                    w.variance(g_bar)
            if synced:
                if not fused:
                    for w in ranks:
                        w.push_pack(peers)
                for w in ranks:
                    w.push_serve(peers)
                for w in ranks:
                    w.apply()
            torch.cuda.synchronize()
            _compare_ranks_with_oracle(ranks, cpu, chunk, n, t, synced)
            _compare_ranks_with_single_handle(ranks, ref, chunk, n, t, synced)
        for w in ranks:
            w.opt.check_device()
    finally:
        ref.close()
        for w in ranks:
            w.close()


def test_peer_store_entry_points_reject_bad_tables():
    from paper_2202_06009_b200 import ZoaError, binding as B
    n, chunk = 5 * 1024, 1024
    one, two = Zoa(n, 1, chunk=chunk), Zoa(n, 2, chunk=chunk)
    buf = torch.zeros(n, dtype=torch.int32, device="cuda")
    ptr = buf.data_ptr()
    try:
        with pytest.raises(ZoaError):      # more than one worker in the handle
            B.zoa_dist_pack_push(two.h, [0, 5], [ptr], [ptr])
        with pytest.raises(ZoaError):      # ranges do not end at the number of chunks
            B.zoa_dist_pack_push(one.h, [0, 4], [ptr], [ptr])
        with pytest.raises(ZoaError):      # decreasing
            B.zoa_dist_pack_push(one.h, [0, 3, 2, 5], [ptr, ptr, ptr], [ptr, ptr, ptr])
        with pytest.raises(ZoaError):      # a serving rank without a buffer
            B.zoa_dist_pack_push(one.h, [0, 2, 5], [ptr, None], [ptr, ptr])
        with pytest.raises(ZoaError):      # step index must increase
            B.zoa_dist_step_pack_push(one.h, buf.view(torch.float32).data_ptr(), 1e-3, -1, [0, 5], [ptr], [ptr])
        with pytest.raises(ZoaError):
            B.zoa_dist_server_push(one.h, ptr, 64, ptr, 8, 1, 0, 5, [None], [ptr])
        B.zoa_dist_pack_push(one.h, [0, 5, 5], [ptr, None], [ptr, None])      # a rank that serves nothing needs none
        one.check_device()
    finally:
        one.close()
        two.close()


def test_pushed_driver_over_symmetric_memory_one_rank():
    """world_size 1 over NCCL with the buffers in torch's symmetric memory: the rendezvous, the
    address arithmetic of PeerTable.symmetric and the copy back into the handle run for real."""
    dist = _one_rank_process_group()
    rng = np.random.default_rng(5)
    n, chunk = 6 * 1024 + 50, 1024
    ref = Zoa(n, 1, chunk=chunk)
    cpu = zo.Oracle(n, 1, chunk, dtype=np.float32)
    w = WorkerPerGpu(n, chunk, 0, 1, var_steps=(0, 2), sync_boundaries=(0, 2), sync_intervals=(1, 2))
    try:
        try:
            peers = PeerTable.symmetric(w)
        except Exception as err:                      # symmetric memory is an optional torch feature
            pytest.skip(f"torch symmetric memory is not usable here: {err}")
        ref.set_policies((0, 2), (0, 2), (1, 2))
        for t in range(5):
            g = torch.from_numpy(rng.standard_normal((1, n)).astype(np.float32)).cuda()
            ref.step_auto(list(g), 1e-3, t)
            w.step_pushed(g[0], 1e-3, t, peers)      # default: the one-element all-reduce
            torch.cuda.synchronize()
            assert cpu.step(g.cpu().numpy(), np.float32(1e-3), t, ref.sync_due(t), t in (0, 2)) == 0
            _compare_ranks_with_oracle([w], cpu, chunk, n, t, ref.sync_due(t))
            for name in ("x", "m", "u", "delta_w"):
                assert np.array_equal(w.opt.read(name, 0), ref.read(name, 0)), (name, t)
            assert np.array_equal(w.opt.read("v"), ref.read("v")) and np.array_equal(w.opt.read("delta_s"), ref.read("delta_s"))
    finally:
        ref.close()
        w.close()
        dist.destroy_process_group()


def test_driver_with_real_collectives_one_rank():
    """world_size 1 over NCCL: every collective of WorkerPerGpu.step runs for real; W = 1 must
    equal the plain single-worker handle."""
    dist = _one_rank_process_group()
    rng = np.random.default_rng(3)
    n, chunk = 6 * 1024 + 50, 1024
    ref = Zoa(n, 1, chunk=chunk)
    cpu = zo.Oracle(n, 1, chunk, dtype=np.float32)
    w = WorkerPerGpu(n, chunk, 0, 1, var_steps=(0, 2), sync_boundaries=(0, 2), sync_intervals=(1, 2))
    try:
        ref.set_policies((0, 2), (0, 2), (1, 2))
        for t in range(5):
            g = torch.from_numpy(rng.standard_normal((1, n)).astype(np.float32)).cuda()
            ref.step_auto(list(g), 1e-3, t)
            w.step(g[0], 1e-3, t)
            torch.cuda.synchronize()
            assert cpu.step(g.cpu().numpy(), np.float32(1e-3), t, ref.sync_due(t), t in (0, 2)) == 0
            _compare_ranks_with_oracle([w], cpu, chunk, n, t, ref.sync_due(t))
            for name in ("x", "m", "u", "delta_w"):
                assert np.array_equal(w.opt.read(name, 0), ref.read(name, 0)), (name, t)
            assert np.array_equal(w.opt.read("v"), ref.read("v")) and np.array_equal(w.opt.read("delta_s"), ref.read("delta_s"))
    finally:
        ref.close()
        w.close()
        dist.destroy_process_group()
