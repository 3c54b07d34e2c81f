"""The exchange of the one-worker-per-GPU mapping on CPU: three gloo ranks send each chunk
range's packed words and magnitudes to the rank that serves it (all-to-all) and spread the
servers' results back (all-gather); every word must land where the plan says."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))



def _free_port():
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]

def _worker(rank, world, port, n, chunk, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2202_06009_b200.distributed import ExchangePlan, exchange_packed, gather_server
    plan = ExchangePlan.make(n, chunk, world)
    n_words, n_chunks = (n + 31) // 32, -(-n // chunk)
    # cover: ranges tile the vector, word ranges follow the chunk ranges
    assert plan.chunks[0].start == 0 and plan.chunks[-1].stop == n_chunks
    assert all(a.stop == b.start for a, b in zip(plan.chunks, plan.chunks[1:]))
    assert all(a.stop == b.start for a, b in zip(plan.words, plan.words[1:])) and plan.words[-1].stop == n_words
    assert all(w.start == c.start * chunk // 32 for w, c in zip(plan.words, plan.chunks))
    # worker -> server: word k of worker r carries (r, k)
    words = torch.arange(n_words, dtype=torch.int32) + rank * 1_000_000
    scales = torch.arange(n_chunks, dtype=torch.float32) + rank * 1000.0
    recv_words, recv_scales = exchange_packed(plan, rank, words, scales)
    mine_w, mine_c = plan.words[rank], plan.chunks[rank]
    for w in range(world):
        assert torch.equal(recv_words[w], torch.arange(mine_w.start, mine_w.stop, dtype=torch.int32) + w * 1_000_000)
        assert torch.equal(recv_scales[w], torch.arange(mine_c.start, mine_c.stop, dtype=torch.float32) + w * 1000.0)
    # server -> workers: each server's range carries its rank
    words_s = torch.full((n_words,), -1, dtype=torch.int32)
    scales_s = torch.full((n_chunks,), -1.0)
    words_s[mine_w.start:mine_w.stop] = rank
    scales_s[mine_c.start:mine_c.stop] = float(rank)
    gather_server(plan, rank, words_s, scales_s)
    for r in range(world):
        assert (words_s[plan.words[r].start:plan.words[r].stop] == r).all()
        assert (scales_s[plan.chunks[r].start:plan.chunks[r].stop] == float(r)).all()
    dist.barrier()
    if rank == 0:
        open(os.path.join(out_dir, "ok"), "w").write("ok")
    dist.destroy_process_group()


def _round_worker(rank, world, port, n, chunk, out_dir):
    """Two consecutive rounds of Algorithm 3 with one worker per rank: each rank compresses its own
    buffer (the oracle's compressor), the packed buffers travel through the exchange, the rank serves
    its chunk range, the packed results travel back.  After every round, every rank's output and
    errors must equal the single-process oracle that holds all the workers."""
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import numpy as np
    from oracle import zoa_oracle as zo
    from paper_2202_06009_b200.distributed import ExchangePlan, exchange_packed, gather_server
    plan = ExchangePlan.make(n, chunk, world)
    n_words, n_chunks = (n + 31) // 32, -(-n // chunk)
    rng = np.random.default_rng(77)                        # same seeded inputs on every rank
    z_rounds = rng.standard_normal((2, world, n)).astype(np.float32)
    whole = zo.Oracle(n, world, chunk, dtype=np.float32)   # the single-process run
    delta = np.zeros(n, np.float32)                        # this rank's worker error
    mine_c = plan.chunks[rank]
    lo, hi = mine_c.start * chunk, min(mine_c.stop * chunk, n)
    delta_bar = np.zeros(max(hi - lo, 0), np.float32)      # the server error of the range this rank serves

    def decode(words, scales, first, count):
        """+-scale of `count` coordinates from `first` (a chunk boundary), words starting at first / 32."""
        bits = np.unpackbits(np.ascontiguousarray(words).view(np.uint8), bitorder="little")[:count].astype(bool)
        mag = np.repeat(scales, chunk)[:count]
        return np.where(bits, mag, -mag).astype(np.float32)

    for k in range(2):
        a = z_rounds[k, rank] + delta
        hat, words, scales = zo.compress(a, chunk)
        delta = a - hat
        recv_words, recv_scales = exchange_packed(plan, rank, torch.from_numpy(words.view(np.int32)), torch.from_numpy(scales))
        words_s = torch.zeros(n_words, dtype=torch.int32)
        scales_s = torch.zeros(n_chunks, dtype=torch.float32)
        if hi > lo:
            total = np.zeros(hi - lo, np.float64)
            for w in range(world):                         # worker order, binary64
                total += decode(recv_words[w].numpy().view(np.uint32), recv_scales[w].numpy(), lo, hi - lo)
            a_s = (total / world + delta_bar).astype(np.float32)
            hat_s, w_s, s_s = zo.compress(a_s, chunk)
            delta_bar = a_s - hat_s
            wr = plan.words[rank]
            words_s[wr.start:wr.stop] = torch.from_numpy(w_s.view(np.int32))
            scales_s[mine_c.start:mine_c.stop] = torch.from_numpy(s_s)
        gather_server(plan, rank, words_s, scales_s)
        z_bar = decode(words_s.numpy().view(np.uint32), scales_s.numpy(), 0, n)
        want = whole.onebit_allreduce(z_rounds[k])
        assert np.array_equal(z_bar, want), (rank, k)
        assert np.array_equal(words_s.numpy().view(np.uint32), whole.words_server), (rank, k)
        assert np.array_equal(delta, whole.delta[rank]), (rank, k)
        assert np.array_equal(delta_bar, whole.delta_bar[lo:hi]), (rank, k)
    dist.barrier()
    if rank == 0:
        open(os.path.join(out_dir, "ok"), "w").write("ok")
    dist.destroy_process_group()


def test_two_consecutive_rounds_equal_the_single_process_oracle(tmp_path):
    port = _free_port()
    mp.spawn(_round_worker, args=(3, port, 9 * 128 + 50, 128, str(tmp_path)), nprocs=3, join=True)
    assert (tmp_path / "ok").exists()


def test_packed_exchange_three_ranks(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(3, port, 10 * 256 + 77, 256, str(tmp_path)), nprocs=3, join=True)
    assert (tmp_path / "ok").exists()


def test_packed_exchange_more_ranks_than_chunks(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(4, port, 3 * 64 + 5, 64, str(tmp_path)), nprocs=4, join=True)
    assert (tmp_path / "ok").exists()
