"""The N > 1 path on CPU: two gloo ranks each own a chunk range of one flat
vector, run the method on their range alone (here with the oracle standing in
for a GPU's handle) and never exchange data; gathered, the pieces equal the
single-process run."""
import os
import sys

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))



def _free_port():
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]

def _load_sharding():
    import importlib.util
    spec = importlib.util.spec_from_file_location("_sharding", os.path.join(ROOT, "paper_2202_06009_b200", "sharding.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def _run(x0, g, lo, hi, W, chunk, T):
    from oracle import zoa_oracle as zo
    o = zo.Oracle(hi - lo, W, chunk)
    o.set_params(x0[lo:hi])
    for t in range(T):
        o.step(g[t][:, lo:hi], np.float32(1e-3), t, t % 2 == 0, t < 3)
    return o


def _worker(rank, world, port, n, W, chunk, T, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sh = _load_sharding()
    rng = np.random.default_rng(123)                      # same seeded inputs on every rank
    x0 = rng.standard_normal(n).astype(np.float32)
    g = rng.standard_normal((T, W, n)).astype(np.float32)
    lo, hi = sh.param_range(n, chunk, world, rank)
    ranges = [None] * world
    dist.all_gather_object(ranges, (lo, hi))              # bookkeeping only, no optimizer data
    assert ranges[0][0] == 0 and ranges[-1][1] == n
    assert all(ranges[r][1] == ranges[r + 1][0] and ranges[r][0] % chunk == 0 for r in range(world - 1))
    o = _run(x0, g, lo, hi, W, chunk, T)
    pieces = [None] * world
    dist.all_gather_object(pieces, {k: getattr(o, k) for k in ("x", "m", "u", "delta", "v", "delta_bar")})
    # max-over-ranks timing, as bench.py does it
    import torch
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert t.item() == world
    if rank == 0:
        full = _run(x0, g, 0, n, W, chunk, T)
        for k in ("x", "m", "u", "delta"):
            assert np.array_equal(np.concatenate([p[k] for p in pieces], axis=1), getattr(full, k)), k
        for k in ("v", "delta_bar"):
            assert np.array_equal(np.concatenate([p[k] for p in pieces]), getattr(full, k)), k
        open(os.path.join(out_dir, "ok"), "w").write("ok")
    dist.destroy_process_group()


def test_two_ranks_own_chunk_ranges(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, 5 * 256 + 77, 3, 256, 6, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok").exists()


def test_chunk_ranges_cover_without_overlap():
    sh = _load_sharding()
    for n_chunks in (1, 2, 7, 82087):
        for world in (1, 2, 3, 8):
            edges = [sh.chunk_range(n_chunks, world, r) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == n_chunks
            assert all(a[1] == b[0] for a, b in zip(edges, edges[1:]))
            sizes = [b - a for a, b in edges]
            assert max(sizes) - min(sizes) <= 1
    assert sh.param_range(1000, 256, 2, 1) == (512, 1000)
