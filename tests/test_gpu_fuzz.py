"""Randomised differential test: random sizes, worker counts, chunk sizes, policies, gradient
types and mixes of entry points (fused, two-call, Algorithm 2, host gradients), each case
compared with the oracle after every step.  Seeds are fixed; ZOA_FUZZ_CASES widens the run."""
import os

import numpy as np
import pytest
import torch

from helpers import Pair

pytestmark = pytest.mark.gpu

CHUNKS = [32, 64, 96, 256, 1024, 2048, 2048, 4096, 4096, 8192, 12288, 16384, 16416, 32768, 1 << 20]
DTYPES = [torch.float32, torch.float32, torch.float16, torch.bfloat16]


def _case(seed):
    rng = np.random.default_rng(seed)
    chunk = int(rng.choice(CHUNKS))
    W = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 16, 17, 32, 64]))
    n_chunks = int(rng.integers(1, 12))
    n = min(int(n_chunks * min(chunk, 40000) + rng.integers(0, min(chunk, 5000))), 400_000 // max(1, W // 4))
    n = max(n, 1)
    steps = int(rng.integers(3, 8))
    var_steps = tuple(int(t) for t in range(steps) if rng.random() < 0.4)
    interval = int(rng.choice([1, 1, 2, 3]))
    dtype = DTYPES[int(rng.integers(0, len(DTYPES)))]
    algorithm = "alg2" if rng.random() < 0.25 else "alg1"
    x0 = rng.standard_normal(n) * 0.02
    p = Pair(n, W, chunk, var_steps=var_steps, sync=((0,), (interval,)), x0=x0,
             beta1=float(rng.choice([0.9, 0.5, 0.0])), beta2=float(rng.choice([0.999, 0.9])), eps=float(rng.choice([1e-8, 1e-3])))
    try:
        p.gpu.set_grad_dtype(dtype)
        for t in range(steps):
            lr = float(rng.choice([1e-3, 3e-4, 1e-2]))
            g32 = rng.standard_normal((W, n)).astype(np.float32) * np.float32(10.0 ** rng.integers(-3, 2))
            g32[rng.random((W, n)) < 0.01] *= np.float32(100.0)
            gdev = torch.from_numpy(g32).cuda().to(dtype)
            gref = gdev.float().cpu().numpy()
            sync, var = p.gpu.sync_due(t), p.gpu.var_due(t)
            if algorithm == "alg2":
                p.gpu.alg2_step(list(gdev), lr, t)
                p.cpu.alg2_step(gref, np.float32(lr), var)
            else:
                how = int(rng.integers(0, 3))
                if how == 0:
                    p.gpu.step_auto(list(gdev), lr, t)
                elif how == 1:
                    p.gpu.step(list(gdev), lr, t)
                    if sync:
                        p.gpu.onebit_reduce()
                else:
                    p.gpu.step_host(list(gdev.cpu().pin_memory()), lr, t)
                assert p.cpu.step(gref, np.float32(lr), t, sync, var) == 0
            torch.cuda.synchronize()
            # packed words (bit-exact) and magnitudes are compared whenever the step ran the 1-bit AllReduce
            wire = (not var) if algorithm == "alg2" else sync
            p.compare(f"seed={seed} n={n} W={W} chunk={chunk} {algorithm} {dtype} t={t}", wire=wire)
        p.padding_is_zero()
    finally:
        p.close()      # also checks the device error flag and the guard areas


@pytest.mark.parametrize("seed", range(int(os.environ.get("ZOA_FUZZ_CASES", "40"))))
def test_random_case(seed):
    _case(1000 + seed)
