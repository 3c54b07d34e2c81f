"""The C ABI used from plain C: tests/c_client/zoa_client.c is compiled with gcc against
include/zoa.h and libzoa.so (no Python, no torch in that process) and its results are compared
with the oracle."""
import os
import subprocess

import numpy as np
import pytest

from oracle import zoa_oracle as zo
from paper_2202_06009_b200 import build as zoa_build
from helpers import assert_close

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def test_plain_c_program_matches_the_oracle(tmp_path):
    lib = zoa_build.build()
    exe = str(tmp_path / "zoa_client")
    subprocess.check_call(["gcc", "-std=c99", "-O1", "-Wall", "-Werror", os.path.join(ROOT, "tests", "c_client", "zoa_client.c"),
                           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(CUDA, "include"),
                           "-L", os.path.dirname(lib), "-lzoa", "-L", os.path.join(CUDA, "lib64"), "-lcudart",
                           "-Wl,-rpath," + os.path.dirname(lib), "-Wl,-rpath," + os.path.join(CUDA, "lib64"), "-o", exe])
    n, W, chunk, steps, interval = 5 * 2048 + 77, 3, 2048, 6, 2
    var_steps = [0, 2]
    rng = np.random.default_rng(11)
    x0 = (rng.standard_normal(n) * 0.02).astype(np.float32)
    g = rng.standard_normal((steps, W, n)).astype(np.float32)
    with open(tmp_path / "in.bin", "wb") as f:
        np.array([n, W, chunk, steps, interval, len(var_steps)], np.int64).tofile(f)
        np.array(var_steps, np.int64).tofile(f)
        x0.tofile(f)
        g.tofile(f)
    out = subprocess.run([exe, str(tmp_path / "in.bin"), str(tmp_path / "out.bin")], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stderr
    assert out.stdout.startswith(f"steps {steps} syncs {steps // interval}")
    got = np.fromfile(tmp_path / "out.bin", np.float32).reshape(4, n)

    o = zo.Oracle(n, W, chunk, 0.9, 0.999, 1e-8, dtype=np.float32)
    o.set_params(x0)
    for t in range(steps):
        assert o.step(g[t], np.float32(1e-3), t, t % interval == 0, t in var_steps) == 0
    assert_close(got[0], o.x[0], "x[0]")
    assert_close(got[1], o.m[0], "m[0]")
    assert_close(got[2], o.u[0], "u[0]")
    assert_close(got[3], o.v, "v")
