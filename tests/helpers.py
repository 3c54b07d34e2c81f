"""Shared machinery of the GPU parity tests: drive the CUDA library and the CPU
oracle with the very same float32 buffers and compare every state."""
import numpy as np
import torch

from oracle import zoa_oracle as zo
from paper_2202_06009_b200 import Zoa

RTOL, ATOL = 1e-5, 1e-7      # the tolerance the benchmark spec states for the float32 states
FLOAT_STATES = ("x", "m", "u", "delta_w")


def assert_close(got, want, what):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    assert got.shape == want.shape, what
    same = (np.isnan(got) & np.isnan(want)) | (got == want)      # NaN with NaN, equal infinities
    with np.errstate(invalid="ignore"):
        err = np.abs(got - want)
        bad = ~(err <= ATOL + RTOL * np.abs(want)) & ~same
    if bad.any():
        k = int(np.argmax(np.where(bad, err, 0)))
        raise AssertionError(f"{what}: {int(bad.sum())} of {got.size} outside tolerance; worst at {k}: "
                             f"got {got.flat[k]!r}, want {want.flat[k]!r}")


class Pair:
    """A zoa handle and an oracle state for the same problem."""

    def __init__(self, n, W, chunk, beta1=0.9, beta2=0.999, eps=1e-8, var_steps=(), sync=((0,), (1,)), x0=None):
        self.n, self.W, self.chunk = n, W, chunk
        self.gpu = Zoa(n, W, beta1, beta2, eps, chunk)
        self.gpu.set_pipeline("force")          # small test problems still go through the ring kernels
        self.gpu.set_policies(var_steps, sync[0], sync[1])
        self.cpu = zo.Oracle(n, W, chunk, beta1, beta2, eps, dtype=np.float32)
        if x0 is not None:
            x0 = np.asarray(x0, np.float32)
            self.gpu.set_params(torch.from_numpy(x0))
            self.cpu.set_params(x0)

    def close(self):
        try:
            self.gpu.check_device()      # also verifies the guard areas around every state buffer
        finally:
            self.gpu.close()

    def step(self, g, lr, t, mode):
        """g: float32 array [W][n] (numpy).  mode: 'fused' (zoa_step_auto) or 'two_call'."""
        g = np.ascontiguousarray(g, np.float32)
        gd = torch.from_numpy(g).cuda()
        sync, var = self.gpu.sync_due(t), self.gpu.var_due(t)
        if mode == "fused":
            self.gpu.step_auto(list(gd), lr, t)
        else:
            self.gpu.step(list(gd), lr, t)
            if sync:
                self.gpu.onebit_reduce()
        torch.cuda.synchronize()
        rc = self.cpu.step(g, np.float32(lr), t, sync, var)
        assert rc == 0
        return sync, var

    def compare(self, what="", wire=True):
        o, g = self.cpu, self.gpu
        for i in range(self.W):
            assert_close(g.read("x", i), o.x[i], f"{what} x[{i}]")
            assert_close(g.read("m", i), o.m[i], f"{what} m[{i}]")
            assert_close(g.read("u", i), o.u[i], f"{what} u[{i}]")
            assert_close(g.read("delta_w", i), o.delta[i], f"{what} delta_w[{i}]")
        assert_close(g.read("v"), o.v, f"{what} v")
        assert_close(g.read("delta_s"), o.delta_bar, f"{what} delta_s")
        assert_close(g.read("x_sync"), o.x_sync, f"{what} x_sync")
        if wire:
            for i in range(self.W):
                assert np.array_equal(g.read("words_w", i), o.words_worker[i]), f"{what} words_w[{i}]"
                assert_close(g.read("scales_w", i), o.scales_worker[i], f"{what} scales_w[{i}]")
            assert np.array_equal(g.read("words_s"), o.words_server), f"{what} words_s"
            assert_close(g.read("scales_s"), o.scales_server, f"{what} scales_s")

    def padding_is_zero(self):
        g = self.gpu
        pad = (-self.n) % 128
        if pad == 0:
            return
        for name in ("x", "m", "u", "delta_w"):
            for i in range(self.W):
                assert not g.read(name, i, self.n, pad).any(), f"padding of {name}[{i}] was written"
        for name in ("v", "delta_s", "x_sync"):
            assert not g.read(name, 0, self.n, pad).any(), f"padding of {name} was written"
