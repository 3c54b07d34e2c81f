"""0/1 Adam optimizer step for W simulated data-parallel workers on one B200.

`binding` exposes the C ABI of include/zoa.h (libzoa.so, hand-written sm_100a
kernels); `Zoa` is a small convenience wrapper around a handle that takes
torch tensors for the gradients; `synth` builds the seeded synthetic workloads.
"""
from . import binding
from .binding import ZoaError
from .optimizer import Zoa

__all__ = ["binding", "Zoa", "ZoaError"]
