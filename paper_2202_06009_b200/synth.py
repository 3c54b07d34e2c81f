"""Seeded synthetic workloads: parameter-set shapes, T_v / T_u policies as plain
data, and the gradient streams.  Holds none of the method's arithmetic; both the
CUDA path and the test oracle are fed the very same buffers made here.

The paper trains BERT-Base/Large and GPT-2 on text corpora that are not
available here; these workloads keep only the parameter-set shapes (flat
concatenation of the model's tensors) and stand in for the gradient streams with
per-tensor-scaled Gaussian (or Student-t) noise that is partly shared between
the workers.
"""
import math
from dataclasses import dataclass, field
from typing import List, Tuple

import torch

DEFAULT_SEED = 20220206


def _bert_tensors(layers: int, hidden: int, ffn: int, vocab: int = 30522) -> List[int]:
    h = hidden
    t = [vocab * h, 512 * h, 2 * h, h, h]                       # embeddings + LayerNorm
    for _ in range(layers):
        t += [h * h, h] * 4                                     # Q, K, V, output projection
        t += [h, h]                                             # LayerNorm
        t += [h * ffn, ffn, ffn * h, h]                         # feed-forward
        t += [h, h]                                             # LayerNorm
    t += [h * h, h]                                             # pooler
    t += [h * h, h, h, h, vocab, 2 * h, 2]                      # pre-training heads
    return t


def _gpt2_tensors(layers: int = 48, hidden: int = 1600, vocab: int = 50257, ctx: int = 1024) -> List[int]:
    h = hidden
    t = [vocab * h, ctx * h]
    for _ in range(layers):
        t += [h, h, h * 3 * h, 3 * h, h * h, h, h, h, h * 4 * h, 4 * h, 4 * h * h, h]
    t += [h, h]
    return t


@dataclass
class Workload:
    name: str
    tensors: List[int]                 # sizes of the concatenated tensors, in order
    W: int
    chunk: int
    steps: int
    var_steps: Tuple[int, ...]         # T_v
    sync_boundaries: Tuple[int, ...]   # T_u: piece r starts at sync_boundaries[r] ...
    sync_intervals: Tuple[int, ...]    # ... and syncs every sync_intervals[r] steps from there
    shared: float                      # amplitude of the signal all workers share
    noise: float                       # amplitude of the per-worker noise
    noise_kind: str = "gauss"          # "gauss" or "student3" (unit-variance Student-t, 3 d.o.f.)
    tensor_scale: bool = True          # one lognormal(0, 1) scale per tensor
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    lr: float = 1e-3
    x0_std: float = 0.02
    n: int = field(init=False)

    def __post_init__(self):
        self.n = sum(self.tensors)

    def in_T_u(self, t: int) -> bool:
        r = max(k for k, b in enumerate(self.sync_boundaries) if b <= t)
        return (t - self.sync_boundaries[r]) % self.sync_intervals[r] == 0

    def in_T_v(self, t: int) -> bool:
        return t in self.var_steps

    def lr_at(self, t: int) -> float:
        return self.lr


def tiny(n: int = 1 << 20, W: int = 4, chunk: int = 2048, steps: int = 64) -> Workload:
    return Workload("tiny", [n], W, chunk, steps, (0, 1, 2, 4, 8, 16), (0, 16), (1, 2),
                    shared=1.0, noise=0.5, tensor_scale=False)


def bert_base() -> Workload:
    return Workload("bert_base", _bert_tensors(12, 768, 3072), 8, 4096, 200,
                    (0, 1, 2, 4, 8, 16, 32, 64, 128), (0, 64, 128), (1, 2, 4),
                    shared=math.sqrt(0.7), noise=math.sqrt(0.3))


def bert_large() -> Workload:
    return Workload("bert_large", _bert_tensors(24, 1024, 4096), 16, 4096, 100,
                    (0, 1, 2, 4, 8, 16, 32, 64, 128), (0, 64, 128), (1, 2, 4),
                    shared=math.sqrt(0.7), noise=math.sqrt(0.3))


def gpt2_xl() -> Workload:
    return Workload("gpt2_1p5b", _gpt2_tensors(), 4, 8192, 50,
                    (0, 1, 2, 4, 8, 16, 32), (0, 16), (1, 4),
                    shared=math.sqrt(0.7), noise=math.sqrt(0.3), noise_kind="student3")


def scaled(base: Workload, divisor: int, steps: int = None) -> Workload:
    """The same layout with every tensor shrunk by `divisor` (for quick tests)."""
    w = Workload(f"{base.name}/{divisor}", [max(1, s // divisor) for s in base.tensors], base.W, base.chunk,
                 steps or base.steps, base.var_steps, base.sync_boundaries, base.sync_intervals,
                 base.shared, base.noise, base.noise_kind, base.tensor_scale,
                 base.beta1, base.beta2, base.eps, base.lr, base.x0_std)
    return w


WORKLOADS = {"tiny": tiny, "bert_base": bert_base, "bert_large": bert_large, "gpt2_1p5b": gpt2_xl}


def _generator(device, *key) -> torch.Generator:
    g = torch.Generator(device=device)
    seed = 0x9E3779B97F4A7C15
    for k in key:
        seed = (seed * 6364136223846793005 + int(k) + 1442695040888963407) % (1 << 63)
    g.manual_seed(seed)
    return g


def initial_params(wl: Workload, device, seed: int = DEFAULT_SEED) -> torch.Tensor:
    g = _generator(device, seed, 0x7830)
    return torch.randn(wl.n, generator=g, device=device, dtype=torch.float32) * wl.x0_std


def tensor_scales(wl: Workload, seed: int = DEFAULT_SEED) -> List[float]:
    if not wl.tensor_scale:
        return [1.0] * len(wl.tensors)
    g = _generator("cpu", seed, 0x5CA1E)
    return torch.randn(len(wl.tensors), generator=g, dtype=torch.float64).exp().tolist()


class GradientStream:
    """g_t^(i) = sigma_T * (shared * s_t + noise * n_t^(i)) per tensor T, written
    into W preallocated float32 buffers of n elements."""

    def __init__(self, wl: Workload, device, seed: int = DEFAULT_SEED, slice_elems: int = 1 << 26):
        self.wl, self.device, self.seed, self.slice = wl, torch.device(device), seed, slice_elems
        self.bufs = [torch.empty(wl.n, device=device, dtype=torch.float32) for _ in range(wl.W)]
        self._shared = torch.empty(wl.n, device=device, dtype=torch.float32)
        self._scales = tensor_scales(wl, seed)

    def _noise_into(self, out: torch.Tensor, gen: torch.Generator):
        if self.wl.noise_kind == "gauss":
            out.normal_(generator=gen)
            return
        for lo in range(0, out.numel(), self.slice):     # Student-t(3) / sqrt(3), in bounded slices
            part = out[lo:lo + self.slice]
            part.normal_(generator=gen)
            chi = torch.zeros_like(part)
            tmp = torch.empty_like(part)
            for _ in range(3):
                tmp.normal_(generator=gen)
                chi.addcmul_(tmp, tmp)
            part.div_(chi.div_(3.0).sqrt_()).div_(math.sqrt(3.0))

    def fill(self, t: int) -> List[torch.Tensor]:
        wl = self.wl
        self._shared.normal_(generator=_generator(self.device, self.seed, t, 0xFFFF))
        for i, buf in enumerate(self.bufs):
            self._noise_into(buf, _generator(self.device, self.seed, t, i))
            buf.mul_(wl.noise).add_(self._shared, alpha=wl.shared)
            if wl.tensor_scale:
                views, off = [], 0
                for size in wl.tensors:
                    views.append(buf[off:off + size])
                    off += size
                torch._foreach_mul_(views, self._scales)
        return self.bufs
