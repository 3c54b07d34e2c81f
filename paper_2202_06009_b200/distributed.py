"""One worker per GPU: the paper's own mapping of Algorithm 3.

Every rank owns one worker's state (x, m, u, its compression error) and is the
server for a contiguous range of chunks (the server error of that range).  A sync
step is

    local step, pack u + delta                 (zoa_step, zoa_onebit_compress)
    all-to-all: each range's words and scales  -> the range's server
    server part on the own range               (zoa_dist_server_range)
    all-gather of the servers' packed results  -> every worker
    m, x, u from the packed result             (zoa_dist_apply)

so a worker sends n/8 bytes of signs plus one float per chunk and receives the
same, instead of 4n bytes.  The collectives are torch.distributed's (NCCL over
NVLink on GPUs); the arithmetic is the library's kernels.  The exchange itself
(`ExchangePlan`, `exchange_packed`, `gather_server`) works on tensors of any
device, which is how it is tested with the gloo backend.

A second form lets the kernels do both exchanges themselves, as stores through
peer pointers (`PeerTable`, `WorkerPerGpu.step_pushed`):

    local updates + pack, stored into the servers' receive buffers   (zoa_dist_step_pack_push)
    stream_barrier between the ranks
    server part, result stored into every rank's words_s / scales_s  (zoa_dist_server_push)
    stream_barrier
    m, x, u from the packed result                                   (zoa_dist_apply)

No kernel waits for another rank; on a sync step the half-step momentum, model and
buffer are never written (32 bytes per parameter instead of 52).
"""
from dataclasses import dataclass
from typing import List, Sequence

import torch
import torch.distributed as dist

from .sharding import chunk_range


@dataclass
class ExchangePlan:
    """Who serves which chunks, in chunks, words (32 signs) and parameters."""
    n: int
    chunk: int
    world: int
    chunks: List[range]       # chunks[r]: the chunks rank r serves
    words: List[range]        # words[r]: the 32-bit words of those chunks in a worker's packed stream

    @staticmethod
    def make(n: int, chunk: int, world: int) -> "ExchangePlan":
        n_chunks = -(-n // chunk)
        chunks, words = [], []
        for r in range(world):
            c0, c1 = chunk_range(n_chunks, world, r)
            chunks.append(range(c0, c1))
            first = c0 * chunk
            last = min(c1 * chunk, n)
            words.append(range(first // 32, first // 32 + (-(-(last - first) // 32) if last > first else 0)))
        return ExchangePlan(n, chunk, world, chunks, words)

    def max_words(self) -> int:
        return max(len(w) for w in self.words)

    def max_chunks(self) -> int:
        return max(len(c) for c in self.chunks)


def exchange_packed(plan: ExchangePlan, rank: int, words: torch.Tensor, scales: torch.Tensor, group=None):
    """All-to-all of the packed buffers: `words` / `scales` are this worker's whole packed stream;
    returns (recv_words [world][len(plan.words[rank])], recv_scales [world][len(plan.chunks[rank])]),
    row w holding worker w's part of the range this rank serves."""
    world = plan.world
    my_w, my_c = len(plan.words[rank]), len(plan.chunks[rank])
    recv_words = torch.empty((world, my_w), dtype=words.dtype, device=words.device)
    recv_scales = torch.empty((world, my_c), dtype=scales.dtype, device=scales.device)
    total_w, total_c = (plan.n + 31) // 32, -(-plan.n // plan.chunk)
    dist.all_to_all_single(recv_words.view(-1), words[:total_w].contiguous(), [my_w] * world,
                           [len(w) for w in plan.words], group=group)
    dist.all_to_all_single(recv_scales.view(-1), scales[:total_c].contiguous(), [my_c] * world,
                           [len(c) for c in plan.chunks], group=group)
    return recv_words, recv_scales


def gather_server(plan: ExchangePlan, rank: int, words_s: torch.Tensor, scales_s: torch.Tensor, group=None):
    """All-gather of the servers' packed results, in place: on entry `words_s` / `scales_s` hold this
    rank's own range, on return the whole vector's."""
    world = plan.world
    mw, mc = plan.max_words(), plan.max_chunks()
    send_w = torch.zeros(mw, dtype=words_s.dtype, device=words_s.device)
    send_c = torch.zeros(mc, dtype=scales_s.dtype, device=scales_s.device)
    w, c = plan.words[rank], plan.chunks[rank]
    send_w[:len(w)] = words_s[w.start:w.stop]
    send_c[:len(c)] = scales_s[c.start:c.stop]
    all_w = torch.empty((world, mw), dtype=words_s.dtype, device=words_s.device)
    all_c = torch.empty((world, mc), dtype=scales_s.dtype, device=scales_s.device)
    dist.all_gather_into_tensor(all_w.view(-1), send_w, group=group)
    dist.all_gather_into_tensor(all_c.view(-1), send_c, group=group)
    for r in range(world):
        w, c = plan.words[r], plan.chunks[r]
        words_s[w.start:w.stop] = all_w[r, :len(w)]
        scales_s[c.start:c.stop] = all_c[r, :len(c)]


_BARRIER_TOKENS = {}


def stream_barrier(group=None):
    """Orders the ranks on the current CUDA stream with a one-element all-reduce.

    Why this orders the peer stores: torch enqueues the collective behind everything this rank
    has already put on the current stream, and makes the current stream wait for the collective
    before anything enqueued later runs.  The sum a rank receives depends on every rank's input,
    so the collective cannot finish anywhere before every rank has started it, that is, before
    every rank's earlier kernels (and the stores they made into other ranks' memory) are done.
    The host does not block."""
    dev = torch.cuda.current_device()
    token = _BARRIER_TOKENS.get(dev)
    if token is None:
        token = _BARRIER_TOKENS[dev] = torch.zeros(1, dtype=torch.int32, device=torch.device("cuda", dev))
    dist.all_reduce(token, op=dist.ReduceOp.SUM, group=group)


@dataclass
class PeerTable:
    """Device addresses through which every rank stores into the others' buffers.  Entry r belongs
    to rank r: its receive buffers ([world][max_words] uint32, [world][max_chunks] float32; row w
    is filled by worker w) and the whole-vector buffers that receive the servers' results."""
    recv_words: List[int]
    recv_scales: List[int]
    words_s: List[int]
    scales_s: List[int]
    copy_back: bool = False     # words_s / scales_s above are staging buffers, not the handles' own

    @staticmethod
    def local(workers: Sequence["WorkerPerGpu"]) -> "PeerTable":
        """All ranks live in this process (on one GPU): plain device pointers."""
        for w in workers:
            w.alloc_receive_buffers()
        return PeerTable([w.recv_words.data_ptr() for w in workers], [w.recv_scales.data_ptr() for w in workers],
                         [w.opt.device_view("words_s").data_ptr() for w in workers],
                         [w.opt.device_view("scales_s").data_ptr() for w in workers])

    @staticmethod
    def symmetric(worker: "WorkerPerGpu", group=None) -> "PeerTable":
        """One rank per process and GPU: the buffers are carved out of one block of torch's
        symmetric memory, whose rendezvous hands every rank the others' addresses."""
        import torch.distributed._symmetric_memory as symm_mem
        plan, world = worker.plan, worker.world
        mw, mc = plan.max_words(), plan.max_chunks()
        total_w, total_c = (plan.n + 31) // 32, -(-plan.n // plan.chunk)
        sizes = [world * mw, world * mc, total_w, total_c]          # 4-byte elements each
        offsets = [0]
        for sz in sizes:
            offsets.append(offsets[-1] + (sz + 63) // 64 * 64)
        block = symm_mem.empty(offsets[-1], dtype=torch.int32, device=torch.device("cuda", torch.cuda.current_device()))
        block.zero_()
        group = group if group is not None else dist.group.WORLD
        handle = symm_mem.rendezvous(block, group=group)
        worker.symmetric_block = block
        worker.recv_words = block[offsets[0]:offsets[0] + sizes[0]].view(world, mw)
        worker.recv_scales = block[offsets[1]:offsets[1] + sizes[1]].view(torch.float32).view(world, mc)
        worker.staged_words_s = block[offsets[2]:offsets[2] + sizes[2]]
        worker.staged_scales_s = block[offsets[3]:offsets[3] + sizes[3]].view(torch.float32)
        bases = [int(p) for p in handle.buffer_ptrs]
        return PeerTable([b + 4 * offsets[0] for b in bases], [b + 4 * offsets[1] for b in bases],
                         [b + 4 * offsets[2] for b in bases], [b + 4 * offsets[3] for b in bases], copy_back=True)


class WorkerPerGpu:
    """This rank's worker and server shard.  `var_steps` is T_v (kept here: the mean gradient of a
    T_v step comes from an all-reduce, not from the handle); the sync policy lives in the handle."""

    def __init__(self, n_params: int, chunk: int, rank: int, world: int, var_steps: Sequence[int] = (),
                 sync_boundaries: Sequence[int] = (0,), sync_intervals: Sequence[int] = (1,),
                 beta1=0.9, beta2=0.999, eps=1e-8, group=None):
        from .optimizer import Zoa
        self.rank, self.world, self.group = rank, world, group
        self.plan = ExchangePlan.make(n_params, chunk, world)
        self.opt = Zoa(n_params, 1, beta1, beta2, eps, chunk)
        self.opt.set_policies((), sync_boundaries, sync_intervals)
        self.var_steps = frozenset(var_steps)
        self.recv_words = self.recv_scales = None
        self.staged_words_s = self.staged_scales_s = None

    def close(self):
        self.opt.close()

    # -- the phases of a sync, separately, so that a test can stand in for the collectives --
    def pack(self):
        self.opt.onebit_compress()
        return self.opt.device_view("words_w", 0), self.opt.device_view("scales_w", 0)

    def serve(self, recv_words: torch.Tensor, recv_scales: torch.Tensor):
        from . import binding as B
        c = self.plan.chunks[self.rank]
        B.zoa_dist_server_range(self.opt.h, recv_words.data_ptr(), recv_words.stride(0), recv_scales.data_ptr(),
                                recv_scales.stride(0), self.world, c.start, len(c),
                                torch.cuda.current_stream().cuda_stream)
        return self.opt.device_view("words_s"), self.opt.device_view("scales_s")

    def apply(self):
        from . import binding as B
        B.zoa_dist_apply(self.opt.h, torch.cuda.current_stream().cuda_stream)

    def variance(self, g_bar: torch.Tensor):
        from . import binding as B
        B.zoa_dist_variance(self.opt.h, g_bar.data_ptr(), torch.cuda.current_stream().cuda_stream)

    # -- one iteration of Algorithm 1 on this rank ------------------------------------
    def step(self, grad: torch.Tensor, lr: float, t: int):
        self.opt.step([grad], lr, t)
        if t in self.var_steps:
            g_bar = grad.clone()
            dist.all_reduce(g_bar, op=dist.ReduceOp.SUM, group=self.group)
            g_bar.div_(self.world)
            self.variance(g_bar)
        if self.opt.sync_due(t):
            words, scales = self.pack()
            recv_words, recv_scales = exchange_packed(self.plan, self.rank, words, scales, self.group)
            words_s, scales_s = self.serve(recv_words, recv_scales)
            gather_server(self.plan, self.rank, words_s, scales_s, self.group)
            self.apply()

    # -- the same round with the exchanges done by the kernels' own stores -------------
    def alloc_receive_buffers(self):
        if self.recv_words is None:
            dev = torch.device("cuda", torch.cuda.current_device())
            self.recv_words = torch.zeros((self.world, max(1, self.plan.max_words())), dtype=torch.int32, device=dev)
            self.recv_scales = torch.zeros((self.world, max(1, self.plan.max_chunks())), dtype=torch.float32, device=dev)

    def _push_tables(self, peers: PeerTable):
        """This rank's row in every server's receive buffers (None where a rank serves nothing)."""
        mw, mc = self.recv_words.shape[1], self.recv_scales.shape[1]
        begin = [c.start for c in self.plan.chunks] + [self.plan.chunks[-1].stop]
        words = [peers.recv_words[s] + 4 * self.rank * mw if len(self.plan.chunks[s]) else None for s in range(self.world)]
        scales = [peers.recv_scales[s] + 4 * self.rank * mc if len(self.plan.chunks[s]) else None for s in range(self.world)]
        return begin, words, scales

    def push_pack(self, peers: PeerTable, grad: torch.Tensor = None, lr: float = 0.0, t: int = 0):
        """Worker side, stored into the servers' receive buffers; with `grad` it also stands for the
        local updates of the sync step t."""
        from . import binding as B
        begin, words, scales = self._push_tables(peers)
        stream = torch.cuda.current_stream().cuda_stream
        if grad is None:
            B.zoa_dist_pack_push(self.opt.h, begin, words, scales, stream)
        else:
            B.zoa_dist_step_pack_push(self.opt.h, grad.data_ptr(), lr, t, begin, words, scales, stream)

    def push_serve(self, peers: PeerTable):
        from . import binding as B
        c = self.plan.chunks[self.rank]
        B.zoa_dist_server_push(self.opt.h, self.recv_words.data_ptr(), self.recv_words.stride(0),
                               self.recv_scales.data_ptr(), self.recv_scales.stride(0), self.world, c.start, len(c),
                               peers.words_s, peers.scales_s, torch.cuda.current_stream().cuda_stream)

    def step_pushed(self, grad: torch.Tensor, lr: float, t: int, peers: PeerTable, barrier=None):
        """One iteration of Algorithm 1 on this rank.  `barrier()` must order the ranks on the
        current stream: nothing enqueued after it may start before every rank has finished what it
        enqueued before.  Default: `stream_barrier` on this worker's group."""
        if barrier is None:
            barrier = lambda: stream_barrier(self.group)
        if not self.opt.sync_due(t):
            self.opt.step([grad], lr, t)
        else:
            self.push_pack(peers, grad, lr, t)
        if t in self.var_steps:
            g_bar = grad.clone()
            dist.all_reduce(g_bar, op=dist.ReduceOp.SUM, group=self.group)
            g_bar.div_(self.world)
            self.variance(g_bar)
        if self.opt.sync_due(t):
            barrier()
            self.push_serve(peers)
            barrier()
            if peers.copy_back:
                self.opt.device_view("words_s")[:self.staged_words_s.numel()].copy_(self.staged_words_s)
                self.opt.device_view("scales_s")[:self.staged_scales_s.numel()].copy_(self.staged_scales_s)
            self.apply()
