#!/usr/bin/env python
"""Benchmark of the 0/1 Adam optimizer-step path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload bert_large]
    python bench.py --impl reference ...        # the CPU oracle on the host cores

A step is one iteration of Algorithm 1 for all W workers under the workload's
own T_u / T_v policies (fused sync kernel on sync steps, local-step kernel
otherwise, variance update where due), over one batch of synthetic gradients
that is already resident in device memory.  Prints ONE JSON line (rank 0).
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "optimizer step throughput (params*workers/s)"
UNIT = "params*workers/s"
FALLBACK_HBM_GBS = 6650.0
# Measured DRAM bytes (ncu dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic bytes of one launch, per
# kernel, each from a capture on the BERT-Large-shaped layout shrunk 16x (traffic is proportional to n*W, so
# the ratio carries to a full launch), with the summary under profiles/ that holds it.  A kernel without a
# capture reports traffic null.
DRAM_TRAFFIC_RATIO = {
    "step_sync_pipelined_kernel": (0.995, "step_sync_pipelined_kernel_bert_large_div16.md"),
    "local_step_pipelined_kernel": (0.994, "step_sync_pipelined_kernel_bert_large_div16.md"),
    "step_sync_kernel": (0.995, "step_sync_kernel_alg2_compressed_kernel_chunk_per_block_bert_large_div16.md"),
    "step_sync_kernel@16384": (1.004, "step_sync_kernel_alg2_compressed_kernel_chunk_per_block_bert_large_div16.md"),
    "alg2_compressed_kernel": (1.007, "step_sync_kernel_alg2_compressed_kernel_chunk_per_block_bert_large_div16.md"),
    "alg2_pipelined_kernel": (0.994, "alg2_kernels_bert_large_div16.md"),
    "alg2_full_kernel": (0.992, "alg2_kernels_bert_large_div16.md"),
    "local_step_pipelined_kernel + compress_kernel + reduce_pipelined_kernel": (0.987, "compress_kernel_reduce_pipelined_kernel_two_call_bert_large_div16.md"),
    "lc_worker_pack_kernel + lc_server_pack_kernel + dist_apply_kernel (large-chunk kernels)": (1.004, "large_chunk_kernels_whole_vector_bert_large_div16.md"),
}


# ---- byte model: what the method must move, per launch -------------------------
def sync_step_bytes(n, W, chunk, g_bytes=4):
    """Fused sync step: per parameter and worker read g, m, u, delta (16 B), write
    delta, x, m, u (16 B) and 1 sign bit, plus one scale per chunk; per parameter
    read delta_bar, v, x_sync (12 B), write delta_bar, x_sync (8 B) and 1 sign bit."""
    n_chunks = -(-n // chunk)
    return n * W * (28 + g_bytes + 1 / 8) + n_chunks * W * 4 + n * (20 + 1 / 8) + n_chunks * 4


def local_step_bytes(n, W, g_bytes=4):
    """Local step: per parameter and worker read g, m, x, u and write m, x, u (28 B); v read once."""
    return n * W * (24 + g_bytes) + n * 4


def variance_bytes(n, W):
    return n * W * 4 + n * 8


def two_call_sync_bytes(n, W, chunk, g_bytes=4):
    """zoa_step then zoa_onebit_reduce: the local step writes m, x, u (24 + g B in, 12 B out),
    the compress kernel reads u, delta and writes delta and the packed form (12 1/8 B), the
    reduce kernel reads the packed form and writes m, x, u (12 1/8 B) plus the per-parameter
    server traffic (20 1/8 B)."""
    n_chunks = -(-n // chunk)
    return (local_step_bytes(n, W, g_bytes) + n * W * (12 + 1 / 8) + 4 * n_chunks * W
            + n * W * (12 + 1 / 8) + 4 * n_chunks * W + n * (20 + 1 / 8) + 4 * n_chunks)


def alg2_compressed_bytes(n, W, chunk, g_bytes=4):
    """Algorithm 2, compressed step: per parameter and worker read g, delta, m, x (16 B), write
    delta, m, x (12 B) and 1 sign bit + a scale per chunk; per parameter read delta_bar, v,
    write delta_bar (12 B) and 1 sign bit."""
    n_chunks = -(-n // chunk)
    return n * W * (24 + g_bytes + 1 / 8) + n_chunks * W * 4 + n * (12 + 1 / 8) + n_chunks * 4


def alg2_full_bytes(n, W, g_bytes=4):
    """Algorithm 2, T_v step: per parameter and worker read g, m, x, write m, x (20 B); v in and out."""
    return n * W * (16 + g_bytes) + n * 8


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---- clocks during the timed region ----------------------------------------------
class ClockSampler:
    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._dev, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                 "sw_thermal_slowdown": 0x20, "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._dev, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._dev)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._dev)
                self.reasons.update(k for k, bit in names.items() if mask & bit)
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        if self._nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---- which steps are timed, and the config block both arms print ---------------------------
def step_window(wl, K):
    """The K step indices a run times.  K >= the workload's own length: its whole schedule from
    t = 0.  Shorter runs start four steps before the schedule's first local step, so that the window
    holds sync steps, sync + variance steps and local steps (the first steps of every schedule are
    all sync steps)."""
    if K >= wl.steps:
        return list(range(K))
    first_local = next((t for t in range(wl.steps) if not wl.in_T_u(t)), 0)
    t0 = max(0, first_local - 4)
    return list(range(t0, t0 + K))


def config_block(wl, args, steps, world):
    kinds = [("sync" if wl.in_T_u(t) else "local") + ("+var" if wl.in_T_v(t) else "") for t in steps]
    mix = ", ".join(f"{kinds.count(k)} {k}" for k in sorted(set(kinds)))
    return {"workload": wl.name, "n_params": wl.n, "W": wl.W, "chunk": wl.chunk,
            "algorithm": "Algorithm 1 (0/1 Adam)" if args.algorithm == "alg1" else
                         "Algorithm 2 (gradients through the 1-bit AllReduce, full precision on T_v steps)",
            "schedule": f"t={steps[0]}..{steps[-1]} of the workload's T_u/T_v policies ({mix})",
            "grad_dtype": args.grad_dtype,
            "l2": "inputs larger than L2 (gradients and state are read once per step)",
            "parallelism": f"{world} x independent chunk ranges, no collective"}


# ---- the CPU oracle, timed as it stands (baseline and --impl reference) ---------------
def time_oracle(wl, steps, grads_of, x0, budget_elems, algorithm="alg1"):
    """Times the oracle (oracle/zoa_oracle.c, float build, untouched and single-threaded) on a
    slice of the workload: one oracle instance per chunk range on every core the process may
    use, each called from its own thread (the C call releases the interpreter lock).
    grads_of(t) returns the step's W gradient buffers (the ones the CUDA arm consumes for that
    t); their first d elements are copied to the host, untimed.  Returns
    (params*workers/s, cores, description, seconds per step scaled to the full vector)."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor
    from oracle import zoa_oracle as zo

    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    # slice: a chunk range per core (4 Mi parameters at most), about 10-30 s of oracle work in all
    per = max(wl.chunk, min(budget_elems // cores, 1 << 22) // wl.chunk * wl.chunk)
    if per * cores > wl.n:
        per = max(wl.chunk, wl.n // cores // wl.chunk * wl.chunk)
    if per * cores > wl.n:
        cores = max(1, wl.n // per)
    if per > wl.n:
        per, cores = wl.n, 1
    d = per * cores
    x0 = np.asarray(x0[:d].cpu() if hasattr(x0, "cpu") else x0[:d], np.float32)
    oracles = []
    for c in range(cores):
        o = zo.Oracle(per, wl.W, wl.chunk, wl.beta1, wl.beta2, wl.eps, dtype=np.float32)
        for a in (o.x, o.m, o.u, o.delta, o.v, o.delta_bar, o.x_sync, o.z_hat, o.u_bar):
            a.fill(0)                                    # touch every page before the clock starts
        o.set_params(x0[c * per:(c + 1) * per])
        oracles.append(o)
    host = np.empty((wl.W, d), np.float32)
    dt = 0.0
    with ThreadPoolExecutor(cores) as pool:
        for t in steps:
            for i, g in enumerate(grads_of(t)):
                host[i] = g[:d].float().cpu().numpy()
            parts = [np.ascontiguousarray(host[:, c * per:(c + 1) * per]) for c in range(cores)]
            lr = np.float32(wl.lr_at(t))
            if algorithm == "alg2":
                call = lambda c: oracles[c].alg2_step(parts[c], lr, wl.in_T_v(t))
            else:
                call = lambda c: oracles[c].step(parts[c], lr, t, wl.in_T_u(t), wl.in_T_v(t))
            t0 = time.perf_counter()
            list(pool.map(call, range(cores)))
            dt += time.perf_counter() - t0
    n_sync = sum(wl.in_T_u(t) for t in steps)
    desc = (f"first {d} parameters x {wl.W} workers of {wl.name} ({cores} chunk ranges of {per}, one oracle instance and "
            f"one thread per core), steps t={steps[0]}..{steps[-1]} of its schedule ({n_sync} sync, {len(steps) - n_sync} local) "
            f"on the gradient buffers the CUDA arm consumes for those steps, oracle/zoa_oracle.c float build")
    return d * wl.W * len(steps) / dt, cores, desc, dt / len(steps) * (wl.n / d)


def oracle_inputs(wl, synth, seed):
    """The gradient stream and x_0 of the CUDA arm, regenerated from the same seeds (on the GPU when
    there is one, so that the oracle sees the very same bits; on the host otherwise)."""
    import torch
    if torch.cuda.is_available():
        stream = synth.GradientStream(wl, "cuda", seed)
        return stream.fill, synth.initial_params(wl, "cuda", seed), "generated on the GPU by the CUDA arm's seeded stream"
    # no CUDA device: only a slice-sized layout is generated, from the host generator
    small = synth.Workload(wl.name, [min(wl.n, 1 << 25)], wl.W, wl.chunk, wl.steps, wl.var_steps, wl.sync_boundaries,
                           wl.sync_intervals, wl.shared, wl.noise, wl.noise_kind, False)
    stream = synth.GradientStream(small, "cpu", seed)
    return stream.fill, synth.initial_params(small, "cpu", seed), "generated on the host (no CUDA device)"


def run_reference(args, wl, synth):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = step_window(wl, args.steps)
    timed = steps[:max(1, min(len(steps), args.cpu_steps))]
    grads_of, x0, how = oracle_inputs(wl, synth, synth.DEFAULT_SEED)
    for _ in range(min(args.warmup, 1)):
        time_oracle(wl, timed[:1], grads_of, x0, 1 << 20, args.algorithm)
    value, cores, desc, s_per_step = time_oracle(wl, timed, grads_of, x0, args.cpu_sample, args.algorithm)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": s_per_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": config_block(wl, args, steps, int(os.environ.get("WORLD_SIZE", "1"))),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc + "; inputs " + how},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0,
            "note": f"each timed step is a bounded sample (the first {len(timed)} of the {len(steps)} step indices, a slice of "
                    "the parameters); ms_per_step is the sampled time per step scaled to the full parameter count"}
    print(json.dumps(line))


# ---- the CUDA path -------------------------------------------------------------------
def run_ours(args, wl):
    import torch
    import torch.distributed as dist
    from paper_2202_06009_b200 import Zoa, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    # Under torchrun the process group is set up even for one rank, so that the barrier and the
    # max-over-ranks reduction of the N > 1 launch are the same code at every N.
    use_dist = world > 1 or ("MASTER_ADDR" in os.environ and "RANK" in os.environ)
    if use_dist:
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", local_rank))

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    # Every rank owns a contiguous chunk range of an N-times larger flat vector: the
    # method is chunk-local, so there is no exchange between ranks (weak scaling).
    seed = synth.DEFAULT_SEED + rank
    opt = Zoa(wl.n, wl.W, wl.beta1, wl.beta2, wl.eps, wl.chunk)
    opt.set_params(synth.initial_params(wl, "cuda", seed))
    opt.set_policies(wl.var_steps, wl.sync_boundaries, wl.sync_intervals)
    if args.no_pipeline:
        opt.set_pipeline(False)
    stream = synth.GradientStream(wl, "cuda", seed)
    from paper_2202_06009_b200 import binding as B

    gdt = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[args.grad_dtype]
    g_bytes = 4 if gdt == torch.float32 else 2
    opt.set_grad_dtype(gdt)
    g16 = None if g_bytes == 4 else [torch.empty(wl.n, device="cuda", dtype=gdt) for _ in range(wl.W)]

    def batch(t):
        """The step's gradients, resident in device memory in the dtype the handle expects (untimed)."""
        bufs = stream.fill(t)
        if g16 is None:
            return bufs
        for dst, src in zip(g16, bufs):
            dst.copy_(src)
        return g16

    K, Wu = args.steps, max(args.warmup, 3)
    steps = step_window(wl, K)
    t_first = steps[0]

    def one_step(bufs, t):
        if args.algorithm == "alg2":
            opt.alg2_step(bufs, wl.lr_at(t), t)
            return "alg2_full" if wl.in_T_v(t) else "alg2_compressed"
        if args.two_call and wl.in_T_u(t):
            opt.step(bufs, wl.lr_at(t), t)
            opt.onebit_reduce()
            return "two_call_sync" + ("+var" if wl.in_T_v(t) else "")
        opt.step_auto(bufs, wl.lr_at(t), t)
        return ("sync" if wl.in_T_u(t) else "local") + ("+var" if wl.in_T_v(t) else "")

    # warm-up: the local-step kernel once, then the Wu steps of the schedule that precede the window
    # (or its first Wu steps again when the window starts at 0), with the step counter rewound
    # after each part (timing does not depend on the values in the state)
    opt.step(batch(0), wl.lr, 0)
    B.zoa_set_scalars(opt.h, 0.0, 0, -1)
    for t in (range(t_first - Wu, t_first) if t_first >= Wu else range(Wu)):
        one_step(batch(t), t)
    if t_first < Wu:
        B.zoa_set_scalars(opt.h, 0.0, 0, -1)
    barrier()

    launches0 = opt.stats()["n_launches"]
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    kinds = []
    with ClockSampler(local_rank) as clocks:
        barrier()
        wall0 = time.perf_counter()
        for k, t in enumerate(steps):
            bufs = batch(t)                               # untimed: the batch is resident before the step starts
            ev[k][0].record()
            kinds.append(one_step(bufs, t))
            ev[k][1].record()
        barrier()
        wall = time.perf_counter() - wall0
    opt.check_device()
    ms = [a.elapsed_time(b) for a, b in ev]
    total_ms = sum(ms)
    if use_dist:
        tt = torch.tensor([total_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt.item())
    launches = opt.stats()["n_launches"] - launches0

    by_kind = {}
    for k, m in zip(kinds, ms):
        by_kind.setdefault(k, []).append(m)
    peak, peak_kind = measured_hbm_peak()
    bytes_of = {"sync": sync_step_bytes(wl.n, wl.W, wl.chunk, g_bytes), "local": local_step_bytes(wl.n, wl.W, g_bytes)}
    # the variance update needs nothing beyond writing v_{t+1}: g and v are read anyway
    bytes_of["sync+var"] = bytes_of["sync"] + wl.n * 4
    bytes_of["local+var"] = bytes_of["local"] + wl.n * 4
    bytes_of["two_call_sync"] = two_call_sync_bytes(wl.n, wl.W, wl.chunk, g_bytes)
    bytes_of["two_call_sync+var"] = bytes_of["two_call_sync"] + wl.n * 4
    bytes_of["alg2_compressed"] = alg2_compressed_bytes(wl.n, wl.W, wl.chunk, g_bytes)
    bytes_of["alg2_full"] = alg2_full_bytes(wl.n, wl.W, g_bytes)
    step_types = {k: {"count": len(v), "ms": statistics.mean(v), "ms_median": statistics.median(v), "algorithmic_GB": bytes_of[k] / 1e9,
                      "GBps": bytes_of[k] / 1e6 / statistics.mean(v)} for k, v in by_kind.items()}
    total_bytes = sum(bytes_of[k] for k in kinds)
    dominant = next((k for k in ("sync", "sync+var", "two_call_sync", "alg2_compressed") if k in by_kind), kinds[0])
    achieved = bytes_of[dominant] / 1e6 / statistics.mean(by_kind[dominant])
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    # which kernels the library picks (mirrors its dispatch): ring kernels once every SM has a few units
    ring_chunks = (128, 256, 512, 1024, 2048, 4096, 8192, 16384)
    uses_ring = (not args.no_pipeline and wl.chunk in ring_chunks and wl.n // max(wl.chunk, 2048) >= 4 * sm_count)
    fused_ring = uses_ring and wl.chunk <= 8192          # chunk 16384: the chunk-per-block kernel is the faster one
    sync_kernel = "step_sync_pipelined_kernel" if fused_ring else "step_sync_kernel"
    if wl.chunk > 16384:
        sync_kernel = "lc_worker_pack_kernel + lc_server_pack_kernel + dist_apply_kernel (large-chunk kernels)"
    alg2_ring = uses_ring and wl.chunk in (2048, 4096, 8192)
    local_ring = not args.no_pipeline and wl.n // 2048 >= 4 * sm_count
    kernel_of = {"sync": sync_kernel, "sync+var": sync_kernel,
                 "two_call_sync": ("local_step_pipelined_kernel" if local_ring else "local_step_kernel") + " + compress_kernel + "
                                  + ("reduce_pipelined_kernel" if uses_ring else "reduce_kernel"),
                 "alg2_compressed": "alg2_pipelined_kernel" if alg2_ring else "alg2_compressed_kernel",
                 "alg2_full": "alg2_full_kernel"}
    kernel = kernel_of.get(dominant, "local_step_pipelined_kernel" if local_ring else "local_step_kernel")
    ratio, summary = DRAM_TRAFFIC_RATIO.get(f"{kernel}@{wl.chunk}", DRAM_TRAFFIC_RATIO.get(kernel, (None, None)))
    roofline = {"bound": "hbm", "kernel": kernel,
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": f"of {peak_kind}", "frac_of_8TBps_nominal": achieved / 8000.0,
                "traffic": ratio * bytes_of[dominant] if ratio else None,
                "traffic_how": (f"ncu capture of the same kernel on the layout shrunk 16x (profiles/{summary}: DRAM bytes = "
                                f"{ratio} x algorithmic), scaled by n*W") if ratio else "no ncu capture of this kernel",
                "launch_ms": statistics.mean(by_kind[dominant]),
                "algorithmic_bytes_per_launch": bytes_of[dominant]}

    # ---- end to end: host gradients in, worker 0's model out, through zoa_step_host ----
    e2e = None
    if args.e2e_steps > 0 and args.algorithm == "alg1":
        ke = max(1, min(args.e2e_steps, K))
        host_g = [torch.empty(wl.n, dtype=gdt, pin_memory=True) for _ in range(wl.W)]   # every worker's own pinned buffer
        for dst, src in zip(host_g, batch(0)):
            dst.copy_(src)
        host_x = torch.empty(wl.n, dtype=torch.float32, pin_memory=True)
        B.zoa_set_scalars(opt.h, 0.0, 0, -1)
        opt.step_host(host_g, wl.lr, 0, host_x)           # allocates the staging area; untimed
        B.zoa_set_scalars(opt.h, 0.0 if wl.in_T_u(steps[0]) else wl.lr, 0, -1)
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for t in steps[:ke]:
            opt.step_host(host_g, wl.lr_at(t), t, host_x)
        b.record()
        barrier()
        e_ms = a.elapsed_time(b)
        if use_dist:
            tt = torch.tensor([e_ms], device="cuda", dtype=torch.float64)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            e_ms = float(tt.item())
        e2e = {"value": wl.n * wl.W * ke * world / (e_ms / 1e3), "unit": UNIT,
               "h2d_bytes_per_step": wl.n * wl.W * g_bytes, "d2h_bytes_per_step": wl.n * 4, "steps": ke,
               "ms_per_step": e_ms / ke,
               "how": "zoa_step_host: the W workers' gradients copied from W pinned host buffers in eight chunk "
                      "ranges overlapped with the step's kernels, worker 0's model copied back to pinned host memory"}
    opt.close()

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            timed = steps[:max(1, min(len(steps), args.cpu_steps))]
            value, cores, desc, _ = time_oracle(wl, timed, stream.fill, synth.initial_params(wl, "cuda", seed),
                                                args.cpu_sample, args.algorithm)
            cpu = {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
        line = {"metric": METRIC, "value": wl.n * wl.W * K * world / (total_ms / 1e3), "unit": UNIT,
                "n_gpus": world, "steps": K, "warmup": Wu, "ms_per_step": total_ms / K,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "grad_dtype": args.grad_dtype,
                "config": config_block(wl, args, steps, world),
                "hbm_GBps": total_bytes / 1e6 / total_ms, "hbm_frac_of_measured_peak": total_bytes / 1e6 / total_ms / peak,
                "step_types": step_types, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
                "gpu_launches": launches, "clocks": clocks.summary(), "wall_s_timed_region": wall}
        print(json.dumps(line))
    if use_dist:
        dist.destroy_process_group()


# ---- the paper's own mapping: one worker per GPU, packed buffers exchanged --------------------
def run_worker_per_gpu(args, wl):
    """Every rank is one worker (W = number of ranks) and the server of a chunk range; sync steps
    exchange packed words and magnitudes through torch.distributed.  Strong scaling in the
    paper's sense: the parameter vector is fixed, workers are added."""
    import torch
    import torch.distributed as dist
    from paper_2202_06009_b200 import synth
    from paper_2202_06009_b200.distributed import WorkerPerGpu

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29555")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", local_rank))
    w = WorkerPerGpu(wl.n, wl.chunk, rank, world, wl.var_steps, wl.sync_boundaries, wl.sync_intervals,
                     wl.beta1, wl.beta2, wl.eps)
    w.opt.set_params(synth.initial_params(wl, "cuda"))
    one = synth.Workload(wl.name, wl.tensors, 1, wl.chunk, wl.steps, wl.var_steps, wl.sync_boundaries, wl.sync_intervals,
                         wl.shared, wl.noise, wl.noise_kind, wl.tensor_scale)
    stream = synth.GradientStream(one, "cuda", synth.DEFAULT_SEED + rank)
    K, Wu = args.steps, max(args.warmup, 3)
    if args.exchange == "push":          # the kernels store into the peers' buffers themselves
        from paper_2202_06009_b200.distributed import PeerTable
        peers = PeerTable.symmetric(w)
        step = lambda g, lr, t: w.step_pushed(g, lr, t, peers)      # ranks ordered by a one-element all-reduce on the stream
    else:
        step = w.step
    for t in range(Wu):
        step(stream.fill(t)[0], wl.lr_at(t), t)
    from paper_2202_06009_b200 import binding as B
    B.zoa_set_scalars(w.opt.h, 0.0, 0, -1)
    dist.barrier(); torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for t in range(K):
        g = stream.fill(t)[0]
        ev[t][0].record()
        step(g, wl.lr_at(t), t)
        ev[t][1].record()
    dist.barrier(); torch.cuda.synchronize()
    total_ms = torch.tensor([sum(a.elapsed_time(b) for a, b in ev)], device="cuda", dtype=torch.float64)
    dist.all_reduce(total_ms, op=dist.ReduceOp.MAX)
    launches = w.opt.stats()["n_launches"]
    w.close()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": wl.n * world * K / (total_ms.item() / 1e3), "unit": UNIT,
                          "n_gpus": world, "steps": K, "warmup": Wu, "ms_per_step": total_ms.item() / K,
                          "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32",
                          "data": "synthetic",
                          "config": {"workload": wl.name, "n_params": wl.n, "W": world, "chunk": wl.chunk,
                                     "parallelism": f"one worker per GPU x {world}, " + ("packed buffers stored into the peers' memory by the kernels, two barriers"
                                                                                         if args.exchange == "push" else "packed all-to-all + all-gather (NCCL)")},
                          "gpu_launches": launches}))
    dist.destroy_process_group()


# ---- kernel sweep: worker compression and W-way decompress-average on flat vectors ---------
def run_sweep(args):
    """Times the two halves of Algorithm 3 alone on flat vectors, n = 2^20 .. 2^30 in powers of 4,
    W in {2,4,8,16}, chunk in {1024,4096,16384}; inputs N(0,1) with 1 % of the elements scaled by 100.
    `compress`: worker side (z, delta in; delta, bits, magnitudes out).  `average_alone`: server side
    and nothing else (bits, magnitudes, server error in; server error, result, bits out), through a
    handle that holds only Algorithm 3's state (zoa_create_allreduce), so that 2^30 x 16 fits.
    `average_sync`: zoa_onebit_average of a full handle, i.e. the server side plus the post-sync
    rows m, x, u of Algorithm 1 for all W workers (skipped where the full state does not fit).
    One JSON line per combination."""
    import torch
    from paper_2202_06009_b200 import Zoa, ZoaError, binding as B

    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    peak, peak_kind = measured_hbm_peak()
    exps = [20, 22] if args.sweep == "quick" else [20, 22, 24, 26, 28, 30]
    if args.sweep_exp:
        exps = args.sweep_exp
    workers = args.sweep_workers or (2, 4, 8, 16)
    chunks = args.sweep_chunks or (1024, 4096, 16384)
    gen = torch.Generator("cuda").manual_seed(5)

    def fill(t):                                   # N(0,1), 1 % of the elements x100, in bounded slices
        tmp = torch.empty(min(t.numel(), 1 << 26), device="cuda")
        for lo in range(0, t.numel(), tmp.numel()):
            part = t[lo:lo + tmp.numel()]
            part.normal_(generator=gen)
            u = tmp[:part.numel()].uniform_(generator=gen)
            part.mul_(torch.where(u < 0.01, 100.0, 1.0))

    def timed(calls, reps):
        """calls: list of (name, fn); returns {name: [ms per rep]} with events between consecutive calls."""
        out = {name: [] for name, _ in calls}
        for _ in range(reps):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)]
            ev[0].record()
            for k, (_, fn) in enumerate(calls):
                fn()
                ev[k + 1].record()
            torch.cuda.synchronize()
            for k, (name, _) in enumerate(calls):
                out[name].append(ev[k].elapsed_time(ev[k + 1]))
        return out

    for e in exps:
        n = 1 << e
        for W in workers:
            for chunk in chunks:
                n_chunks = n // chunk
                row = {"sweep": True, "n": n, "W": W, "chunk": chunk, "peak_kind": peak_kind}
                bytes_c = n * W * (12 + 1 / 8) + 4 * n_chunks * W
                bytes_alone = n * W / 8 + 4 * n_chunks * W + n * (12 + 1 / 8) + 4 * n_chunks
                bytes_sync = n * W * (12 + 1 / 8) + 4 * n_chunks * W + n * (20 + 1 / 8) + 4 * n_chunks
                free, _ = torch.cuda.mem_get_info()
                light_bytes = (2 * W + 2) * n * 4 + (W + 1) * n // 8
                if light_bytes > 0.97 * free:
                    row["skipped"] = f"memory: inputs, errors and packed buffers need {light_bytes / 1e9:.0f} GB"
                    print(json.dumps(row), flush=True)
                    continue
                # -- the two halves alone, on a handle that holds only Algorithm 3's state --
                z = [torch.empty(n, device="cuda") for _ in range(W)]
                for t in z:
                    fill(t)
                z_bar = torch.empty(n, device="cuda")
                opt = Zoa(n, W, chunk=chunk, allreduce_only=True)
                t = timed([("compress", lambda: opt.allreduce_compress(z)), ("average_alone", lambda: opt.allreduce_average(z_bar))],
                          args.sweep_reps + 1)             # rep 0: errors start at zero; later reps: non-zero errors
                opt.check_device()
                opt.close()
                del z_bar
                tc, ta = statistics.median(t["compress"][1:]), statistics.median(t["average_alone"][1:])
                row.update({"compress_ms_zero_errors": t["compress"][0], "compress_ms": tc, "compress_GBps": bytes_c / 1e6 / tc,
                            "compress_frac_of_peak": bytes_c / 1e6 / tc / peak,
                            "average_alone_ms": ta, "average_alone_GBps": bytes_alone / 1e6 / ta,
                            "average_alone_frac_of_peak": bytes_alone / 1e6 / ta / peak,
                            "both_GBps": (bytes_c + bytes_alone) / 1e6 / (tc + ta),
                            "l2_resident": light_bytes < 126e6})
                # -- the server side with the post-sync rows of Algorithm 1, on a full handle --
                del z
                torch.cuda.empty_cache()
                free, _ = torch.cuda.mem_get_info()
                full_bytes = (4 * W + 4) * n * 4 + (W + 1) * n // 8
                if full_bytes > 0.97 * free:
                    row["average_sync_skipped"] = f"memory: a full handle needs {full_bytes / 1e9:.0f} GB"
                else:
                    try:
                        opt = Zoa(n, W, chunk=chunk)
                        for i in range(W):
                            fill(opt.device_view("u", i)[:n])
                        ts = []
                        for rep in range(args.sweep_reps + 1):
                            B.zoa_set_scalars(opt.h, 1e-3, 0, rep)
                            t = timed([("compress", opt.onebit_compress), ("average_sync", opt.onebit_average)], 1)
                            ts.append(t["average_sync"][0])
                        opt.check_device()
                        opt.close()
                        tsync = statistics.median(ts[1:])
                        row.update({"average_sync_ms": tsync, "average_sync_GBps": bytes_sync / 1e6 / tsync,
                                    "average_sync_frac_of_peak": bytes_sync / 1e6 / tsync / peak})
                    except ZoaError as err:
                        row["average_sync_skipped"] = f"memory: {err}"
                print(json.dumps(row), flush=True)
                torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="bert_large",
                    help="tiny | bert_base | bert_large (default, the headline) | gpt2_1p5b | all (one line each)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-sample", type=int, default=1 << 25,
                    help="upper bound on the parameters in the oracle's timed sample (4 Mi per core at most)")
    ap.add_argument("--cpu-steps", type=int, default=8, help="how many of the window's first steps the oracle is timed on")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--scale", type=int, default=1, help="shrink every tensor by this factor (profiling captures)")
    ap.add_argument("--no-pipeline", action="store_true", help="fused sync step through the chunk-per-block kernel")
    ap.add_argument("--mapping", default="simulated", choices=["simulated", "worker-per-gpu"],
                    help="simulated: W workers as state buffers on each GPU (the headline); worker-per-gpu: "
                         "the paper's own mapping, one worker per rank with the packed buffers exchanged")
    ap.add_argument("--exchange", default="nccl", choices=["nccl", "push"],
                    help="worker-per-gpu mapping: exchange the packed buffers with NCCL collectives, or let the "
                         "kernels store them into the peers' buffers (symmetric memory) between two barriers")
    ap.add_argument("--two-call", action="store_true",
                    help="sync steps as zoa_step + zoa_onebit_reduce (three kernels) instead of the fused call")
    ap.add_argument("--grad-dtype", default="f32", choices=["f32", "f16", "bf16"],
                    help="element type of the gradient buffers (state and arithmetic stay f32)")
    ap.add_argument("--chunk", type=int, default=0,
                    help="override the workload's chunk (e.g. 1073741824 = one magnitude for the whole vector, Eq. 3 as printed)")
    ap.add_argument("--algorithm", default="alg1", choices=["alg1", "alg2"],
                    help="alg1: 0/1 Adam (the headline); alg2: the paper's frozen-variance 1-bit framework")
    ap.add_argument("--sweep", nargs="?", const="full", default=None, choices=["full", "quick"],
                    help="time the compress / decompress-average kernels over the size grid instead")
    ap.add_argument("--sweep-reps", type=int, default=3)
    ap.add_argument("--sweep-exp", type=int, nargs="*", help="restrict the sweep to n = 2^EXP for these exponents")
    ap.add_argument("--sweep-workers", type=int, nargs="*", help="restrict the sweep to these worker counts")
    ap.add_argument("--sweep-chunks", type=int, nargs="*", help="restrict the sweep to these chunk sizes")
    args = ap.parse_args()

    if args.sweep:
        return run_sweep(args)
    if args.impl == "reference":
        # the oracle needs no CUDA library; import only the workload tables
        import importlib.util
        spec = importlib.util.spec_from_file_location("_synth", os.path.join(ROOT, "paper_2202_06009_b200", "synth.py"))
        synth = importlib.util.module_from_spec(spec)
        sys.modules["_synth"] = synth
        spec.loader.exec_module(synth)
        wl = synth.WORKLOADS[args.workload]()
        if args.scale > 1:
            wl = synth.scaled(wl, args.scale)
        if args.chunk:
            wl.chunk = args.chunk
        if args.steps is None:
            args.steps = wl.steps
        return run_reference(args, wl, synth)

    from paper_2202_06009_b200 import synth
    if args.workload == "all":      # one JSON line per shaped workload, BERT-Large (the headline) last
        import copy
        for name in ("bert_base", "gpt2_1p5b", "bert_large"):
            sub = copy.copy(args)
            sub.workload, sub.steps = name, None
            sub.no_cpu_baseline = args.no_cpu_baseline or name != "bert_large"
            wl = synth.WORKLOADS[name]()
            sub.steps = wl.steps
            run_ours(sub, wl)
            import torch
            torch.cuda.empty_cache()
        return
    wl = synth.WORKLOADS[args.workload]()
    if args.scale > 1:
        wl = synth.scaled(wl, args.scale)
    if args.chunk:
        wl.chunk = args.chunk
    if args.steps is None:
        args.steps = wl.steps
    if args.mapping == "worker-per-gpu":
        return run_worker_per_gpu(args, wl)
    run_ours(args, wl)


if __name__ == "__main__":
    main()
