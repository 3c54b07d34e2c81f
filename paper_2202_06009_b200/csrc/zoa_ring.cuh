// Building blocks of the persistent bulk-copy-ring kernels (zoa_pipeline.cu, zoa_reduce_pipeline.cu):
// mbarrier and bulk-copy wrappers with bounded waits, the consumers' named barrier and block-wide
// sums, and the copy-issuing lane's bookkeeping.  Everything here has internal linkage.
#pragma once

#include "zoa_internal.h"

namespace zoa {
namespace {

constexpr int kConsumers = 512;                 // consumer threads (16 warps)
constexpr int kConsumerWarps = kConsumers / 32;
constexpr int kThreads = kConsumers + 32;       // + one producer warp
constexpr int kTile = 4 * kConsumers;           // coordinates per ring stage and array
constexpr int kTileBytes = kTile * 4;
constexpr int kStageBytes = 4 * kTileBytes;     // g, m, u, delta  |  delta_bar, v, x_sync, (unused)
constexpr int kSyncStages = 6;                  // ring depth of the fused sync kernel (32 KB stages)
constexpr int kMaxStages = 12;                  // of the Algorithm 2 kernel (16 KB stages)

struct PipeArgs {
    StateView st;
    GradPtrs g;
    Consts c;
    float gamma, gamma_sum;
    long long first_chunk;    // the launch covers the full chunks [first_chunk, first_chunk + n_full_chunks)
    long long n_full_chunks;
    int stages;
    ErrorWords error_flag;  // set non-zero when a wait ran out
    unsigned long long *sched;  // device: [0] next chunk to hand out, [1] blocks that have finished
    int grad_fmt;                      // kGradF32 / kGradF16 / kGradBF16 (| kGradAligned, always set here)
    unsigned long long wait_limit_ns;  // how long a thread waits on an mbarrier before it gives up
    long long test_stop_after_tiles;   // > 0: each producer stops after this many tiles (error-path test)
};

// Shared-memory header (the ring follows, 1024-byte aligned).
struct PipeShared {
    unsigned long long full[kMaxStages];
    unsigned long long empty[kMaxStages];
    double sums[2][kConsumerWarps];
    long long chunk_queue[kMaxStages + 2];   // chunk ids in the order the producer took them; -1 = no more
    int abort;
    uint32_t sink[32];                       // one word per warp, see release_stage
};

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false if the block has been aborted or the limit ran out
// (in which case it raises both flags).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, const ErrorWords &error_flag,
                                          unsigned long long limit_ns)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long start = global_timer_ns();
    for (unsigned it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((it & 63u) == 0 && global_timer_ns() - start > limit_ns) {
            *abort_flag = 1;
            atomicExch(error_flag.device, 1);
            if (error_flag.host_mapped) {      // the host sees this one without synchronising
                *reinterpret_cast<volatile int *>(error_flag.host_mapped) = 1;
                __threadfence_system();
            }
            return false;
        }
    }
}
// 1-D bulk asynchronous copy global -> this block's shared memory, completion counted on `bar`.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }
// Barrier over the consumers that also tells every one of them whether any had `flag` set.
__device__ __forceinline__ bool consumer_any(bool flag)
{
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"((uint32_t)flag), "n"(kConsumers)
        : "memory");
    return out != 0;
}

// Hands a ring stage back to the producer once this warp has read it.  `dep` must be computed from what
// the warp loaded from the stage.  A shared-memory load only *issues* in program order: behind a full
// store queue its data can return after a later mbarrier arrive has already let the producer refill
// the stage, and the warp then reads the next tile's bytes (seen on an L2-resident problem, where the
// refill lands within a few hundred nanoseconds).  The store of `dep` cannot issue before every
// lane's loads have returned, and the arrive follows that store.
__device__ __forceinline__ void release_stage(PipeShared *sh, int stage, uint32_t dep)
{
    *reinterpret_cast<volatile uint32_t *>(&sh->sink[(threadIdx.x >> 5) & 31]) = dep;
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(smem_addr(&sh->empty[stage]));
}
__device__ __forceinline__ uint32_t dep_bits(float4 a) { return __float_as_uint(a.x); }
__device__ __forceinline__ uint32_t dep_bits(float4 a, float4 b) { return __float_as_uint(a.x) ^ __float_as_uint(b.x); }
__device__ __forceinline__ uint32_t dep_bits(float4 a, float4 b, float4 c, float4 d)
{
    return __float_as_uint(a.x) ^ __float_as_uint(b.x) ^ __float_as_uint(c.x) ^ __float_as_uint(d.x);
}

// Sum over the 512 consumers in binary64; every consumer gets the same value.
// One named barrier per call (the two partial-sum arrays alternate).
__device__ __forceinline__ double consumer_sum(double v, PipeShared *sh, int &flip)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) sh->sums[flip][threadIdx.x >> 5] = v;
    consumer_barrier();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kConsumerWarps; ++w) t += sh->sums[flip][w];
    flip ^= 1;
    return t;
}

// Sum over the consumer warps that share a chunk (WPC consecutive warps), in warp order, in
// binary64; every thread gets its own chunk's total.  One named barrier per call.
template <int WPC>
__device__ __forceinline__ double consumer_group_sum(double v, PipeShared *sh, int &flip)
{
    if constexpr (WPC == kConsumerWarps) {
        return consumer_sum(v, sh, flip);
    } else {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) sh->sums[flip][warp] = v;
    consumer_barrier();
    const int first = warp / WPC * WPC;
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < WPC; ++w) t += sh->sums[flip][first + w];
    flip ^= 1;
    return t;
    }
}

// Packs the sign bits of a float4-per-lane tile: lane l holds coordinates 4l..4l+3,
// eight lanes make one word.  Returns the word in every lane of the 8-lane group.
__device__ __forceinline__ uint32_t pack_group(const bool b[4])
{
    const int lane = threadIdx.x & 31;
    const uint32_t nib = (b[0] ? 1u : 0u) | (b[1] ? 2u : 0u) | (b[2] ? 4u : 0u) | (b[3] ? 8u : 0u);
    return __reduce_or_sync(0xFFu << (lane & 24), nib << ((lane & 7) * 4));
}

// Set-up shared by the ring kernels: stage barriers and the abort flag, then a block barrier.
__device__ __forceinline__ void ring_init(PipeShared *sh, int stages)
{
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_addr(&sh->full[s]), 1);
            mbar_init(smem_addr(&sh->empty[s]), kConsumerWarps);
        }
        sh->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
}

// The copy-issuing lane's side of the ring: which stage comes next, chunk ids from the global
// counter, and the orderly way out when a wait runs out.
struct RingProducer {
    const PipeArgs &a;
    PipeShared *sh;
    unsigned char *ring;
    int stage_bytes;
    int s = 0;
    uint32_t phase = 0;
    long long issued = 0;
    bool ok = true;

    __device__ RingProducer(const PipeArgs &args, PipeShared *shared, unsigned char *ring_base, int bytes)
        : a(args), sh(shared), ring(ring_base), stage_bytes(bytes) {}

    // Waits until the consumers have released the current stage.
    __device__ __forceinline__ bool stage_free()
    {
        if (!ok) return false;
        if (!mbar_wait(smem_addr(&sh->empty[s]), phase ^ 1u, &sh->abort, a.error_flag, a.wait_limit_ns)) ok = false;
        return ok;
    }
    // Takes the k-th chunk of this block from the global counter and tells the consumers: the id
    // travels through shared memory and the arrive on the chunk's first tile publishes it.  The queue
    // cannot wrap onto an unread entry: the producer is at most `stages` tiles, hence chunks, ahead.
    // Returns false when no chunk is left (the consumers are told) or a wait ran out.
    __device__ __forceinline__ bool next_chunk(long long k, long long *chunk) { return publish(k, take(), chunk); }
    // The two halves of next_chunk, for a producer that takes its chunks ahead of time: the number of a
    // chunk from the global counter, and (later) the announcement of it as this block's k-th chunk.
    __device__ __forceinline__ long long take() { return (long long)atomicAdd(&a.sched[0], 1ull); }
    __device__ __forceinline__ bool publish(long long k, long long taken, long long *chunk)
    {
        const bool last = taken >= a.n_full_chunks;
        *chunk = a.first_chunk + taken;
        if (!stage_free()) return false;
        sh->chunk_queue[k % (kMaxStages + 2)] = last ? -1 : *chunk;
        if (last) mbar_arrive(smem_addr(&sh->full[s]));   // an empty "tile": wakes the consumers to read the -1
        return !last;
    }
    __device__ __forceinline__ uint32_t stage_addr() const { return smem_addr(ring + (size_t)s * stage_bytes); }
    __device__ __forceinline__ uint32_t full_barrier() const { return smem_addr(&sh->full[s]); }
    // The current stage's copies have been issued.
    __device__ __forceinline__ void advance()
    {
        ++issued;
        if (++s == a.stages) { s = 0; phase ^= 1u; }
        if (a.test_stop_after_tiles > 0 && issued >= a.test_stop_after_tiles) ok = false;
    }
    // After the last chunk, or after giving up: let copies still in flight land before the block's
    // shared memory is released, and let the last block to finish rearm the counters.
    __device__ __forceinline__ void finish()
    {
        if (!ok) {
            const long long R = a.stages, outstanding = issued < R ? issued : R;
            for (long long k = 1; k <= outstanding; ++k) {
                const long long q = issued - k;                      // sequence number of an issued tile
                const uint32_t bar = smem_addr(&sh->full[q % R]);
                const uint32_t par = (uint32_t)((q / R) & 1);
                const unsigned long long start = global_timer_ns();
                while (!mbar_try_wait(bar, par) && global_timer_ns() - start < a.wait_limit_ns) {}
            }
        }
        if (atomicAdd(&a.sched[1], 1ull) == gridDim.x - 1) {
            a.sched[0] = 0;
            a.sched[1] = 0;
        }
    }
};

}  // namespace
}  // namespace zoa
