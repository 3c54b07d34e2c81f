// Device-side building blocks shared by the zoa kernels: the binary32
// "one rounding per operation" arithmetic, 128-bit accesses, the block-wide
// binary64 sum and the sign-bit packing.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace zoa {

constexpr int kMaxWorkers = 64;
constexpr int kMaxChunk = 16384;
constexpr int kRowAlign = 128;  // elements; state rows are padded to this

// W gradient pointers travel as one kernel argument.
struct GradPtrs {
    const float *p[kMaxWorkers];
};

// beta1, 1 - beta1, beta2, 1 - beta2, eps, all already rounded to binary32 on the host.
struct Consts {
    float b1, ob1, b2, ob2, eps;
};

// Borrowed view of a handle's device state (see include/zoa.h for the layout).
struct StateView {
    float *x, *m, *u, *dw;  // [W][n_pad]
    const float *v;         // [n_pad] v_t
    float *v_next;          // [n_pad] v_{t+1}, written on T_v steps
    float *ds, *xs;         // [n_pad] server error, model at the last sync
    uint32_t *words_w;      // [W][words_stride]
    float *scales_w;        // [W][n_chunks]
    uint32_t *words_s;      // [words_stride]
    float *scales_s;        // [n_chunks]
    long long n, n_pad, n_chunks, words_stride;
    int W, chunk;
};

// One worker per GPU: where a rank's packed buffers go.  Rank s serves the chunks
// [chunk_begin[s], chunk_begin[s + 1]); words[s] / scales[s] point at the first word /
// magnitude of that range inside a buffer that rank s can read (its own memory: the
// pointer is a peer pointer for every other rank, and the stores cross NVLink).
struct PushPlan {
    int world;
    long long chunk_begin[kMaxWorkers + 1];
    uint32_t *words[kMaxWorkers];
    float *scales[kMaxWorkers];
};
// Where a server's packed result goes: the whole-vector words_s / scales_s of every rank.
struct PeerOut {
    int world;
    uint32_t *words_s[kMaxWorkers];
    float *scales_s[kMaxWorkers];
};

// ---- binary32 arithmetic, one IEEE rounding per operation, never contracted ----
__device__ __forceinline__ float f_add(float a, float b) { return __fadd_rn(a, b); }
__device__ __forceinline__ float f_sub(float a, float b) { return __fsub_rn(a, b); }
__device__ __forceinline__ float f_mul(float a, float b) { return __fmul_rn(a, b); }
__device__ __forceinline__ float f_div(float a, float b) { return __fdiv_rn(a, b); }
__device__ __forceinline__ float f_sqrt(float a) { return __fsqrt_rn(a); }

// Momentum update of Algorithm 1: m_{t+1/2} = beta1 m_t + (1 - beta1) g_t.
__device__ __forceinline__ float momentum(const Consts &c, float m, float g)
{
    return f_add(f_mul(c.b1, m), f_mul(c.ob1, g));
}
// Denominator of both model updates of Algorithm 1: sqrt(v_t + eps).
__device__ __forceinline__ float denom(const Consts &c, float v) { return f_sqrt(f_add(v, c.eps)); }
// Variance update of Algorithm 1: v_{t+1} = beta2 v_t + (1 - beta2) g_bar^2.
__device__ __forceinline__ float variance(const Consts &c, float v, float g_bar)
{
    return f_add(f_mul(c.b2, v), f_mul(c.ob2, f_mul(g_bar, g_bar)));
}
// x / count in binary64, as the IEEE division gives it.  A binary64 division is a long instruction
// sequence and the server side runs one per coordinate; when the count is a power of two (every worker
// count and chunk size of the benchmark configurations) the quotient is x scaled by 2^-k, which is
// exact, so one multiplication gives the same bits (x is zero or a sum of binary32 magnitudes: the
// scaled value cannot fall into the subnormal range of binary64).
__device__ __forceinline__ double div_by_count(double x, int count)
{
    if ((count & (count - 1)) == 0)
        return __dmul_rn(x, __longlong_as_double((long long)(1023 - (31 - __clz(count))) << 52));
    return __ddiv_rn(x, (double)count);
}
// Mean over W workers of a binary64 sum, rounded once (Algorithm 4).
__device__ __forceinline__ float mean_round(double sum, int W)
{
    return __double2float_rn(div_by_count(sum, W));
}
// Eq. 3 magnitude of a chunk: l1 / len, rounded once.
__device__ __forceinline__ float chunk_scale(double l1, int len)
{
    return __double2float_rn(div_by_count(l1, len));
}
// Server input of Algorithm 3: mean of the compressed buffers plus the server error.
__device__ __forceinline__ float server_input(double sum_hat, int W, float delta_bar)
{
    return __double2float_rn(__dadd_rn(div_by_count(sum_hat, W), (double)delta_bar));
}

// ---- the server's sum over the workers (Algorithm 3), looked up instead of added bit by bit ----
// The workers are taken in groups of four; a group's sixteen possible signed sums of magnitudes sit
// in a table of 128 bytes (one entry per pair of shared-memory banks, so a warp's lookups never
// conflict).  A thread owns eight consecutive coordinates = one byte of every worker's words;
// gather_bytes puts that byte of four workers into one register, and for coordinate c one mask, one
// multiplication and one shift turn the four workers' bits into the byte offset of the table entry.
// Adding the groups' entries gives the bits of the worker-by-worker binary64 sum whenever every
// partial sum is exact: all magnitudes are multiples of the smallest one's last place, so it is
// enough that W * 2^(e_max + 1) stays below 2^53 of those units, i.e. that the exponents of the
// non-zero magnitudes differ by at most 29 - ceil(log2 W).  With up to four workers the single
// table holds the sequential sum itself.  Otherwise the caller adds worker by worker.
constexpr uint32_t kGatherMul = 0x10204080u;   // 2^28 + 2^21 + 2^14 + 2^7: bits 0, 8, 16, 24 -> bits 28 ... 31

// Warp-wide.  Lane l passes the magnitudes of workers l and l + 32 (0 beyond W).
__device__ __forceinline__ bool table_sum_is_exact(float s_lo, float s_hi, int W)
{
    if (W <= 4) return true;
    int e_max = 0, e_min = 255;
    bool bad = false;
    const float both[2] = {s_lo, s_hi};
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const uint32_t u = __float_as_uint(both[q]);
        int e = (int)((u >> 23) & 0xFFu);
        if (e == 255 || (u >> 31)) bad = true;            // not finite
        else if (u << 1) {                                // not zero
            e = e < 1 ? 1 : e;                            // subnormals share the exponent of the smallest normals
            e_max = e > e_max ? e : e_max;
            e_min = e < e_min ? e : e_min;
        }
    }
    e_max = __reduce_max_sync(0xffffffffu, e_max);
    e_min = __reduce_min_sync(0xffffffffu, e_min);
    bad = __any_sync(0xffffffffu, bad);
    return !bad && e_max - e_min <= 29 - (32 - __clz(W - 1));
}
// Entry e = 16 * group + m of the tables: the signed sum of the group's workers in worker order, worker
// 4 * group + k taken positive where bit k of m is set.
__device__ __forceinline__ double table_entry(const float *scales, int W, int e)
{
    const int g = e >> 4, m = e & 15;
    double acc = 0.0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int i = 4 * g + k;
        if (i < W) acc = __dadd_rn(acc, ((m >> k) & 1) ? (double)scales[i] : -(double)scales[i]);
    }
    return acc;
}
// Byte b of each of four words, worker k's in byte k; sel = b | ((4 + b) << 4).
__device__ __forceinline__ uint32_t gather_bytes(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, uint32_t sel)
{
    return __byte_perm(__byte_perm(w0, w1, sel), __byte_perm(w2, w3, sel), 0x5410u);
}
// Byte offset (8 * the four workers' bits) of coordinate c's entry; x from gather_bytes, c a constant
// after unrolling.
__device__ __forceinline__ uint32_t table_offset(uint32_t x, int c)
{
    return ((x & (0x01010101u << c)) * (kGatherMul >> c)) >> 25;
}

// ---- 128-bit accesses ----
__device__ __forceinline__ float4 ld4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ void st4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
// Streaming variants: data touched once per step should not displace the rest of L2.
__device__ __forceinline__ float4 ld4_stream(const float *p)
{
    return __ldcs(reinterpret_cast<const float4 *>(p));
}
__device__ __forceinline__ void st4_stream(float *p, float4 v) { __stcs(reinterpret_cast<float4 *>(p), v); }

// ---- bulk asynchronous stores (the copy engine reads shared memory and writes global memory) ----
// A thread that wrote the shared-memory source with ordinary stores runs store_fence() before the
// block barrier that precedes the bulk store; the issuing thread commits its stores as a group and
// waits until the engine has read the source before the block reuses or releases it.  Both
// addresses must be 16-byte aligned and the size a multiple of 16 bytes.
__device__ __forceinline__ void store_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void bulk_store(void *dst_global, const void *src_shared, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst_global), "r"((uint32_t)__cvta_generic_to_shared(src_shared)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Returns once the source of every committed group but the newest `N` has been read.
template <int N>
__device__ __forceinline__ void bulk_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }

// How the W gradient buffers are to be read: bit 0 = every pointer is aligned for the
// vector path (16 bytes for binary32, 8 for the 16-bit types), bits 1-2 = element type.
// Gradients in binary16 / bfloat16 are converted to binary32 exactly on load; all
// arithmetic and all state stay binary32.
constexpr int kGradAligned = 1;
constexpr int kGradF32 = 0, kGradF16 = 1 << 1, kGradBF16 = 2 << 1, kGradTypeMask = 3 << 1;

__device__ __forceinline__ float grad16_to_float(unsigned short bits, int fmt)
{
    return (fmt & kGradTypeMask) == kGradBF16 ? __uint_as_float((unsigned)bits << 16)
                                              : __half2float(__ushort_as_half(bits));
}
__device__ __forceinline__ float4 grad16x4_to_float4(uint2 raw, int fmt)
{
    return make_float4(grad16_to_float((unsigned short)(raw.x & 0xFFFFu), fmt), grad16_to_float((unsigned short)(raw.x >> 16), fmt),
                       grad16_to_float((unsigned short)(raw.y & 0xFFFFu), fmt), grad16_to_float((unsigned short)(raw.y >> 16), fmt));
}

// Four consecutive gradient values starting at j (j % 4 == 0); the user's buffer
// has exactly n elements and may be unaligned, so the ragged end and the
// unaligned case go through guarded scalar loads (zero beyond n).  `fmt` as above
// (0 and 1 are plain binary32, unaligned and aligned).
__device__ __forceinline__ float4 ld_grad4(const float *g, long long j, long long n, int fmt)
{
    const bool aligned = fmt & kGradAligned;
    if ((fmt & kGradTypeMask) == kGradF32) {
        if (aligned && j + 4 <= n) return ld4_stream(g + j);
        float4 r;
        r.x = j + 0 < n ? g[j + 0] : 0.f;
        r.y = j + 1 < n ? g[j + 1] : 0.f;
        r.z = j + 2 < n ? g[j + 2] : 0.f;
        r.w = j + 3 < n ? g[j + 3] : 0.f;
        return r;
    }
    const unsigned short *h = reinterpret_cast<const unsigned short *>(g);
    if (aligned && j + 4 <= n) return grad16x4_to_float4(__ldcs(reinterpret_cast<const uint2 *>(h + j)), fmt);
    float4 r;
    r.x = j + 0 < n ? grad16_to_float(h[j + 0], fmt) : 0.f;
    r.y = j + 1 < n ? grad16_to_float(h[j + 1], fmt) : 0.f;
    r.z = j + 2 < n ? grad16_to_float(h[j + 2], fmt) : 0.f;
    r.w = j + 3 < n ? grad16_to_float(h[j + 3], fmt) : 0.f;
    return r;
}

// ---- block-wide binary64 sum; every thread gets the result ----
// `scratch` holds 33 doubles.  Fixed tree, so a launch is reproducible.
__device__ __forceinline__ double block_sum(double v, double *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();  // scratch may still be read from the previous sum
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    if (warp == 0) {
        double t = lane < n_warps ? scratch[lane] : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (lane == 0) scratch[32] = t;
    }
    __syncthreads();
    return scratch[32];
}

// ---- sign-bit packing for the "lane l holds coordinates 4l..4l+3" layout ----
// Spreads the 8 bits of `byte` to bit positions 0, 4, 8, ..., 28.
__device__ __forceinline__ uint32_t spread8(uint32_t x)
{
    x = (x | (x << 12)) & 0x000F000Fu;
    x = (x | (x << 6)) & 0x03030303u;
    x = (x | (x << 3)) & 0x11111111u;
    return x;
}
// A warp covers 128 consecutive coordinates = 4 words.  b[k] says whether the
// lane's k-th coordinate is non-negative (and valid).  Returns, in lanes 0..3,
// word `lane` of the tile (undefined in the other lanes).  All 32 lanes call it.
__device__ __forceinline__ uint32_t pack_tile(const bool b[4])
{
    const int w = threadIdx.x & 3;
    uint32_t word = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t ballot = __ballot_sync(0xffffffffu, b[k]);
        word |= spread8((ballot >> (8 * w)) & 0xFFu) << k;
    }
    return word;
}

}  // namespace zoa
