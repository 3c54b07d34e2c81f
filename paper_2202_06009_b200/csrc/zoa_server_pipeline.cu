// server_prefetch_kernel: the server side of Algorithm 3 by itself (zoa_allreduce_average, the second
// half of zoa_onebit_allreduce, the server step of the one-worker-per-GPU mapping) for whole chunks.
//
// The step moves 12 to 14 bytes per coordinate (W bit streams and the server error in; the server
// error, the result and one bit stream out), so what it costs is instructions and latency, not
// bandwidth.  Instructions: the sum over the workers is looked up in tables (zoa_device.cuh), and a
// thread takes 32 or more coordinates, so that what a block does once (tables, sums) is spread thin.
// Latency: one block per chunk; its first thread starts bulk copies of the chunk's server errors and
// of its W packed word rows into shared memory before anything else, so they arrive while the
// magnitudes are fetched and the tables built; no register holds prefetched data, and many small
// blocks are resident per SM (a persistent ring of 16 consumer warps per SM was tried and ran out
// of issue slots: 1.16 ms where this kernel takes 0.51, n = 2^28, W = 4).  The server input a
// replaces the server error in shared memory between the two passes, so the registers do not grow
// with the chunk.  The wait for the copies is bounded.
#include "zoa_internal.h"
#include "zoa_ring.cuh"

namespace zoa {
namespace {

struct PrefetchLayout {
    int tables_off, scales_off, ds_off, words_off, total;   // bytes from the start of dynamic shared memory
};
__host__ __device__ inline PrefetchLayout prefetch_layout(int W, int chunk)
{
    PrefetchLayout l;
    l.tables_off = 512;                                   // after the barrier, two flags and 34 doubles of scratch
    l.scales_off = l.tables_off + ((W + 3) / 4) * 128;
    l.ds_off = (l.scales_off + W * 4 + 127) & ~127;
    l.words_off = l.ds_off + chunk * 4;
    l.total = l.words_off + W * (chunk / 8);
    return l;
}

}  // namespace

// Chunk first_chunk + blockIdx.x, which has its full length.  words_in[w][range words] and
// scales_in[w][range chunks] start at the range's first chunk; 16-byte aligned rows; chunk % 128 == 0;
// z_bar NULL or 16-byte aligned.  skip_copies: test hook, the copies are never started.
__global__ void __launch_bounds__(512, 2) server_prefetch_kernel(const __grid_constant__ StateView st, const uint32_t *words_in, long long words_in_stride,
                                       const float *scales_in, long long scales_in_stride, int W_total, long long first_chunk,
                                       const __grid_constant__ PeerOut out, float *z_bar, ErrorWords error_flag,
                                       unsigned long long wait_limit_ns, int skip_copies)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned long long *bar = reinterpret_cast<unsigned long long *>(smem_raw);
    int *abort_flag = reinterpret_cast<int *>(smem_raw + 8);
    int *exact_flag = reinterpret_cast<int *>(smem_raw + 12);
    double *scratch = reinterpret_cast<double *>(smem_raw + 16);
    const PrefetchLayout lay = prefetch_layout(W_total, st.chunk);
    double *table = reinterpret_cast<double *>(smem_raw + lay.tables_off);       // [groups][16]
    float *scales = reinterpret_cast<float *>(smem_raw + lay.scales_off);        // [W_total]
    float *ds_s = reinterpret_cast<float *>(smem_raw + lay.ds_off);              // [chunk]
    const uint32_t *words_s = reinterpret_cast<const uint32_t *>(smem_raw + lay.words_off);   // [W_total][chunk / 32]
    const long long chunk_id = first_chunk + blockIdx.x;
    const long long c0 = chunk_id * st.chunk;
    const int lane = threadIdx.x & 31;
    const int groups = (W_total + 3) >> 2;
    const int wpc = st.chunk >> 5;                   // words per chunk and worker

    if (threadIdx.x == 0) {
        const uint32_t b = smem_addr(bar);
        mbar_init(b, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive_expect_tx(b, (uint32_t)(st.chunk * 4 + W_total * (st.chunk / 8)));
        if (!skip_copies) {
            bulk_load(smem_addr(ds_s), st.ds + c0, st.chunk * 4, b);
            const uint32_t *row = words_in + (long long)blockIdx.x * wpc;
            for (int i = 0; i < W_total; ++i) bulk_load(smem_addr(words_s + i * wpc), row + (long long)i * words_in_stride, st.chunk / 8, b);
        }
    }
    if (threadIdx.x < 32) {
        __syncwarp();
        const float s_lo = lane < W_total ? scales_in[(long long)lane * scales_in_stride + blockIdx.x] : 0.0f;
        const float s_hi = lane + 32 < W_total ? scales_in[(long long)(lane + 32) * scales_in_stride + blockIdx.x] : 0.0f;
        if (lane < W_total) scales[lane] = s_lo;
        if (lane + 32 < W_total) scales[lane + 32] = s_hi;
        const bool exact = table_sum_is_exact(s_lo, s_hi, W_total);
        if (lane == 0) *exact_flag = exact;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < 16 * groups; e += blockDim.x) table[e] = table_entry(scales, W_total, e);
    const bool arrived = mbar_wait(smem_addr(bar), 0, abort_flag, error_flag, wait_limit_ns);
    if (__syncthreads_or(!arrived)) return;          // unanimous; also publishes the tables
    const bool fast = *exact_flag != 0;

    const uint32_t sel = (threadIdx.x & 3u) | ((4u + (threadIdx.x & 3u)) << 4);   // byte (idx / 8) % 4 of two words
    const bool w_pow2 = (W_total & (W_total - 1)) == 0;
    const double inv_w = __longlong_as_double((long long)(1023 - (31 - __clz(W_total))) << 52);
    const int last = W_total - 1;
    double l1 = 0.0;
    for (int idx = 8 * threadIdx.x; idx < st.chunk; idx += 8 * blockDim.x) {
        const float4 e0 = ld4(ds_s + idx), e1 = ld4(ds_s + idx + 4);
        double A[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
        const uint32_t *col = words_s + (idx >> 5);
        for (int g = 0; g < groups; ++g) {
            // a worker index past the last one repeats the last worker's word: its bits select among equal table entries
            const int i1 = min(4 * g + 1, last), i2 = min(4 * g + 2, last), i3 = min(4 * g + 3, last);
            const uint32_t x = gather_bytes(col[4 * g * wpc], col[i1 * wpc], col[i2 * wpc], col[i3 * wpc], sel);
            if (fast) {
                const char *tb = reinterpret_cast<const char *>(table + g * 16);
#pragma unroll
                for (int c = 0; c < 8; ++c) A[c] = __dadd_rn(A[c], *reinterpret_cast<const double *>(tb + table_offset(x, c)));
            } else {
                for (int q = 0; q < 4 && 4 * g + q < W_total; ++q) {   // worker order
                    const double sc = (double)scales[4 * g + q];
                    const uint32_t byte = x >> (8 * q);
#pragma unroll
                    for (int c = 0; c < 8; ++c) A[c] = __dadd_rn(A[c], ((byte >> c) & 1u) ? sc : -sc);
                }
            }
        }
        float a[8] = {e0.x, e0.y, e0.z, e0.w, e1.x, e1.y, e1.z, e1.w};
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const double q = w_pow2 ? __dmul_rn(A[c], inv_w) : __ddiv_rn(A[c], (double)W_total);
            a[c] = __double2float_rn(__dadd_rn(q, (double)a[c]));          // = server_input(A[c], W_total, the server error)
            l1 += fabs((double)a[c]);
        }
        st4(ds_s + idx, make_float4(a[0], a[1], a[2], a[3]));             // the thread's own slots
        st4(ds_s + idx + 4, make_float4(a[4], a[5], a[6], a[7]));
    }
    const float scale = chunk_scale(block_sum(l1, scratch), st.chunk);
    for (int idx = 8 * threadIdx.x; idx < st.chunk; idx += 8 * blockDim.x) {
        const float4 a0 = ld4(ds_s + idx), a1 = ld4(ds_s + idx + 4);
        float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
        float hat[8];
        uint32_t bits = 0;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const bool b = a[c] >= 0.0f;               // +0 and -0 count as non-negative, NaN as negative
            hat[c] = b ? scale : -scale;
            a[c] = f_sub(a[c], hat[c]);
            bits |= (b ? 1u : 0u) << c;
        }
        // four neighbouring lanes hold the four bytes of a word
        bits <<= 8 * (lane & 3);
        bits |= __shfl_xor_sync(0xffffffffu, bits, 1);
        bits |= __shfl_xor_sync(0xffffffffu, bits, 2);
        if ((lane & 3) == 0) {
            const long long w = (c0 + idx) >> 5;
            st.words_s[w] = bits;
            for (int r = 0; r < out.world; ++r) out.words_s[r][w] = bits;
        }
        st4(st.ds + c0 + idx, make_float4(a[0], a[1], a[2], a[3]));
        st4(st.ds + c0 + idx + 4, make_float4(a[4], a[5], a[6], a[7]));
        if (z_bar) {
            st4_stream(z_bar + c0 + idx, make_float4(hat[0], hat[1], hat[2], hat[3]));
            st4_stream(z_bar + c0 + idx + 4, make_float4(hat[4], hat[5], hat[6], hat[7]));
        }
    }
    if (threadIdx.x == 0) {
        st.scales_s[chunk_id] = scale;
        for (int r = 0; r < out.world; ++r) out.scales_s[r][chunk_id] = scale;
    }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
// Whether server_prefetch_kernel takes these buffers: bulk copies want 16-byte aligned rows of a
// multiple of 16 bytes, the eight-coordinate layout a chunk of whole 256-coordinate passes of a
// warp, and at least two blocks should fit an SM.
bool server_prefetch_applies(const StateView &st, const uint32_t *words_in, long long words_in_stride, int W_total, const float *z_bar)
{
    if (st.chunk % 256 != 0) return false;
    if ((reinterpret_cast<uintptr_t>(words_in) & 15u) || (words_in_stride & 3) || (reinterpret_cast<uintptr_t>(z_bar) & 15u)) return false;
    return prefetch_layout(W_total, st.chunk).total <= 110 * 1024;
}

// Server side of Algorithm 3 alone for the whole chunks [first_chunk, first_chunk + count).
cudaError_t launch_server_prefetch(const StateView &st, const uint32_t *words_in, long long words_in_stride,
                                   const float *scales_in, long long scales_in_stride, int W_total, long long first_chunk,
                                   long long count, const PeerOut &out, float *z_bar, ErrorWords error_flag,
                                   unsigned long long wait_limit_ns, bool skip_copies, cudaStream_t s)
{
    static SmemLimitOnce once;
    const cudaError_t e = once.ensure(server_prefetch_kernel, 110 * 1024);
    if (e != cudaSuccess) return e;
    // 32 coordinates per thread up to chunk 8192 (64 at 16384): measured best at n = 2^28 for W = 4 and 16
    int thr = st.chunk / 32;
    thr = thr < 32 ? 32 : thr > 256 ? 256 : thr;
    const PrefetchLayout lay = prefetch_layout(W_total, st.chunk);
    server_prefetch_kernel<<<(unsigned)count, thr, lay.total, s>>>(st, words_in, words_in_stride, scales_in, scales_in_stride, W_total,
                                                                 first_chunk, out, z_bar, error_flag, wait_limit_ns, skip_copies ? 1 : 0);
    return cudaGetLastError();
}

}  // namespace zoa
