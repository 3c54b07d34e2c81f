// The zoa kernels other than the bulk-copy ring kernel (zoa_pipeline.cu).
//
// Elementwise, one float4 per thread:
//   local_step_kernel        Algorithm 1: momentum, model and buffer updates (+ variance update on T_v steps)
//   variance_kernel          Algorithm 1: the variance update alone
//   alg2_full_kernel         Algorithm 2 on a T_v step (full-precision exchange)
// One block per chunk (any chunk that is a multiple of 32 up to 16384, ragged last
// chunk, unaligned or 16-bit gradient buffers):
//   compress_kernel          Algorithm 3 worker side (Eq. 3 per chunk, error feedback)
//   reduce_kernel            Algorithm 3 server side + Algorithm 1: momentum approximation, model sync, buffer reset
//   step_sync_kernel         a whole sync step of Algorithm 1 in one pass over memory
//   alg2_compressed_kernel   Algorithm 2 on any other step (gradients through Algorithm 3)
// Chunks larger than a block can hold, up to the whole vector (Eq. 3 as printed):
//   lc_* kernels             per-segment partial l1 sums, fixed-order chunk sums, apply passes
#include <cooperative_groups.h>

#include "zoa_internal.h"

namespace cg = cooperative_groups;

namespace zoa {

// ---------------------------------------------------------------------------
// Local step: elementwise, one thread per 4 coordinates, loop over workers so
// that v is read once and the gradient mean for the variance comes for free.
// ---------------------------------------------------------------------------
// GFMT: the gradient format when it is known at compile time (the aligned cases, which are
// the fast path), or -1 to read it from the argument.
// With 16-bit gradients a thread has fewer bytes in flight, and a fifth resident block per SM
// pays (measured 5.9 -> 6.4 TB/s); with binary32 gradients it does not (6.7 -> 6.4 TB/s).
template <bool DO_VAR, int GFMT>
__global__ void __launch_bounds__(256, (GFMT > 0 && (GFMT & kGradTypeMask) != kGradF32) ? 5 : 4)
local_step_kernel(StateView st, GradPtrs g, Consts c, float gamma, int g_fmt_arg, long long first4, long long end4)
{
    const int g_aligned = GFMT >= 0 ? GFMT : g_fmt_arg;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long q = first4 + (long long)blockIdx.x * blockDim.x + threadIdx.x; q < end4; q += stride) {   // float4 groups [first4, end4)
        const long long j = q << 2;
        const float4 v4 = ld4(st.v + j);
        const float d[4] = {denom(c, v4.x), denom(c, v4.y), denom(c, v4.z), denom(c, v4.w)};
        double G[4] = {0.0, 0.0, 0.0, 0.0};
        for (int i = 0; i < st.W; ++i) {
            const long long row = (long long)i * st.n_pad + j;
            const float4 g4 = ld_grad4(g.p[i], j, st.n, g_aligned);
            const float4 m4 = ld4(st.m + row), x4 = ld4(st.x + row), u4 = ld4(st.u + row);
            const float gg[4] = {g4.x, g4.y, g4.z, g4.w};
            const float mm[4] = {m4.x, m4.y, m4.z, m4.w};
            const float xx[4] = {x4.x, x4.y, x4.z, x4.w};
            const float uu[4] = {u4.x, u4.y, u4.z, u4.w};
            float mo[4], xo[4], uo[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                mo[k] = momentum(c, mm[k], gg[k]);              // momentum update
                const float s = f_mul(gamma, mo[k]);
                xo[k] = f_sub(xx[k], f_div(s, d[k]));           // model update
                uo[k] = f_add(uu[k], s);                        // buffer update
                if (DO_VAR) G[k] += (double)gg[k];
            }
            st4(st.m + row, make_float4(mo[0], mo[1], mo[2], mo[3]));
            st4(st.x + row, make_float4(xo[0], xo[1], xo[2], xo[3]));
            st4(st.u + row, make_float4(uo[0], uo[1], uo[2], uo[3]));
        }
        if (DO_VAR) {
            const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
            float vo[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) vo[k] = variance(c, vv[k], mean_round(G[k], st.W));  // variance update
            st4(st.v_next + j, make_float4(vo[0], vo[1], vo[2], vo[3]));
        }
    }
}

__global__ void __launch_bounds__(256)
variance_kernel(StateView st, GradPtrs g, Consts c, int g_aligned, long long first4, long long end4)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long q = first4 + (long long)blockIdx.x * blockDim.x + threadIdx.x; q < end4; q += stride) {
        const long long j = q << 2;
        double G[4] = {0.0, 0.0, 0.0, 0.0};
        for (int i = 0; i < st.W; ++i) {
            const float4 g4 = ld_grad4(g.p[i], j, st.n, g_aligned);
            G[0] += (double)g4.x; G[1] += (double)g4.y; G[2] += (double)g4.z; G[3] += (double)g4.w;
        }
        const float4 v4 = ld4(st.v + j);
        st4(st.v_next + j, make_float4(variance(c, v4.x, mean_round(G[0], st.W)),
                                       variance(c, v4.y, mean_round(G[1], st.W)),
                                       variance(c, v4.z, mean_round(G[2], st.W)),
                                       variance(c, v4.w, mean_round(G[3], st.W))));
    }
}

// ---------------------------------------------------------------------------
// Chunk-per-block helpers.  A warp owns tiles of 128 consecutive coordinates of
// the chunk (4 words), lane l the coordinates 4l..4l+3 of the tile; a thread
// touches the same coordinates in every pass, so shared memory needs no
// barrier beyond those of the block sums.
// ---------------------------------------------------------------------------
struct ChunkGeom {
    long long c0;  // first coordinate of the chunk
    int len;       // its true length (the last chunk may be short)
};
__device__ __forceinline__ ChunkGeom chunk_geom(const StateView &st, long long c)
{
    ChunkGeom g;
    g.c0 = c * st.chunk;
    const long long rest = st.n - g.c0;
    g.len = rest < st.chunk ? (int)rest : st.chunk;
    return g;
}

// Second half of Eq. 3 for one tile: sign bits, compressed values, error
// (written back in place of the input), packed word.  z[k] is the value being
// compressed; on return z[k] holds z - z_hat (0 where invalid) and hat[k] the
// compressed value (0 where invalid).  Lanes 0..3 hold the tile's words.
__device__ __forceinline__ uint32_t compress_tile(float z[4], float hat[4], float scale, int idx, int len)
{
    bool b[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const bool valid = idx + k < len;
        b[k] = valid && (z[k] >= 0.0f);  // +0 and -0 count as non-negative, NaN as negative
        hat[k] = valid ? (b[k] ? scale : -scale) : 0.0f;
        z[k] = valid ? f_sub(z[k], hat[k]) : 0.0f;
    }
    return pack_tile(b);
}

// A chunk above 4096 coordinates is shared by a thread-block cluster of CS blocks (2 or 4), each
// taking chunk / CS consecutive coordinates, so that a block stays as small as the ones that move
// chunk 4096 fastest.  The blocks' binary64 partial l1 sums meet through distributed shared
// memory: every block writes its partial into slot [its rank] of every block's `slots`, and after
// the cluster barrier every thread adds the CS slots in rank order.
template <int CS>
__device__ __forceinline__ double cluster_sum(double block_total, double *slots)
{
    if (CS == 1) return block_total;
    cg::cluster_group cluster = cg::this_cluster();
    const unsigned rank = cluster.block_rank();
    if (threadIdx.x < CS) cluster.map_shared_rank(slots, threadIdx.x)[rank] = block_total;
    cluster.sync();
    double total = 0.0;
#pragma unroll
    for (int q = 0; q < CS; ++q) total += slots[q];
    return total;
}

// The coordinates [lo, lo + mine) of the chunk that block `rank` of a CS-block cluster takes.
struct BlockSpan {
    int lo, mine;
};
template <int CS>
__device__ __forceinline__ BlockSpan block_span(const StateView &st, const ChunkGeom &cg, int rank)
{
    BlockSpan b;
    const int span = st.chunk / CS;
    b.lo = rank * span;
    const int hi = b.lo + span < cg.len ? b.lo + span : cg.len;
    b.mine = hi > b.lo ? hi - b.lo : 0;
    return b;
}

// Worker side of Algorithm 3 for (chunk first_chunk + blockIdx.x, worker blockIdx.y), the chunk
// held in registers: thread t takes the float4 groups t, t + blockDim, ... (ITER of them), issues
// all its loads before the first use, and keeps z = u + delta in registers across the block sum.
// The block needs no shared memory for the chunk and has 2 ITER 128-bit loads in flight per
// thread, which is what fills the memory pipeline (measured at n = 2^28, W = 16: chunk 4096
// 6.94 TB/s against 6.74 with the chunk staged in shared memory by a loop of dependent
// iterations; chunk 16384 6.54 against 5.62).
// EXTERNAL: what is compressed is z + delta with z read from caller-owned buffers (Algorithm 3 on an
// arbitrary input, zoa_onebit_allreduce) instead of u + delta; 1 = by guarded loads (any alignment,
// exactly n elements), 2 = the buffers are 16-byte aligned and the chunk is full, so plain
// 128-bit loads do (a format known at compile time keeps all the loads ahead of the first use).
template <int ITER, int EXTERNAL>
__global__ void __launch_bounds__(512, 2) compress_kernel(StateView st, long long first_chunk, const __grid_constant__ GradPtrs z_in, int z_fmt)
{
    __shared__ double scratch[34];
    const long long chunk_id = first_chunk + blockIdx.x;
    const ChunkGeom cg = chunk_geom(st, chunk_id);
    const int i = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const long long row = (long long)i * st.n_pad + cg.c0;
    const float *z_row = EXTERNAL ? z_in.p[i] : nullptr;
    // Loads go out in batches of BATCH float4 pairs, every load of a batch before its first use (with
    // caller-owned inputs sixteen pairs at once do not fit the registers two resident blocks leave).
    constexpr int BATCH = (EXTERNAL && ITER > 4) ? 4 : ITER;
    float z[ITER][4];
    double l1 = 0.0;
#pragma unroll
    for (int h = 0; h < ITER; h += BATCH) {
        float4 u4[BATCH], e4[BATCH];
#pragma unroll
        for (int q = 0; q < BATCH; ++q) {
            const int idx = 4 * ((h + q) * blockDim.x + threadIdx.x);
            const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
            if (EXTERNAL == 2 && cg.len == st.chunk) u4[q] = idx < cg.len ? ld4_stream(z_row + cg.c0 + idx) : zero;
            else if (EXTERNAL) u4[q] = idx < cg.len ? ld_grad4(z_row, cg.c0 + idx, st.n, z_fmt) : zero;
            else u4[q] = idx < cg.len ? ld4_stream(st.u + row + idx) : zero;     // whole float4 groups: the rows' padding is zero
            e4[q] = idx < cg.len ? ld4_stream(st.dw + row + idx) : zero;
        }
#pragma unroll
        for (int q = 0; q < BATCH; ++q) {
            const int it = h + q;
            z[it][0] = f_add(u4[q].x, e4[q].x); z[it][1] = f_add(u4[q].y, e4[q].y);
            z[it][2] = f_add(u4[q].z, e4[q].z); z[it][3] = f_add(u4[q].w, e4[q].w);
            l1 += fabs((double)z[it][0]) + fabs((double)z[it][1]) + fabs((double)z[it][2]) + fabs((double)z[it][3]);
        }
    }
    const float scale = chunk_scale(block_sum(l1, scratch), cg.len);
#pragma unroll
    for (int it = 0; it < ITER; ++it) {
        const int idx = 4 * (it * blockDim.x + threadIdx.x);
        const int base = idx - 4 * lane;                   // first coordinate of the warp's 128
        float hat[4];
        const uint32_t word = compress_tile(z[it], hat, scale, idx, cg.len);
        if (idx < cg.len) st4_stream(st.dw + row + idx, make_float4(z[it][0], z[it][1], z[it][2], z[it][3]));
        if (lane < 4 && base + 32 * lane < cg.len)
            st.words_w[(long long)i * st.words_stride + ((cg.c0 + base) >> 5) + lane] = word;
    }
    if (threadIdx.x == 0) st.scales_w[(long long)i * st.n_chunks + chunk_id] = scale;
}

// Server side of Algorithm 3 and the post-sync updates of Algorithm 1 for one tile whose
// server input a[k] is known: compress it, keep the server error, rebuild m and x,
// clear u, on every worker.  `scale` is the chunk's server magnitude.
__device__ __forceinline__ void server_tile(const StateView &st, const Consts &c, const ChunkGeom &cg,
                                            int base, int lane, float a[4], float scale, float gamma_sum)
{
    const int idx = base + 4 * lane;
    float hat[4];
    const uint32_t word = compress_tile(a, hat, scale, idx, cg.len);  // a[] now holds the new server error
    if (lane < 4 && base + 32 * lane < cg.len) st.words_s[((cg.c0 + base) >> 5) + lane] = word;
    if (idx >= cg.len) return;
    const long long j = cg.c0 + idx;
    st4(st.ds + j, make_float4(a[0], a[1], a[2], a[3]));
    const float4 v4 = ld4(st.v + j), xs4 = ld4(st.xs + j);
    const float vv[4] = {v4.x, v4.y, v4.z, v4.w}, xs[4] = {xs4.x, xs4.y, xs4.z, xs4.w};
    float mo[4], xo[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const bool valid = idx + k < cg.len;
        mo[k] = valid ? f_div(hat[k], gamma_sum) : 0.0f;                        // momentum approximation
        xo[k] = valid ? f_sub(xs[k], f_div(hat[k], denom(c, vv[k]))) : 0.0f;    // model sync
    }
    const float4 m4 = make_float4(mo[0], mo[1], mo[2], mo[3]);
    const float4 x4 = make_float4(xo[0], xo[1], xo[2], xo[3]);
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    st4(st.xs + j, x4);
    for (int i = 0; i < st.W; ++i) {
        const long long row = (long long)i * st.n_pad + j;
        st4(st.m + row, m4);
        st4(st.x + row, x4);
        st4(st.u + row, zero);                                                   // buffer reset
    }
}

// Server side for chunk first_chunk + blockIdx.x / CS, reading what compress_kernel sent: the
// chunks the ring kernel (zoa_reduce_pipeline.cu) leaves over, and every shape it does not take.
template <int CS>
__global__ void __launch_bounds__(512) reduce_kernel(StateView st, Consts c, float gamma_sum, long long first_chunk)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *scratch = reinterpret_cast<double *>(smem_raw);
    double *slots = scratch + 34;
    float *scales = reinterpret_cast<float *>(smem_raw + 42 * sizeof(double));  // kMaxWorkers floats
    float *a_s = scales + kMaxWorkers;                                           // [span]: the server input
    const long long chunk_id = first_chunk + blockIdx.x / CS;
    const ChunkGeom cg = chunk_geom(st, chunk_id);
    const BlockSpan bs = block_span<CS>(st, cg, blockIdx.x % CS);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const long long j0 = cg.c0 + bs.lo;          // this block's first coordinate

    for (int i = threadIdx.x; i < st.W; i += blockDim.x) scales[i] = st.scales_w[(long long)i * st.n_chunks + chunk_id];
    __syncthreads();

    double l1 = 0.0;
    for (int base = warp * 128; base < bs.mine; base += n_warps * 128) {
        const int idx = base + 4 * lane;
        if (idx < bs.mine) {
            double A[4] = {0.0, 0.0, 0.0, 0.0};
            const long long word_idx = (j0 + idx) >> 5;
            const int shift = idx & 31;
            for (int i = 0; i < st.W; ++i) {  // worker order
                const uint32_t nib = st.words_w[(long long)i * st.words_stride + word_idx] >> shift;
                const double s = (double)scales[i];
#pragma unroll
                for (int k = 0; k < 4; ++k) A[k] += ((nib >> k) & 1u) ? s : -s;
            }
            const float4 e4 = ld4(st.ds + j0 + idx);
            const float ee[4] = {e4.x, e4.y, e4.z, e4.w};
            float a[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                a[k] = idx + k < bs.mine ? server_input(A[k], st.W, ee[k]) : 0.0f;
                l1 += fabs((double)a[k]);
            }
            st4(a_s + idx, make_float4(a[0], a[1], a[2], a[3]));
        }
    }
    const float scale = chunk_scale(cluster_sum<CS>(block_sum(l1, scratch), slots), cg.len);
    ChunkGeom mine;             // this block's coordinates seen as a short chunk, for server_tile
    mine.c0 = j0;
    mine.len = bs.mine;
    for (int base = warp * 128; base < bs.mine; base += n_warps * 128) {
        const int idx = base + 4 * lane;
        float a[4] = {0.f, 0.f, 0.f, 0.f};
        if (idx < bs.mine) {
            const float4 a4 = ld4(a_s + idx);
            a[0] = a4.x; a[1] = a4.y; a[2] = a4.z; a[3] = a4.w;
        }
        server_tile(st, c, mine, base, lane, a, scale, gamma_sum);
    }
    if (threadIdx.x == 0 && blockIdx.x % CS == 0) st.scales_s[chunk_id] = scale;
}

// A whole sync step for chunk chunk_offset + blockIdx.x: the local updates in registers, worker
// compression, server, the post-sync updates.  The half-step m, x, u never reach memory;
// x is not even read (the model sync rebuilds it from x_sync).  Takes every shape: ragged last
// chunk, unaligned or 16-bit gradients, any chunk that is a multiple of 32 up to 16384.
// Thread t takes the float4 groups t, t + blockDim, ... (ITER of them) of every worker in turn:
// loads in batches of two groups (eight 128-bit loads in flight), z in registers across the block
// sum; each worker's sign words stay in shared memory and the server part rebuilds the mean from
// them in worker order, so nothing per coordinate is kept between workers.
// GFMT as in local_step_kernel (aligned binary32 at compile time, or -1 for the argument).
template <int ITER, int GFMT>
__global__ void __launch_bounds__(ITER > 4 ? 512 : 256, ITER > 4 ? 2 : 4)
step_sync_kernel(StateView st, GradPtrs g, Consts c, float gamma, float gamma_sum, int g_fmt_arg, long long chunk_offset)
{
    const int g_aligned = GFMT >= 0 ? GFMT : g_fmt_arg;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *scratch = reinterpret_cast<double *>(smem_raw);                      // 34 doubles
    float *scales = reinterpret_cast<float *>(smem_raw + 34 * sizeof(double));   // kMaxWorkers floats
    uint32_t *bits_sm = reinterpret_cast<uint32_t *>(scales + kMaxWorkers);      // [W][chunk / 32]
    const long long chunk_id = chunk_offset + blockIdx.x;
    const ChunkGeom cg = chunk_geom(st, chunk_id);
    const int lane = threadIdx.x & 31;
    const int words_per_chunk = st.chunk >> 5;
    constexpr int BATCH = ITER < 2 ? 1 : 2;

    for (int i = 0; i < st.W; ++i) {
        const long long row = (long long)i * st.n_pad + cg.c0;
        const float *gi = g.p[i];
        float z[ITER][4];
        double l1 = 0.0;
#pragma unroll
        for (int h = 0; h < ITER; h += BATCH) {
            float4 g4[BATCH], m4[BATCH], u4[BATCH], e4[BATCH];
#pragma unroll
            for (int q = 0; q < BATCH; ++q) {
                const int idx = 4 * ((h + q) * blockDim.x + threadIdx.x);
                const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
                g4[q] = idx < cg.len ? ld_grad4(gi, cg.c0 + idx, st.n, g_aligned) : zero;
                m4[q] = idx < cg.len ? ld4_stream(st.m + row + idx) : zero;
                u4[q] = idx < cg.len ? ld4_stream(st.u + row + idx) : zero;
                e4[q] = idx < cg.len ? ld4_stream(st.dw + row + idx) : zero;
            }
#pragma unroll
            for (int q = 0; q < BATCH; ++q) {
                const float gg[4] = {g4[q].x, g4[q].y, g4[q].z, g4[q].w}, mm[4] = {m4[q].x, m4[q].y, m4[q].z, m4[q].w};
                const float uu[4] = {u4[q].x, u4[q].y, u4[q].z, u4[q].w}, ee[4] = {e4[q].x, e4[q].y, e4[q].z, e4[q].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float step = f_mul(gamma, momentum(c, mm[k], gg[k]));     // momentum update, buffer update
                    z[h + q][k] = f_add(f_add(uu[k], step), ee[k]);                 // u_{t+1/2} + delta
                    l1 += fabs((double)z[h + q][k]);
                }
            }
        }
        const float scale = chunk_scale(block_sum(l1, scratch), cg.len);
#pragma unroll
        for (int it = 0; it < ITER; ++it) {
            const int idx = 4 * (it * blockDim.x + threadIdx.x);
            const int base = idx - 4 * lane;                   // first coordinate of the warp's 128
            float hat[4];
            const uint32_t word = compress_tile(z[it], hat, scale, idx, cg.len);
            if (idx < cg.len) st4_stream(st.dw + row + idx, make_float4(z[it][0], z[it][1], z[it][2], z[it][3]));
            if (lane < 4 && base + 32 * lane < cg.len) {
                st.words_w[(long long)i * st.words_stride + ((cg.c0 + base) >> 5) + lane] = word;
                bits_sm[i * words_per_chunk + (base >> 5) + lane] = word;
            }
        }
        if (threadIdx.x == 0) {
            st.scales_w[(long long)i * st.n_chunks + chunk_id] = scale;
            scales[i] = scale;
        }
    }
    __syncthreads();      // every worker's words and magnitude are in shared memory

    // ---- server: mean of the compressed buffers + server error, compress again, post-sync rows ----
    float a[ITER][4];
    double l1 = 0.0;
#pragma unroll
    for (int it = 0; it < ITER; ++it) {
        const int idx = 4 * (it * blockDim.x + threadIdx.x);
        double A[4] = {0.0, 0.0, 0.0, 0.0};
        float4 e4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (idx < cg.len) {
            e4 = ld4(st.ds + cg.c0 + idx);
            const int shift = idx & 31;
            for (int i = 0; i < st.W; ++i) {   // worker order
                const uint32_t nib = bits_sm[i * words_per_chunk + (idx >> 5)] >> shift;
                const double sc = (double)scales[i];
#pragma unroll
                for (int k = 0; k < 4; ++k) A[k] += ((nib >> k) & 1u) ? sc : -sc;
            }
        }
        const float ee[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            a[it][k] = idx + k < cg.len ? server_input(A[k], st.W, ee[k]) : 0.0f;
            l1 += fabs((double)a[it][k]);
        }
    }
    const float scale = chunk_scale(block_sum(l1, scratch), cg.len);
#pragma unroll
    for (int it = 0; it < ITER; ++it) {
        const int idx = 4 * (it * blockDim.x + threadIdx.x);
        server_tile(st, c, cg, idx - 4 * lane, lane, a[it], scale, gamma_sum);
    }
    if (threadIdx.x == 0) st.scales_s[chunk_id] = scale;
}

// ---------------------------------------------------------------------------
// One worker per GPU (the paper's own mapping: workers send packed buffers to the server
// that owns a range of chunks, the server sends its packed result to every worker).
// The collectives run between these two kernels; see distributed.py.
// ---------------------------------------------------------------------------

// Server side of Algorithm 3 alone for chunk first_chunk + blockIdx.x, reading packed buffers
// gathered from W_total workers: words_in[w][range words], scales_in[w][range chunks], both
// starting at the range's first chunk.  Writes the server error, words_s and scales_s, and the
// result itself to z_bar if that is not NULL (caller-owned, exactly n floats, any alignment).
// `out` lists where else the packed result of the range is to be stored (every rank's
// words_s / scales_s, peer pointers included); out.world == 0 for none.
//
// With 12 to 14 bytes per coordinate this step is bound by instructions, not by memory, if the sum
// over the workers is taken bit by bit (W selects and W additions per coordinate), so it is looked
// up in tables (see table_sum_is_exact in zoa_device.cuh); a chunk whose magnitudes are too far
// apart for that takes the worker-by-worker loop.

// One chunk of dist_server_kernel.  FULL: the chunk has its full length and z_bar (if any) takes
// 128-bit stores, so that no coordinate needs a bounds check.
template <int ITER, bool FULL>
__device__ __forceinline__ void server_chunk(const StateView &st, const uint32_t *words_in, long long words_in_stride, int W_total,
                                          long long chunk_word0, const PeerOut &out, float *z_bar, bool z_bar_aligned, const ChunkGeom cg, long long chunk_id,
                                          double *scratch, const double *table, const float *scales, bool fast)
{
    const int lane = threadIdx.x & 31;
    const uint32_t sel = (threadIdx.x & 3u) | ((4u + (threadIdx.x & 3u)) << 4);
    const bool w_pow2 = (W_total & (W_total - 1)) == 0;
    const double inv_w = __longlong_as_double((long long)(1023 - (31 - __clz(W_total))) << 52);
    float a[ITER][8];
    double l1 = 0.0;
#pragma unroll
    for (int it = 0; it < ITER; ++it) {
        const int idx = 8 * (it * blockDim.x + threadIdx.x);
        const bool active = FULL || idx < cg.len;
        float4 e0 = make_float4(0.f, 0.f, 0.f, 0.f), e1 = e0;
        if (active) e0 = ld4(st.ds + cg.c0 + idx);
        if (FULL || idx + 4 < cg.len) e1 = ld4(st.ds + cg.c0 + idx + 4);
        double A[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
        const uint32_t *col = words_in + chunk_word0 + (idx >> 5);
        for (int i0 = 0; i0 < W_total; i0 += 16) {
            uint32_t w[16];
            const int left = W_total - i0;
#pragma unroll
            for (int gg = 0; gg < 4; ++gg) {
                if (4 * gg < left) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        w[4 * gg + k] = active && 4 * gg + k < left ? *col : 0u;
                        col += words_in_stride;
                    }
                }
            }
#pragma unroll
            for (int gg = 0; gg < 4; ++gg) {
                if (4 * gg < left) {
                    const uint32_t x = gather_bytes(w[4 * gg], w[4 * gg + 1], w[4 * gg + 2], w[4 * gg + 3], sel);
                    if (fast) {
                        const char *t = reinterpret_cast<const char *>(table + ((i0 >> 2) + gg) * 16);
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const double entry = *reinterpret_cast<const double *>(t + table_offset(x, c));
                            A[c] = (i0 == 0 && gg == 0) ? entry : __dadd_rn(A[c], entry);
                        }
                    } else {
                        for (int k = 0; k < 4 && 4 * gg + k < left; ++k) {
                            const double sc = (double)scales[i0 + 4 * gg + k];
                            const uint32_t byte = x >> (8 * k);
#pragma unroll
                            for (int c = 0; c < 8; ++c) A[c] = __dadd_rn(A[c], ((byte >> c) & 1u) ? sc : -sc);
                        }
                    }
                }
            }
        }
        const float ee[8] = {e0.x, e0.y, e0.z, e0.w, e1.x, e1.y, e1.z, e1.w};
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const double q = w_pow2 ? __dmul_rn(A[c], inv_w) : __ddiv_rn(A[c], (double)W_total);
            const float v = __double2float_rn(__dadd_rn(q, (double)ee[c]));
            a[it][c] = FULL || idx + c < cg.len ? v : 0.0f;
            l1 += fabs((double)a[it][c]);
        }
    }
    const float scale = chunk_scale(block_sum(l1, scratch), cg.len);
#pragma unroll
    for (int it = 0; it < ITER; ++it) {
        const int idx = 8 * (it * blockDim.x + threadIdx.x);
        float hat[8];
        uint32_t bits = 0;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const bool valid = FULL || idx + c < cg.len;
            const bool b = valid && (a[it][c] >= 0.0f);
            hat[c] = valid ? (b ? scale : -scale) : 0.0f;
            a[it][c] = valid ? f_sub(a[it][c], hat[c]) : 0.0f;
            bits |= (b ? 1u : 0u) << c;
        }
        bits <<= 8 * (lane & 3);
        bits |= __shfl_xor_sync(0xffffffffu, bits, 1);
        bits |= __shfl_xor_sync(0xffffffffu, bits, 2);
        if ((lane & 3) == 0 && (FULL || idx < cg.len)) {
            const long long w = (cg.c0 + idx) >> 5;
            st.words_s[w] = bits;
            for (int r = 0; r < out.world; ++r) out.words_s[r][w] = bits;
        }
        if (FULL || idx < cg.len) st4(st.ds + cg.c0 + idx, make_float4(a[it][0], a[it][1], a[it][2], a[it][3]));
        if (FULL || idx + 4 < cg.len) st4(st.ds + cg.c0 + idx + 4, make_float4(a[it][4], a[it][5], a[it][6], a[it][7]));
        if (z_bar) {
            if (z_bar_aligned && (FULL || idx + 8 <= cg.len)) {
                st4_stream(z_bar + cg.c0 + idx, make_float4(hat[0], hat[1], hat[2], hat[3]));
                st4_stream(z_bar + cg.c0 + idx + 4, make_float4(hat[4], hat[5], hat[6], hat[7]));
            } else {
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    if (idx + c < cg.len) z_bar[cg.c0 + idx + c] = hat[c];
            }
        }
    }
    if (threadIdx.x == 0) {
        st.scales_s[chunk_id] = scale;
        for (int r = 0; r < out.world; ++r) out.scales_s[r][chunk_id] = scale;
    }
}

template <int ITER>
__global__ void __launch_bounds__(512, 2) dist_server_kernel(const __grid_constant__ StateView st, const uint32_t *words_in, long long words_in_stride,
                                   const float *scales_in, long long scales_in_stride, int W_total,
                                   long long first_chunk, const __grid_constant__ PeerOut out, float *z_bar)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *scratch = reinterpret_cast<double *>(smem_raw);
    double *table = scratch + 34;
    float *scales = reinterpret_cast<float *>(table + (kMaxWorkers / 4) * 16);
    int *exact_flag = reinterpret_cast<int *>(scales + kMaxWorkers);
    const long long chunk_id = first_chunk + blockIdx.x;
    const ChunkGeom cg = chunk_geom(st, chunk_id);
    const int lane = threadIdx.x & 31;
    const long long range_word0 = (first_chunk * st.chunk) >> 5;
    const long long chunk_word0 = (cg.c0 >> 5) - range_word0;
    const bool z_bar_aligned = (reinterpret_cast<uintptr_t>(z_bar) & 15u) == 0;
    const int groups = (W_total + 3) >> 2;

    if (threadIdx.x < 32) {
        const float s_lo = lane < W_total ? scales_in[(long long)lane * scales_in_stride + blockIdx.x] : 0.0f;
        const float s_hi = lane + 32 < W_total ? scales_in[(long long)(lane + 32) * scales_in_stride + blockIdx.x] : 0.0f;
        if (lane < W_total) scales[lane] = s_lo;
        if (lane + 32 < W_total) scales[lane + 32] = s_hi;
        const bool exact = table_sum_is_exact(s_lo, s_hi, W_total);
        if (lane == 0) *exact_flag = exact;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < 16 * groups; e += blockDim.x) table[e] = table_entry(scales, W_total, e);
    __syncthreads();
    const bool fast = *exact_flag != 0;
    if (cg.len == st.chunk && 8 * ITER * (int)blockDim.x == st.chunk && (!z_bar || z_bar_aligned))   // every thread has eight valid coordinates per pass
        server_chunk<ITER, true>(st, words_in, words_in_stride, W_total, chunk_word0, out, z_bar, z_bar_aligned, cg, chunk_id, scratch, table, scales, fast);
    else
        server_chunk<ITER, false>(st, words_in, words_in_stride, W_total, chunk_word0, out, z_bar, z_bar_aligned, cg, chunk_id, scratch, table, scales, fast);
}

// Worker side of Algorithm 3 for the handle's single worker and chunk blockIdx.x, the packed
// words and the magnitude stored straight into the receive buffer of the rank that serves the
// chunk (and into the handle's own words_w / scales_w).  FUSED: the step is a sync step, so the
// momentum and buffer updates of Algorithm 1 are formed in registers from g, m, u and only the
// new compression error is written; otherwise u already holds the half-step buffer.
template <bool FUSED, int GFMT>
__global__ void dist_pack_push_kernel(StateView st, const float *g, Consts c, float gamma, int g_fmt_arg, PushPlan plan)
{
    const int g_fmt = GFMT >= 0 ? GFMT : g_fmt_arg;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *scratch = reinterpret_cast<double *>(smem_raw);        // 33 doubles
    float *z_s = reinterpret_cast<float *>(smem_raw + 34 * sizeof(double));
    const long long chunk_id = blockIdx.x;
    const ChunkGeom cg = chunk_geom(st, chunk_id);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    int server = 0;
    while (server + 1 < plan.world && chunk_id >= plan.chunk_begin[server + 1]) ++server;
    const long long range_chunk0 = plan.chunk_begin[server];
    const long long range_word0 = (range_chunk0 * st.chunk) >> 5;
    uint32_t *words_out = plan.words[server];
    float *scales_out = plan.scales[server];

    double l1 = 0.0;
    for (int base = warp * 128; base < cg.len; base += n_warps * 128) {
        const int idx = base + 4 * lane;
        if (idx < cg.len) {
            const long long j = cg.c0 + idx;
            float4 u4 = ld4(st.u + j);
            const float4 e4 = ld4(st.dw + j);
            if (FUSED) {
                const float4 g4 = ld_grad4(g, j, st.n, g_fmt), m4 = ld4(st.m + j);
                u4 = make_float4(f_add(u4.x, f_mul(gamma, momentum(c, m4.x, g4.x))), f_add(u4.y, f_mul(gamma, momentum(c, m4.y, g4.y))),
                                 f_add(u4.z, f_mul(gamma, momentum(c, m4.z, g4.z))), f_add(u4.w, f_mul(gamma, momentum(c, m4.w, g4.w))));
            }
            const float4 z4 = make_float4(f_add(u4.x, e4.x), f_add(u4.y, e4.y), f_add(u4.z, e4.z), f_add(u4.w, e4.w));
            st4(z_s + idx, z4);
            l1 += fabs((double)z4.x) + fabs((double)z4.y) + fabs((double)z4.z) + fabs((double)z4.w);
        }
    }
    const float scale = chunk_scale(block_sum(l1, scratch), cg.len);
    for (int base = warp * 128; base < cg.len; base += n_warps * 128) {
        const int idx = base + 4 * lane;
        float z[4] = {0.f, 0.f, 0.f, 0.f}, hat[4];
        if (idx < cg.len) {
            const float4 z4 = ld4(z_s + idx);
            z[0] = z4.x; z[1] = z4.y; z[2] = z4.z; z[3] = z4.w;
        }
        const uint32_t word = compress_tile(z, hat, scale, idx, cg.len);
        if (idx < cg.len) st4(st.dw + cg.c0 + idx, make_float4(z[0], z[1], z[2], z[3]));
        if (lane < 4 && base + 32 * lane < cg.len) {
            const long long w = ((cg.c0 + base) >> 5) + lane;
            st.words_w[w] = word;
            words_out[w - range_word0] = word;
        }
    }
    if (threadIdx.x == 0) {
        st.scales_w[chunk_id] = scale;
        scales_out[chunk_id - range_chunk0] = scale;
    }
}

// The post-sync updates of Algorithm 1 from the server's packed result (words_s, scales_s of the whole
// vector): m = u_bar / sum(gamma), x = x_sync - u_bar / sqrt(v + eps), u = 0, on this GPU's workers.
__global__ void __launch_bounds__(256)
dist_apply_kernel(StateView st, Consts c, float gamma_sum)
{
    const long long n4 = (st.n + 3) >> 2;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n4; q += stride) {
        const long long j = q << 2;
        const uint32_t nib = st.words_s[j >> 5] >> (j & 31);
        const float scale = st.scales_s[j / st.chunk];
        const float4 v4 = ld4(st.v + j), xs4 = ld4(st.xs + j);
        const float vv[4] = {v4.x, v4.y, v4.z, v4.w}, xs[4] = {xs4.x, xs4.y, xs4.z, xs4.w};
        float mo[4], xo[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool valid = j + k < st.n;
            const float hat = ((nib >> k) & 1u) ? scale : -scale;
            mo[k] = valid ? f_div(hat, gamma_sum) : 0.0f;                       // momentum approximation
            xo[k] = valid ? f_sub(xs[k], f_div(hat, denom(c, vv[k]))) : 0.0f;   // model sync
        }
        const float4 m4 = make_float4(mo[0], mo[1], mo[2], mo[3]), x4 = make_float4(xo[0], xo[1], xo[2], xo[3]);
        st4(st.xs + j, x4);
        for (int i = 0; i < st.W; ++i) {
            const long long row = (long long)i * st.n_pad + j;
            st4(st.m + row, m4);
            st4(st.x + row, x4);
            st4(st.u + row, make_float4(0.f, 0.f, 0.f, 0.f));                   // buffer reset
        }
    }
}

// The variance update of Algorithm 1 when the mean gradient comes from a collective: v_{t+1} from g_bar.
__global__ void __launch_bounds__(256)
dist_variance_kernel(StateView st, Consts c, const float *g_bar)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < st.n; j += stride)
        st.v_next[j] = variance(c, st.v[j], g_bar[j]);
}

// ---------------------------------------------------------------------------
// Algorithm 2: the frozen-variance framework that exchanges gradients instead of
// accumulated updates (1-bit Adam when T_v is an initial run of steps).
// ---------------------------------------------------------------------------

// A T_v step of Algorithm 2 (full-precision AllReduce, variance, momentum, model): mean of the
// gradients, momentum and model update with v_t on every worker, then v_{t+1}.
// GFMT as in local_step_kernel: the gradient format when known at compile time, else -1.
template <int GFMT>
__global__ void __launch_bounds__(256)
alg2_full_kernel(StateView st, GradPtrs g, Consts c, float gamma, int g_fmt_arg)
{
    const int g_aligned = GFMT >= 0 ? GFMT : g_fmt_arg;
    const long long n4 = (st.n + 3) >> 2;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n4; q += stride) {
        const long long j = q << 2;
        double G[4] = {0.0, 0.0, 0.0, 0.0};
        for (int i = 0; i < st.W; ++i) {
            const float4 g4 = ld_grad4(g.p[i], j, st.n, g_aligned);
            G[0] += (double)g4.x; G[1] += (double)g4.y; G[2] += (double)g4.z; G[3] += (double)g4.w;
        }
        const float4 v4 = ld4(st.v + j);
        const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
        float gb[4], d[4], vo[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            gb[k] = mean_round(G[k], st.W);                     // full-precision mean (Algorithm 4)
            d[k] = denom(c, vv[k]);
            vo[k] = variance(c, vv[k], gb[k]);                  // set v_{t+1}
        }
        st4(st.v_next + j, make_float4(vo[0], vo[1], vo[2], vo[3]));
        for (int i = 0; i < st.W; ++i) {
            const long long row = (long long)i * st.n_pad + j;
            const float4 m4 = ld4(st.m + row), x4 = ld4(st.x + row);
            const float mm[4] = {m4.x, m4.y, m4.z, m4.w}, xx[4] = {x4.x, x4.y, x4.z, x4.w};
            float mo[4], xo[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                mo[k] = momentum(c, mm[k], gb[k]);                              // update momentum
                xo[k] = f_sub(xx[k], f_div(f_mul(gamma, mo[k]), d[k]));         // update model (reads v_t)
            }
            st4(st.m + row, make_float4(mo[0], mo[1], mo[2], mo[3]));
            st4(st.x + row, make_float4(xo[0], xo[1], xo[2], xo[3]));
        }
    }
}

// Any other step of Algorithm 2 for chunk chunk_offset + blockIdx.x (Compressed-AllReduce,
// momentum, model): the gradients go through the error-feedback 1-bit AllReduce (Algorithm 3),
// the decompressed mean drives momentum and model on every worker.  Same shape as
// step_sync_kernel: z in registers, the workers' sign words and magnitudes in shared memory.
template <int ITER>
__global__ void __launch_bounds__(ITER > 4 ? 512 : 256, ITER > 4 ? 2 : 4)
alg2_compressed_kernel(StateView st, GradPtrs g, Consts c, float gamma, int g_aligned, long long chunk_offset)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *scratch = reinterpret_cast<double *>(smem_raw);                      // 34 doubles
    float *scales = reinterpret_cast<float *>(smem_raw + 34 * sizeof(double));   // kMaxWorkers floats
    uint32_t *bits_sm = reinterpret_cast<uint32_t *>(scales + kMaxWorkers);      // [W][chunk / 32]
    const long long chunk_id = chunk_offset + blockIdx.x;
    const ChunkGeom cg = chunk_geom(st, chunk_id);
    const int lane = threadIdx.x & 31;
    const int words_per_chunk = st.chunk >> 5;
    constexpr int BATCH = 4;

    for (int i = 0; i < st.W; ++i) {
        const long long row = (long long)i * st.n_pad + cg.c0;
        const float *gi = g.p[i];
        float z[ITER][4];
        double l1 = 0.0;
#pragma unroll
        for (int h = 0; h < ITER; h += BATCH) {
            float4 g4[BATCH], e4[BATCH];
#pragma unroll
            for (int q = 0; q < BATCH; ++q) {
                const int idx = 4 * ((h + q) * blockDim.x + threadIdx.x);
                const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
                g4[q] = idx < cg.len ? ld_grad4(gi, cg.c0 + idx, st.n, g_aligned) : zero;
                e4[q] = idx < cg.len ? ld4_stream(st.dw + row + idx) : zero;
            }
#pragma unroll
            for (int q = 0; q < BATCH; ++q) {
                z[h + q][0] = f_add(g4[q].x, e4[q].x); z[h + q][1] = f_add(g4[q].y, e4[q].y);
                z[h + q][2] = f_add(g4[q].z, e4[q].z); z[h + q][3] = f_add(g4[q].w, e4[q].w);
#pragma unroll
                for (int k = 0; k < 4; ++k) l1 += fabs((double)z[h + q][k]);
            }
        }
        const float scale = chunk_scale(block_sum(l1, scratch), cg.len);
#pragma unroll
        for (int it = 0; it < ITER; ++it) {
            const int idx = 4 * (it * blockDim.x + threadIdx.x);
            const int base = idx - 4 * lane;
            float hat[4];
            const uint32_t word = compress_tile(z[it], hat, scale, idx, cg.len);
            if (idx < cg.len) st4_stream(st.dw + row + idx, make_float4(z[it][0], z[it][1], z[it][2], z[it][3]));
            if (lane < 4 && base + 32 * lane < cg.len) {
                st.words_w[(long long)i * st.words_stride + ((cg.c0 + base) >> 5) + lane] = word;
                bits_sm[i * words_per_chunk + (base >> 5) + lane] = word;
            }
        }
        if (threadIdx.x == 0) {
            st.scales_w[(long long)i * st.n_chunks + chunk_id] = scale;
            scales[i] = scale;
        }
    }
    __syncthreads();

    float a[ITER][4];
    double l1 = 0.0;
#pragma unroll
    for (int it = 0; it < ITER; ++it) {
        const int idx = 4 * (it * blockDim.x + threadIdx.x);
        double A[4] = {0.0, 0.0, 0.0, 0.0};
        float4 e4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (idx < cg.len) {
            e4 = ld4(st.ds + cg.c0 + idx);
            const int shift = idx & 31;
            for (int i = 0; i < st.W; ++i) {   // worker order
                const uint32_t nib = bits_sm[i * words_per_chunk + (idx >> 5)] >> shift;
                const double sc = (double)scales[i];
#pragma unroll
                for (int k = 0; k < 4; ++k) A[k] += ((nib >> k) & 1u) ? sc : -sc;
            }
        }
        const float ee[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            a[it][k] = idx + k < cg.len ? server_input(A[k], st.W, ee[k]) : 0.0f;
            l1 += fabs((double)a[it][k]);
        }
    }
    const float scale = chunk_scale(block_sum(l1, scratch), cg.len);
#pragma unroll 1
    for (int it = 0; it < ITER; ++it) {
        const int idx = 4 * (it * blockDim.x + threadIdx.x);
        const int base = idx - 4 * lane;
        float gb[4];
        const uint32_t word = compress_tile(a[it], gb, scale, idx, cg.len);   // gb = the mean gradient the workers receive
        if (lane < 4 && base + 32 * lane < cg.len) st.words_s[((cg.c0 + base) >> 5) + lane] = word;
        if (idx >= cg.len) continue;
        const long long j = cg.c0 + idx;
        st4(st.ds + j, make_float4(a[it][0], a[it][1], a[it][2], a[it][3]));
        const float4 v4 = ld4(st.v + j);
        const float d[4] = {denom(c, v4.x), denom(c, v4.y), denom(c, v4.z), denom(c, v4.w)};
        // four workers at a time: all eight loads are issued before the first dependent store
        for (int i0 = 0; i0 < st.W; i0 += 4) {
            float4 m4[4], x4[4];
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (i0 + q < st.W) {
                    const long long row = (long long)(i0 + q) * st.n_pad + j;
                    m4[q] = ld4_stream(st.m + row);
                    x4[q] = ld4_stream(st.x + row);
                }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (i0 + q < st.W) {
                    const long long row = (long long)(i0 + q) * st.n_pad + j;
                    const float mm[4] = {m4[q].x, m4[q].y, m4[q].z, m4[q].w}, xx[4] = {x4[q].x, x4[q].y, x4[q].z, x4[q].w};
                    float mo[4], xo[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        mo[k] = momentum(c, mm[k], gb[k]);                              // momentum update
                        xo[k] = f_sub(xx[k], f_div(f_mul(gamma, mo[k]), d[k]));         // model update
                    }
                    st4_stream(st.m + row, make_float4(mo[0], mo[1], mo[2], mo[3]));
                    st4_stream(st.x + row, make_float4(xo[0], xo[1], xo[2], xo[3]));
                }
        }
    }
    if (threadIdx.x == 0) st.scales_s[chunk_id] = scale;
}

// ---------------------------------------------------------------------------
// Large chunks (chunk > 16384, up to the whole vector = Eq. 3 as printed): a chunk no longer fits
// one block, so its l1 norm is taken in two steps - one binary64 partial sum per segment of 4096
// coordinates, then a fixed-order sum of a chunk's partials.  Two facts keep this at one pass over
// the data per side: the sign bits do not depend on the magnitude, so they are packed in the same
// pass that takes the partial sums; and the new error, z - (+-magnitude), can wait - the pass writes
// z itself into the error row, and whoever reads that row next subtracts the magnitude (still in
// scales_w / scales_s) on the way in ("pending" form; zoa_api.cu brings a row to its plain form
// before anything outside these kernels looks at it).
// ---------------------------------------------------------------------------
constexpr int kSegment = 4096;

struct SegGeom {
    long long c;     // chunk
    long long j0;    // first coordinate of the segment
    int len;         // live coordinates in the segment (0 if it lies beyond the chunk's end)
    int chunk_len;   // true length of the chunk
};
__device__ __forceinline__ SegGeom seg_geom(const StateView &st, long long seg, long long segs_per_chunk)
{
    SegGeom g;
    g.c = seg / segs_per_chunk;
    const long long s = seg % segs_per_chunk;
    const long long c0 = g.c * st.chunk;
    const long long rest = st.n - c0;
    const long long clen = rest < st.chunk ? rest : (long long)st.chunk;
    g.chunk_len = (int)clen;
    const long long start = s * kSegment;
    const long long live = clen - start;
    g.len = live <= 0 ? 0 : (live < kSegment ? (int)live : kSegment);
    g.j0 = c0 + start;
    return g;
}

// An error row in pending form holds what was compressed; the error proper is that minus its
// compressed value (Algorithm 3: delta = z - C[z]).
__device__ __forceinline__ float pending_error(float z, float scale) { return f_sub(z, z >= 0.0f ? scale : -scale); }
__device__ __forceinline__ float4 plain_error4(float4 e, bool pending, float scale)
{
    if (!pending) return e;
    return make_float4(pending_error(e.x, scale), pending_error(e.y, scale), pending_error(e.z, scale), pending_error(e.w, scale));
}

// What a worker compresses, four coordinates from j.  SRC 0: u + delta (zoa_onebit_reduce);
// SRC 1: g + delta (Algorithm 2); SRC 2: the half-step buffer formed on the fly,
// (u + gamma m_{t+1/2}) + delta with m_{t+1/2} = beta1 m + (1 - beta1) g (fused sync step).
template <int SRC>
__device__ __forceinline__ float4 lc_worker_input(const StateView &st, const GradPtrs &g, const Consts &c, float gamma,
                                                  int i, long long j, int g_aligned, bool pending, float old_scale)
{
    const long long row = (long long)i * st.n_pad + j;
    const float4 e = plain_error4(ld4(st.dw + row), pending, old_scale);
    float4 a;
    if (SRC == 0) {
        a = ld4(st.u + row);
    } else if (SRC == 1) {
        a = ld_grad4(g.p[i], j, st.n, g_aligned);
    } else {
        const float4 g4 = ld_grad4(g.p[i], j, st.n, g_aligned), m4 = ld4(st.m + row), u4 = ld4(st.u + row);
        a = make_float4(f_add(u4.x, f_mul(gamma, momentum(c, m4.x, g4.x))), f_add(u4.y, f_mul(gamma, momentum(c, m4.y, g4.y))),
                        f_add(u4.z, f_mul(gamma, momentum(c, m4.z, g4.z))), f_add(u4.w, f_mul(gamma, momentum(c, m4.w, g4.w))));
    }
    return make_float4(f_add(a.x, e.x), f_add(a.y, e.y), f_add(a.z, e.z), f_add(a.w, e.w));
}

// Worker side of Algorithm 3, the one pass: z of segment blockIdx.x of worker blockIdx.y goes into
// the error row (pending form), its sign bits into words_w, sum |z| into partials[i][seg].
template <int SRC>
__global__ void __launch_bounds__(512)
lc_worker_pack_kernel(StateView st, GradPtrs g, Consts c, float gamma, int g_aligned, int pending, long long segs_per_chunk,
                      long long n_segs, double *partials)
{
    __shared__ double scratch[34];
    const SegGeom sg = seg_geom(st, blockIdx.x, segs_per_chunk);
    const int i = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const float old_scale = pending ? st.scales_w[(long long)i * st.n_chunks + sg.c] : 0.0f;   // of the previous sync
    double l1 = 0.0;
    for (int base = warp * 128; base < sg.len; base += n_warps * 128) {
        const int idx = base + 4 * lane;
        float z[4] = {0.f, 0.f, 0.f, 0.f};
        if (idx < sg.len) {
            const float4 z4 = lc_worker_input<SRC>(st, g, c, gamma, i, sg.j0 + idx, g_aligned, pending != 0, old_scale);
            z[0] = z4.x; z[1] = z4.y; z[2] = z4.z; z[3] = z4.w;
        }
        bool b[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool valid = idx + k < sg.len;
            if (!valid) z[k] = 0.0f;                 // the rows' padding stays zero
            b[k] = valid && z[k] >= 0.0f;
            l1 += fabs((double)z[k]);
        }
        const uint32_t word = pack_tile(b);
        if (idx < sg.len) st4(st.dw + (long long)i * st.n_pad + sg.j0 + idx, make_float4(z[0], z[1], z[2], z[3]));
        if (lane < 4 && base + 32 * lane < sg.len)
            st.words_w[(long long)i * st.words_stride + ((sg.j0 + base) >> 5) + lane] = word;
    }
    const double total = block_sum(l1, scratch);
    if (threadIdx.x == 0) partials[(long long)i * n_segs + blockIdx.x] = total;
}

// scales[row][c] = (sum of the chunk's partials, in segment order per lane then a fixed tree) / len.
__global__ void lc_scales_kernel(StateView st, const double *partials, long long segs_per_chunk, long long n_segs,
                                 float *scales)
{
    const long long c = blockIdx.x;
    const int row = blockIdx.y;
    const double *p = partials + (long long)row * n_segs + c * segs_per_chunk;
    double sum = 0.0;
    for (long long s = threadIdx.x; s < segs_per_chunk; s += 32) sum += p[s];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (threadIdx.x == 0) {
        const long long rest = st.n - c * st.chunk;
        const int len = (int)(rest < st.chunk ? rest : (long long)st.chunk);
        scales[(long long)row * st.n_chunks + c] = chunk_scale(sum, len);
    }
}

// Server side of Algorithm 3, the one pass: a = mean of the compressed buffers + server error goes
// into the server-error row (pending form), its sign bits into words_s, sum |a| into partials[W][seg].
// 256 threads x 16 coordinates per segment; every load goes out before the first barrier: the W
// word rows of the segment into shared memory, the server errors into registers.
constexpr int kSegIter = kSegment / (4 * 256);

__global__ void __launch_bounds__(256)
lc_server_pack_kernel(StateView st, int pending, long long segs_per_chunk, long long n_segs, double *partials)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *scratch = reinterpret_cast<double *>(smem_raw);
    double *table = scratch + 34;                                                    // [kMaxWorkers / 4][16], see table_sum_is_exact
    float *scales_sm = reinterpret_cast<float *>(table + (kMaxWorkers / 4) * 16);
    int *exact_flag = reinterpret_cast<int *>(scales_sm + kMaxWorkers);
    uint32_t *words_sm = reinterpret_cast<uint32_t *>(exact_flag + 4);               // [W][kSegment / 32]
    const SegGeom sg = seg_geom(st, blockIdx.x, segs_per_chunk);
    const int lane = threadIdx.x & 31;
    constexpr int kWordsPerSeg = kSegment / 32;
    const int n_words = (sg.len + 31) >> 5;
    const long long seg_word0 = sg.j0 >> 5;
    if (threadIdx.x < 32) {
        const float s_lo = lane < st.W ? st.scales_w[(long long)lane * st.n_chunks + sg.c] : 0.0f;
        const float s_hi = lane + 32 < st.W ? st.scales_w[(long long)(lane + 32) * st.n_chunks + sg.c] : 0.0f;
        if (lane < st.W) scales_sm[lane] = s_lo;
        if (lane + 32 < st.W) scales_sm[lane + 32] = s_hi;
        const bool exact = table_sum_is_exact(s_lo, s_hi, st.W);
        if (lane == 0) *exact_flag = exact;
    }
    const float old_scale = pending ? st.scales_s[sg.c] : 0.0f;       // of the previous sync
    const int total = st.W * n_words;
    for (int e0 = threadIdx.x; e0 < total; e0 += 8 * blockDim.x) {
        uint32_t w[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int e = e0 + q * blockDim.x;
            w[q] = e < total ? st.words_w[(long long)(e / n_words) * st.words_stride + seg_word0 + e % n_words] : 0u;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int e = e0 + q * blockDim.x;
            if (e < total) words_sm[(e / n_words) * kWordsPerSeg + e % n_words] = w[q];
        }
    }
    float4 e4[kSegIter];
#pragma unroll
    for (int it = 0; it < kSegIter; ++it) {
        const int idx = 4 * (it * blockDim.x + threadIdx.x);
        e4[it] = idx < sg.len ? ld4(st.ds + sg.j0 + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __syncthreads();
    const int groups = (st.W + 3) >> 2;
    for (int e = threadIdx.x; e < 16 * groups; e += blockDim.x) table[e] = table_entry(scales_sm, st.W, e);
    __syncthreads();
    const bool fast = *exact_flag != 0;
    // the thread's four coordinates are one nibble of a packed word: byte (lane & 7) / 2, its upper half for odd lanes
    const uint32_t byte_sel = ((lane & 7u) >> 1) | ((4u + ((lane & 7u) >> 1)) << 4);
    const int half_shift = (lane & 1) * 4;
    const int last = st.W - 1;
    double l1 = 0.0;
#pragma unroll
    for (int it = 0; it < kSegIter; ++it) {
        const int idx = 4 * (it * blockDim.x + threadIdx.x);
        const int base = idx - 4 * lane;
        float a[4] = {0.f, 0.f, 0.f, 0.f};
        if (idx < sg.len) {
            double A[4] = {0.0, 0.0, 0.0, 0.0};
            const uint32_t *col = words_sm + (idx >> 5);
            for (int g = 0; g < groups; ++g) {
                // a worker index past the last one repeats the last worker's word: its bits select among equal table entries
                const int i1 = min(4 * g + 1, last), i2 = min(4 * g + 2, last), i3 = min(4 * g + 3, last);
                const uint32_t x = gather_bytes(col[4 * g * kWordsPerSeg], col[i1 * kWordsPerSeg], col[i2 * kWordsPerSeg],
                                                col[i3 * kWordsPerSeg], byte_sel) >> half_shift;
                if (fast) {
                    const char *tb = reinterpret_cast<const char *>(table + g * 16);
#pragma unroll
                    for (int k = 0; k < 4; ++k) A[k] = __dadd_rn(A[k], *reinterpret_cast<const double *>(tb + table_offset(x, k)));
                } else {
                    for (int q = 0; q < 4 && 4 * g + q < st.W; ++q) {   // worker order
                        const double sc = (double)scales_sm[4 * g + q];
                        const uint32_t nib = x >> (8 * q);
#pragma unroll
                        for (int k = 0; k < 4; ++k) A[k] += ((nib >> k) & 1u) ? sc : -sc;
                    }
                }
            }
            const float4 p4 = plain_error4(e4[it], pending != 0, old_scale);
            const float ee[4] = {p4.x, p4.y, p4.z, p4.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) a[k] = idx + k < sg.len ? server_input(A[k], st.W, ee[k]) : 0.0f;
        }
        bool b[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            b[k] = idx + k < sg.len && a[k] >= 0.0f;
            l1 += fabs((double)a[k]);
        }
        const uint32_t word = pack_tile(b);
        if (idx < sg.len) st4(st.ds + sg.j0 + idx, make_float4(a[0], a[1], a[2], a[3]));
        if (lane < 4 && base + 32 * lane < sg.len) st.words_s[((sg.j0 + base) >> 5) + lane] = word;
    }
    const double total_l1 = block_sum(l1, scratch);
    if (threadIdx.x == 0) partials[(long long)st.W * n_segs + blockIdx.x] = total_l1;
}

// Momentum and model updates of Algorithm 2 from the server's packed result: g_bar = +-scales_s by words_s.
__global__ void __launch_bounds__(256)
lc_alg2_apply_kernel(StateView st, Consts c, float gamma)
{
    const long long n4 = (st.n + 3) >> 2;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < n4; q += stride) {
        const long long j = q << 2;
        const uint32_t nib = st.words_s[j >> 5] >> (j & 31);
        const float scale = st.scales_s[j / st.chunk];
        const float4 v4 = ld4(st.v + j);
        const float d[4] = {denom(c, v4.x), denom(c, v4.y), denom(c, v4.z), denom(c, v4.w)};
        for (int i = 0; i < st.W; ++i) {
            const long long row = (long long)i * st.n_pad + j;
            const float4 m4 = ld4(st.m + row), x4 = ld4(st.x + row);
            const float mm[4] = {m4.x, m4.y, m4.z, m4.w}, xx[4] = {x4.x, x4.y, x4.z, x4.w};
            float mo[4], xo[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const bool valid = j + k < st.n;
                const float g_bar = ((nib >> k) & 1u) ? scale : -scale;          // what every worker receives
                mo[k] = valid ? momentum(c, mm[k], g_bar) : 0.0f;                               // update momentum
                xo[k] = valid ? f_sub(xx[k], f_div(f_mul(gamma, mo[k]), d[k])) : 0.0f;          // update model
            }
            st4(st.m + row, make_float4(mo[0], mo[1], mo[2], mo[3]));
            st4(st.x + row, make_float4(xo[0], xo[1], xo[2], xo[3]));
        }
    }
}

// Brings an error row from pending to plain form: e = z - (+-scale of its chunk), coordinates [0, n).
__global__ void __launch_bounds__(256)
lc_plain_errors_kernel(float *rows, long long n, long long n_pad, int chunk, const float *scales, long long n_chunks)
{
    float *row = rows + (long long)blockIdx.y * n_pad;
    const float *row_scales = scales + (long long)blockIdx.y * n_chunks;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += stride)
        row[j] = pending_error(row[j], row_scales[j / chunk]);
}

// Debug scan: how many of p[0..count) are NaN or infinite.
__global__ void __launch_bounds__(256) count_nonfinite_kernel(const float *p, long long count, unsigned long long *out)
{
    unsigned long long bad = 0;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += stride)
        bad += !isfinite(p[j]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) bad += __shfl_xor_sync(0xffffffffu, bad, o);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(out, bad);
}

// ---------------------------------------------------------------------------
// Launchers
// ---------------------------------------------------------------------------
static int elementwise_grid(long long n4)
{
    // One float4 per thread and as many blocks as that takes: SMs do not all get the same
    // share of DRAM bandwidth, and the hardware block scheduler evens that out, where a
    // grid capped at a few waves leaves the fast SMs idle at the end (measured: 0.94 ->
    // 1.03 of the copy bandwidth).  The kernels keep their grid-stride loops for n4 > 2^31 * 256.
    long long blocks = (n4 + 255) / 256;
    if (blocks > 0x7fffffffll) blocks = 0x7fffffffll;
    return (int)(blocks < 1 ? 1 : blocks);
}

// The local updates of Algorithm 1 (and the variance update if do_var) for the coordinates [first, end); first is a multiple of 4.
cudaError_t launch_local_step(const StateView &st, const GradPtrs &g, const Consts &c, float gamma,
                              bool do_var, int g_aligned, long long first, long long end, cudaStream_t s)
{
    const long long first4 = first >> 2, end4 = (end + 3) >> 2;
    const int grid = elementwise_grid(end4 - first4);
#define ZOA_LOCAL(VAR, FMT) local_step_kernel<VAR, FMT><<<grid, 256, 0, s>>>(st, g, c, gamma, g_aligned, first4, end4)
    switch (g_aligned) {
    case kGradF32 | kGradAligned: if (do_var) ZOA_LOCAL(true, kGradF32 | kGradAligned); else ZOA_LOCAL(false, kGradF32 | kGradAligned); break;
    case kGradF16 | kGradAligned: if (do_var) ZOA_LOCAL(true, kGradF16 | kGradAligned); else ZOA_LOCAL(false, kGradF16 | kGradAligned); break;
    case kGradBF16 | kGradAligned: if (do_var) ZOA_LOCAL(true, kGradBF16 | kGradAligned); else ZOA_LOCAL(false, kGradBF16 | kGradAligned); break;
    default: if (do_var) ZOA_LOCAL(true, -1); else ZOA_LOCAL(false, -1); break;
    }
#undef ZOA_LOCAL
    return cudaGetLastError();
}

// The variance update of Algorithm 1 for the coordinates [first, end); first is a multiple of 4.
cudaError_t launch_variance(const StateView &st, const GradPtrs &g, const Consts &c, int g_aligned,
                            long long first, long long end, cudaStream_t s)
{
    const long long first4 = first >> 2, end4 = (end + 3) >> 2;
    variance_kernel<<<elementwise_grid(end4 - first4), 256, 0, s>>>(st, g, c, g_aligned, first4, end4);
    return cudaGetLastError();
}

size_t compress_smem(int chunk) { return 34 * sizeof(double) + (size_t)chunk * sizeof(float); }                 // dist_pack_push_kernel

// reduce_kernel: block-sum and cluster scratch, magnitudes, the server input of `span` coordinates
static size_t reduce_span_smem(int span) { return 42 * sizeof(double) + (kMaxWorkers + (size_t)span) * sizeof(float); }

// How many blocks share a chunk in reduce_kernel (see cluster_sum): spans of 4096 coordinates for
// the chunk sizes that divide evenly, one block otherwise.
static int cluster_blocks(int chunk)
{
    if (chunk > 8192 && chunk % 512 == 0) return 4;
    if (chunk > 4096 && chunk % 256 == 0) return 2;
    return 1;
}
// step_sync_kernel, alg2_compressed_kernel: block-sum scratch, the workers' magnitudes and sign words
static size_t step_sync_bits_smem(int W, int chunk) { return 34 * sizeof(double) + kMaxWorkers * sizeof(float) + (size_t)W * (chunk / 32) * sizeof(uint32_t); }

cudaError_t configure_kernels()
{
    cudaError_t e;
    e = cudaFuncSetAttribute(reduce_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)reduce_span_smem(kMaxChunk));
    if (e != cudaSuccess) return e;
    const int sync_smem = (int)step_sync_bits_smem(kMaxWorkers, kMaxChunk);
    e = cudaFuncSetAttribute(alg2_compressed_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, sync_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(alg2_compressed_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, sync_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(step_sync_kernel<4, kGradF32 | kGradAligned>, cudaFuncAttributeMaxDynamicSharedMemorySize, sync_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(step_sync_kernel<8, kGradF32 | kGradAligned>, cudaFuncAttributeMaxDynamicSharedMemorySize, sync_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(step_sync_kernel<4, -1>, cudaFuncAttributeMaxDynamicSharedMemorySize, sync_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(step_sync_kernel<8, -1>, cudaFuncAttributeMaxDynamicSharedMemorySize, sync_smem);
    return e;
}

// A step of Algorithm 2: the whole vector at full precision, or the chunks
// [first_chunk, first_chunk + count) through the 1-bit AllReduce.
cudaError_t launch_alg2(const StateView &st, const GradPtrs &g, const Consts &c, float gamma, bool full_precision,
                        int g_aligned, long long first_chunk, long long count, cudaStream_t s)
{
    if (full_precision) {
        const int grid = elementwise_grid((st.n + 3) / 4);
        switch (g_aligned) {
        case kGradF32 | kGradAligned: alg2_full_kernel<kGradF32 | kGradAligned><<<grid, 256, 0, s>>>(st, g, c, gamma, g_aligned); break;
        case kGradF16 | kGradAligned: alg2_full_kernel<kGradF16 | kGradAligned><<<grid, 256, 0, s>>>(st, g, c, gamma, g_aligned); break;
        case kGradBF16 | kGradAligned: alg2_full_kernel<kGradBF16 | kGradAligned><<<grid, 256, 0, s>>>(st, g, c, gamma, g_aligned); break;
        default: alg2_full_kernel<-1><<<grid, 256, 0, s>>>(st, g, c, gamma, g_aligned); break;
        }
    } else {
        const int iter = st.chunk > 4096 ? 8 : 4;
        const int threads = ((st.chunk + 4 * iter - 1) / (4 * iter) + 31) / 32 * 32;
        const size_t smem = step_sync_bits_smem(st.W, st.chunk);
        if (iter == 8) alg2_compressed_kernel<8><<<(unsigned)count, threads, smem, s>>>(st, g, c, gamma, g_aligned, first_chunk);
        else alg2_compressed_kernel<4><<<(unsigned)count, threads, smem, s>>>(st, g, c, gamma, g_aligned, first_chunk);
    }
    return cudaGetLastError();
}

// Launch of a kernel whose blocks form clusters of CS along x.
template <int CS, typename... KArgs, typename... Args>
static cudaError_t launch_clustered(void (*kern)(KArgs...), dim3 grid, int threads, size_t smem, cudaStream_t s, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

// Worker side of Algorithm 3 for the chunks [first_chunk, first_chunk + count), one block per chunk and worker.
cudaError_t launch_compress(const StateView &st, long long first_chunk, long long count, cudaStream_t s)
{
    // 16 coordinates per thread (32 above chunk 4096), in blocks of at most 512 threads: measured best
    // at every chunk size from 1024 to 16384 (n = 2^28: 6.5 - 6.9 TB/s)
    const int iter = st.chunk > 4096 ? 8 : 4;
    const int thr = ((st.chunk + 4 * iter - 1) / (4 * iter) + 31) / 32 * 32;
    const dim3 grid((unsigned)count, (unsigned)st.W);
    const GradPtrs none{};
    if (iter == 8) compress_kernel<8, 0><<<grid, thr, 0, s>>>(st, first_chunk, none, 0);
    else compress_kernel<4, 0><<<grid, thr, 0, s>>>(st, first_chunk, none, 0);
    return cudaGetLastError();
}

// The same for Algorithm 3 on caller-owned buffers z (W device pointers of n floats, format code as for gradients).
cudaError_t launch_compress_external(const StateView &st, const GradPtrs &z, int z_fmt, cudaStream_t s)
{
    const int iter = st.chunk > 4096 ? 8 : 4;
    const int thr = ((st.chunk + 4 * iter - 1) / (4 * iter) + 31) / 32 * 32;
    const dim3 grid((unsigned)st.n_chunks, (unsigned)st.W);
    if (z_fmt & kGradAligned) {
        if (iter == 8) compress_kernel<8, 2><<<grid, thr, 0, s>>>(st, 0, z, z_fmt);
        else compress_kernel<4, 2><<<grid, thr, 0, s>>>(st, 0, z, z_fmt);
    } else {
        if (iter == 8) compress_kernel<8, 1><<<grid, thr, 0, s>>>(st, 0, z, z_fmt);
        else compress_kernel<4, 1><<<grid, thr, 0, s>>>(st, 0, z, z_fmt);
    }
    return cudaGetLastError();
}

// Server side for the chunks [first_chunk, first_chunk + count), one block (or cluster) per chunk.
cudaError_t launch_reduce(const StateView &st, const Consts &c, float gamma_sum, long long first_chunk, long long count, cudaStream_t s)
{
    const int cs = cluster_blocks(st.chunk), span = st.chunk / cs;
    // With few workers a block has little to move between its barriers, and smaller blocks
    // (more of them per SM) do better.
    const int per_thread = st.W <= 2 ? 32 : 16;
    int thr = 128;
    while (thr < span / per_thread && thr < 512) thr <<= 1;
    const dim3 grid((unsigned)(count * cs));
    const size_t smem = reduce_span_smem(span);
    if (cs == 4) return launch_clustered<4>(reduce_kernel<4>, grid, thr, smem, s, st, c, gamma_sum, first_chunk);
    if (cs == 2) return launch_clustered<2>(reduce_kernel<2>, grid, thr, smem, s, st, c, gamma_sum, first_chunk);
    reduce_kernel<1><<<grid, thr, smem, s>>>(st, c, gamma_sum, first_chunk);
    return cudaGetLastError();
}

// The chunks [first_chunk, first_chunk + count) of a sync step, one block each.
cudaError_t launch_step_sync(const StateView &st, const GradPtrs &g, const Consts &c, float gamma,
                             float gamma_sum, int g_aligned, long long first_chunk, long long count, cudaStream_t s)
{
    // 16 coordinates per thread (32 above chunk 4096), like compress_kernel
    const int iter = st.chunk > 4096 ? 8 : 4;
    const int threads = ((st.chunk + 4 * iter - 1) / (4 * iter) + 31) / 32 * 32;
    const size_t smem = step_sync_bits_smem(st.W, st.chunk);
    const bool fast = g_aligned == (kGradF32 | kGradAligned);
#define ZOA_SYNC(IT, FMT) step_sync_kernel<IT, FMT><<<(unsigned)count, threads, smem, s>>>(st, g, c, gamma, gamma_sum, g_aligned, first_chunk)
    if (iter == 8) { if (fast) ZOA_SYNC(8, kGradF32 | kGradAligned); else ZOA_SYNC(8, -1); }
    else { if (fast) ZOA_SYNC(4, kGradF32 | kGradAligned); else ZOA_SYNC(4, -1); }
#undef ZOA_SYNC
    return cudaGetLastError();
}

}  // namespace zoa

namespace zoa {

long long large_chunk_segments(const StateView &st)
{
    const long long span = st.chunk < st.n ? (long long)st.chunk : st.n;
    return (span + kSegment - 1) / kSegment;
}

// Worker side of Algorithm 3 for chunks too large for one block.  src 0: compress u + delta;
// 1: g + delta (Algorithm 2); 2: the half-step buffer formed on the fly from g, m, u (fused sync
// step; m, x, u are then written by the server pass only).  pending: the worker-error rows are in
// pending form on entry; they are on return in any case.  partials: [W + 1][n_chunks * segments].
cudaError_t launch_large_compress(const StateView &st, const GradPtrs &g, const Consts &c, float gamma, int src,
                                  int g_aligned, bool pending, double *partials, int *launches, cudaStream_t s)
{
    const long long spc = large_chunk_segments(st), n_segs = spc * st.n_chunks;
    const dim3 grid((unsigned)n_segs, (unsigned)st.W);
    if (src == 0) lc_worker_pack_kernel<0><<<grid, 512, 0, s>>>(st, g, c, gamma, g_aligned, pending, spc, n_segs, partials);
    else if (src == 1) lc_worker_pack_kernel<1><<<grid, 512, 0, s>>>(st, g, c, gamma, g_aligned, pending, spc, n_segs, partials);
    else lc_worker_pack_kernel<2><<<grid, 512, 0, s>>>(st, g, c, gamma, g_aligned, pending, spc, n_segs, partials);
    lc_scales_kernel<<<dim3((unsigned)st.n_chunks, (unsigned)st.W), 32, 0, s>>>(st, partials, spc, n_segs, st.scales_w);
    *launches += 2;
    return cudaGetLastError();
}

// Server side.  mode 1: post-sync updates of Algorithm 1 (scalar = sum of learning rates); mode 2:
// momentum and model updates of Algorithm 2 (scalar = learning rate).  pending: as above, for the
// server-error row.
cudaError_t launch_large_server(const StateView &st, const Consts &c, int mode, float scalar, bool pending, double *partials,
                                int *launches, cudaStream_t s)
{
    const long long spc = large_chunk_segments(st), n_segs = spc * st.n_chunks;
    const size_t pack_smem = (34 + (kMaxWorkers / 4) * 16) * sizeof(double) + kMaxWorkers * sizeof(float) + 16
                             + (size_t)st.W * (kSegment / 32) * sizeof(uint32_t);
    lc_server_pack_kernel<<<(unsigned)n_segs, 256, pack_smem, s>>>(st, pending, spc, n_segs, partials);
    lc_scales_kernel<<<dim3((unsigned)st.n_chunks, 1), 32, 0, s>>>(st, partials + (long long)st.W * n_segs, spc, n_segs, st.scales_s);
    if (mode == 1) dist_apply_kernel<<<elementwise_grid((st.n + 3) / 4), 256, 0, s>>>(st, c, scalar);
    else lc_alg2_apply_kernel<<<elementwise_grid((st.n + 3) / 4), 256, 0, s>>>(st, c, scalar);
    *launches += 3;
    return cudaGetLastError();
}

// Error rows from pending to plain form (both kinds, as asked).
cudaError_t launch_plain_errors(const StateView &st, bool workers, bool server, cudaStream_t s)
{
    const unsigned blocks = (unsigned)elementwise_grid((st.n + 3) / 4);
    if (workers) lc_plain_errors_kernel<<<dim3(blocks, (unsigned)st.W), 256, 0, s>>>(st.dw, st.n, st.n_pad, st.chunk, st.scales_w, st.n_chunks);
    if (server) lc_plain_errors_kernel<<<dim3(blocks, 1), 256, 0, s>>>(st.ds, st.n, st.n_pad, st.chunk, st.scales_s, st.n_chunks);
    return cudaGetLastError();
}

}  // namespace zoa

namespace zoa {

cudaError_t launch_dist_server(const StateView &st, const uint32_t *words_in, long long words_in_stride,
                               const float *scales_in, long long scales_in_stride, int W_total,
                               long long first_chunk, long long count, const PeerOut &out, float *z_bar, cudaStream_t s)
{
    // 8, 16 or 32 coordinates per thread: blocks of 128 ... 512 threads for chunks of 1024 ... 16384
    const int iter = st.chunk > 8192 ? 4 : st.chunk > 2048 ? 2 : 1;
    const int thr = ((st.chunk + 8 * iter - 1) / (8 * iter) + 31) / 32 * 32;
    const size_t smem = (34 + (kMaxWorkers / 4) * 16) * sizeof(double) + kMaxWorkers * sizeof(float) + 16;
    switch (iter) {
    case 4: dist_server_kernel<4><<<(unsigned)count, thr, smem, s>>>(st, words_in, words_in_stride, scales_in, scales_in_stride, W_total, first_chunk, out, z_bar); break;
    case 2: dist_server_kernel<2><<<(unsigned)count, thr, smem, s>>>(st, words_in, words_in_stride, scales_in, scales_in_stride, W_total, first_chunk, out, z_bar); break;
    default: dist_server_kernel<1><<<(unsigned)count, thr, smem, s>>>(st, words_in, words_in_stride, scales_in, scales_in_stride, W_total, first_chunk, out, z_bar); break;
    }
    return cudaGetLastError();
}

// Worker side of the 1-bit AllReduce for a single-worker handle with the packed result stored
// through `plan`; g != nullptr: fused with the local updates of a sync step.
cudaError_t launch_dist_pack_push(const StateView &st, const float *g, const Consts &c, float gamma, int g_fmt,
                                  const PushPlan &plan, cudaStream_t s)
{
    static SmemLimitOnce once[3];
    const int max_smem = (int)compress_smem(kMaxChunk);
    cudaError_t e = once[0].ensure(dist_pack_push_kernel<false, -1>, max_smem);
    if (e == cudaSuccess) e = once[1].ensure(dist_pack_push_kernel<true, -1>, max_smem);
    if (e == cudaSuccess) e = once[2].ensure(dist_pack_push_kernel<true, kGradF32 | kGradAligned>, max_smem);
    if (e != cudaSuccess) return e;
    int thr = 128;
    while (thr < st.chunk / 16 && thr < 1024) thr <<= 1;
    const unsigned grid = (unsigned)st.n_chunks;
    const size_t smem = compress_smem(st.chunk);
    if (!g) dist_pack_push_kernel<false, -1><<<grid, thr, smem, s>>>(st, nullptr, c, gamma, g_fmt, plan);
    else if (g_fmt == (kGradF32 | kGradAligned)) dist_pack_push_kernel<true, kGradF32 | kGradAligned><<<grid, thr, smem, s>>>(st, g, c, gamma, g_fmt, plan);
    else dist_pack_push_kernel<true, -1><<<grid, thr, smem, s>>>(st, g, c, gamma, g_fmt, plan);
    return cudaGetLastError();
}

cudaError_t launch_dist_apply(const StateView &st, const Consts &c, float gamma_sum, cudaStream_t s)
{
    dist_apply_kernel<<<elementwise_grid((st.n + 3) / 4), 256, 0, s>>>(st, c, gamma_sum);
    return cudaGetLastError();
}

cudaError_t launch_dist_variance(const StateView &st, const Consts &c, const float *g_bar, cudaStream_t s)
{
    dist_variance_kernel<<<elementwise_grid((st.n + 255) / 256 * 64), 256, 0, s>>>(st, c, g_bar);
    return cudaGetLastError();
}

}  // namespace zoa

namespace zoa {

cudaError_t launch_count_nonfinite(const float *p, long long count, unsigned long long *out, int sm_count, cudaStream_t s)
{
    long long blocks = (count + 255) / 256;
    if (blocks > (long long)sm_count * 32) blocks = (long long)sm_count * 32;
    count_nonfinite_kernel<<<(unsigned)(blocks < 1 ? 1 : blocks), 256, 0, s>>>(p, count, out);
    return cudaGetLastError();
}

}  // namespace zoa
