// reduce_pipelined_kernel: the second half of zoa_onebit_reduce - Algorithm 3, server side, and
// Algorithm 1's sync branch (momentum approximation, model sync, buffer reset) - as a persistent,
// warp-specialised kernel for sm_100a.
//
// This step writes 12 W + 8 bytes per coordinate and reads about 14, and under that much store
// traffic a load takes long (a block that loads, sums and then stores spends most of its time
// waiting for its loads).  So every input (the W packed word rows and magnitudes, the server
// error, v, x_sync) is prefetched through a ring of shared-memory stages by a copy-issuing
// warp, and every row store leaves through the copy engine too: the post-sync m, x and u = 0 are
// the same for all W workers, so the consumers form one tile of each in shared memory and a
// store-issuing warp sends it to the 3 W + 1 rows as bulk asynchronous stores.  The consumers
// only compute.
//
// Blocks take work units from a global counter (see zoa_pipeline.cu for why) and every wait is bounded.
// A unit is `span` = max(chunk, 2048) consecutive coordinates: TILES tiles of 2048 coordinates
// when the chunk is 2048 ... 16384, or one tile holding G = 2048 / chunk whole chunks when it is
// 128 ... 1024 (then a chunk's l1 norm is the sum over the 16 / G consumer warps that own it).
#include "zoa_internal.h"
#include "zoa_ring.cuh"

namespace zoa {
namespace {

constexpr int kStoreBufs = 3;                        // tiles of (x, m) staged for the store-issuing warp
constexpr int kRingThreads = kConsumers + 64;        // consumers + copy-issuing warp + store-issuing warp

// Shared-memory header of reduce_pipelined_kernel.
struct ReduceShared {
    PipeShared ring;
    unsigned long long staged[kStoreBufs];    // consumers -> store warp: buffer b holds a tile
    unsigned long long drained[kStoreBufs];   // store warp -> consumers: buffer b has been read by the copy engine
    long long dst[kStoreBufs];                // first coordinate of the tile in buffer b, -1 = no more
};

struct ReduceLayout {
    int scales_off, zero_off, staging_off, ring_off;   // bytes from the start of dynamic shared memory
    int stage_bytes, words_off, stage_scales_off;      // inside a ring stage
};
__host__ __device__ inline ReduceLayout reduce_layout(int W, int G)
{
    ReduceLayout l;
    l.scales_off = 1024;                                                   // [kConsumerWarps][W] floats
    l.zero_off = (l.scales_off + kConsumerWarps * W * 4 + 1023) & ~1023;   // one tile of zeros
    l.staging_off = l.zero_off + kTileBytes;                               // kStoreBufs x (x tile, m tile)
    l.ring_off = l.staging_off + kStoreBufs * 2 * kTileBytes;
    l.words_off = kTileBytes;                                              // after the server-error tile
    l.stage_scales_off = l.words_off + W * (kTile / 8);
    const int first = l.stage_scales_off + W * G * 4, second = 2 * kTileBytes;
    l.stage_bytes = ((first > second ? first : second) + 1023) & ~1023;
    return l;
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// Server side of Algorithm 3 + the sync branch of Algorithm 1 for the units [0, a.n_full_chunks).
// ---------------------------------------------------------------------------------------------
template <int TILES, int G>
__global__ void __launch_bounds__(kRingThreads, 1) reduce_pipelined_kernel(const __grid_constant__ PipeArgs a)
{
    constexpr int WPC = kConsumerWarps / G;           // consumer warps per chunk
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    ReduceShared *sh = reinterpret_cast<ReduceShared *>(smem_raw);
    const StateView &st = a.st;
    const int W = st.W;
    const ReduceLayout lay = reduce_layout(W, G);
    float *scales_s = reinterpret_cast<float *>(smem_raw + lay.scales_off);
    float *zero_s = reinterpret_cast<float *>(smem_raw + lay.zero_off);
    float *staging = reinterpret_cast<float *>(smem_raw + lay.staging_off);
    unsigned char *ring = smem_raw + lay.ring_off;
    const int R = a.stages;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int *abort_flag = &sh->ring.abort;
    const long long span = (long long)TILES * kTile;

    if (tid == 0) {
        for (int s = 0; s < R; ++s) {
            mbar_init(smem_addr(&sh->ring.full[s]), 2);       // the copies' arrive + the magnitudes' arrive
            mbar_init(smem_addr(&sh->ring.empty[s]), kConsumerWarps);
        }
        for (int b = 0; b < kStoreBufs; ++b) {
            mbar_init(smem_addr(&sh->staged[b]), kConsumerWarps);
            mbar_init(smem_addr(&sh->drained[b]), 1);
        }
        sh->ring.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // ------------------------- copy-issuing warp (all 32 lanes stay) -------------------------
        RingProducer p(a, &sh->ring, ring, lay.stage_bytes);
        // The unit numbers come from a global counter and the magnitudes from global memory: two
        // round trips that would stand between the tiles of every unit (with one tile per unit and
        // few workers they, not the copies, set the pace).  So the warp runs ahead: it holds the
        // numbers of the next two units, and the magnitudes of a unit's first tile are loaded one
        // unit early into registers (two per lane; more than 64 of them are loaded in place).
        const bool ahead = W * G <= 64;
        long long cur = 0, nxt = 0;
        if (lane == 0) { cur = p.take(); nxt = p.take(); }
        float pre_c[2] = {0.f, 0.f}, pre_n[2] = {0.f, 0.f};
        bool have_pre = false;
        auto load_magnitudes = [&](long long unit, float (&dst)[2]) {      // of the unit's first tile
            const long long chunk0 = G > 1 ? unit * span / st.chunk : unit;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int e = lane + 32 * q;
                dst[q] = e < W * G ? st.scales_w[(long long)(e / G) * st.n_chunks + chunk0 + (e % G)] : 0.0f;
            }
        };
        for (long long k = 0;; ++k) {
            long long unit = 0;
            int go = 0;
            if (lane == 0) {
                go = (p.ok && p.publish(k, cur, &unit)) ? 1 : 0;
                if (!go && p.ok) mbar_arrive(p.full_barrier());          // the end mark needs the barrier's second arrival too
            }
            go = __shfl_sync(0xffffffffu, go, 0);
            unit = __shfl_sync(0xffffffffu, unit, 0);
            if (!go) break;
            // next unit's magnitudes and the number of the unit after it: both in flight during this unit's tiles
            const long long next_taken = __shfl_sync(0xffffffffu, nxt, 0);
            const bool next_valid = next_taken < a.n_full_chunks;
            if (ahead && next_valid) load_magnitudes(a.first_chunk + next_taken, pre_n);
            cur = nxt;
            if (lane == 0) nxt = p.take();
            const long long u0 = unit * span;
            int alive = 1;
            for (int t = 0; t < 2 * TILES && alive; ++t) {
                int stage = 0;
                if (lane == 0) {
                    alive = p.stage_free() ? 1 : 0;
                    stage = p.s;
                }
                alive = __shfl_sync(0xffffffffu, alive, 0);
                stage = __shfl_sync(0xffffffffu, stage, 0);
                if (!alive) break;
                unsigned char *stage_ptr = ring + (size_t)stage * lay.stage_bytes;
                if (t < TILES) {            // first pass over the unit: server error, packed words, magnitudes
                    const long long off = u0 + (long long)t * kTile;
                    if (lane == 0) {
                        const uint32_t full = p.full_barrier(), dst = p.stage_addr();
                        mbar_arrive_expect_tx(full, kTileBytes + W * (kTile / 8));
                        bulk_load(dst, st.ds + off, kTileBytes, full);
                        for (int i = 0; i < W; ++i)
                            bulk_load(dst + lay.words_off + i * (kTile / 8), st.words_w + (long long)i * st.words_stride + (off >> 5),
                                      kTile / 8, full);
                    }
                    if (G > 1 || t == 0) {
                        float *dst_scales = reinterpret_cast<float *>(stage_ptr + lay.stage_scales_off);
                        if (have_pre && t == 0) {
#pragma unroll
                            for (int q = 0; q < 2; ++q)
                                if (lane + 32 * q < W * G) dst_scales[lane + 32 * q] = pre_c[q];
                        } else {
                            const long long chunk0 = G > 1 ? off / st.chunk : unit;
                            for (int e = lane; e < W * G; e += 32)
                                dst_scales[e] = st.scales_w[(long long)(e / G) * st.n_chunks + chunk0 + (e % G)];
                        }
                    }
                } else {                    // second pass: v and x_sync
                    const long long off = u0 + (long long)(t - TILES) * kTile;
                    if (lane == 0) {
                        const uint32_t full = p.full_barrier(), dst = p.stage_addr();
                        mbar_arrive_expect_tx(full, 2 * kTileBytes);
                        bulk_load(dst, st.v + off, kTileBytes, full);
                        bulk_load(dst + kTileBytes, st.xs + off, kTileBytes, full);
                    }
                }
                __syncwarp();               // the lanes' magnitudes are in the stage
                if (lane == 0) {
                    mbar_arrive(p.full_barrier());
                    p.advance();
                    alive = p.ok ? 1 : 0;
                }
                alive = __shfl_sync(0xffffffffu, alive, 0);
            }
            if (!alive) break;
            pre_c[0] = pre_n[0];
            pre_c[1] = pre_n[1];
            have_pre = ahead && next_valid;
        }
        if (lane == 0) p.finish();
        return;
    }

    if (warp == kConsumerWarps + 1) {
        // ------------------------------ store-issuing warp ------------------------------
        // Lane l sends the rows of workers l, l + 32, ...; one more lane sends x_sync.  A single
        // lane issuing all 3 W + 1 copies of a tile is held back by the copy engine's queue to
        // less than the SM's share of the bandwidth.
        for (long long q = 0;; ++q) {
            const int b = (int)(q % kStoreBufs);
            int go = 0;
            long long j0 = -1;
            if (lane == 0) {
                go = mbar_wait(smem_addr(&sh->staged[b]), (uint32_t)((q / kStoreBufs) & 1), abort_flag, a.error_flag, a.wait_limit_ns) ? 1 : 0;
                if (go) j0 = sh->dst[b];
            }
            go = __shfl_sync(0xffffffffu, go, 0);
            j0 = __shfl_sync(0xffffffffu, j0, 0);
            if (!go || j0 < 0) break;
            const float *x_s = staging + (size_t)b * 2 * kTile, *m_s = x_s + kTile;
            for (int i = lane; i < W; i += 32) {
                const long long row = (long long)i * st.n_pad + j0;
                bulk_store(st.m + row, m_s, kTileBytes);        // momentum approximation
                bulk_store(st.x + row, x_s, kTileBytes);        // model sync
                bulk_store(st.u + row, zero_s, kTileBytes);     // buffer reset
            }
            if (lane == W % 32) bulk_store(st.xs + j0, x_s, kTileBytes);
            bulk_store_commit();
            bulk_store_wait_read<1>();                          // this lane's copies of every tile but this one have left shared memory
            __syncwarp();
            if (lane == 0 && q > 0) mbar_arrive(smem_addr(&sh->drained[(q - 1) % kStoreBufs]));
        }
        bulk_store_wait_read<0>();
        return;
    }

    // -------------------------------------- consumers --------------------------------------
    int s = 0;
    uint32_t phase = 0;
    int flip = 0;
    long long staged_tiles = 0;
    const int pos = 4 * tid;
    const int word_in_tile = pos >> 5;
    const int shift = (lane & 7) * 4;
    const bool group_leader = (lane & 7) == 0;
    float *my_scales = scales_s + warp * W;
    const int my_chunk_in_tile = G > 1 ? warp / WPC : 0;
    st4(zero_s + pos, make_float4(0.f, 0.f, 0.f, 0.f));

    auto stage_buffer = [&](long long j0, const float xo[4], const bool b[4], float m_pos) {
        const int buf = (int)(staged_tiles % kStoreBufs);
        mbar_wait(smem_addr(&sh->drained[buf]), (uint32_t)(((staged_tiles / kStoreBufs) & 1) ^ 1), abort_flag, a.error_flag, a.wait_limit_ns);
        float *x_s = staging + (size_t)buf * 2 * kTile, *m_s = x_s + kTile;
        st4(x_s + pos, make_float4(xo[0], xo[1], xo[2], xo[3]));
        st4(m_s + pos, make_float4(b[0] ? m_pos : -m_pos, b[1] ? m_pos : -m_pos, b[2] ? m_pos : -m_pos, b[3] ? m_pos : -m_pos));
        store_fence();
        if (tid == 0) sh->dst[buf] = j0;
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_addr(&sh->staged[buf]));
        ++staged_tiles;
    };

    for (long long k = 0;; ++k) {
        const bool gave_up = !mbar_wait(smem_addr(&sh->ring.full[s]), phase, abort_flag, a.error_flag, a.wait_limit_ns);
        if (consumer_any(gave_up)) break;
        const long long unit = sh->ring.chunk_queue[k % (kMaxStages + 2)];
        if (unit < 0) break;
        const long long u0 = unit * span;

        // ---- first pass: mean of the compressed buffers + server error (Algorithm 3, server side) ----
        float av[TILES][4];
        double l1 = 0.0;
#pragma unroll
        for (int t = 0; t < TILES; ++t) {
            const bool ready = mbar_wait(smem_addr(&sh->ring.full[s]), phase, abort_flag, a.error_flag, a.wait_limit_ns);
            const unsigned char *stage = ring + (size_t)s * lay.stage_bytes;
            const float4 d4 = ready ? ld4(reinterpret_cast<const float *>(stage) + pos) : make_float4(0.f, 0.f, 0.f, 0.f);
            if (G > 1 || t == 0) {
                const float *src = reinterpret_cast<const float *>(stage + lay.stage_scales_off);
                for (int i = lane; i < W; i += 32) my_scales[i] = ready ? src[i * G + my_chunk_in_tile] : 0.0f;
                __syncwarp();
            }
            const uint32_t *words = reinterpret_cast<const uint32_t *>(stage + lay.words_off);
            double A[4] = {0.0, 0.0, 0.0, 0.0};
            for (int i = 0; i < W; ++i) {   // worker order
                const uint32_t nib = (ready ? words[i * (kTile / 32) + word_in_tile] : 0u) >> shift;
                const double sc = (double)my_scales[i];
#pragma unroll
                for (int q = 0; q < 4; ++q) A[q] += ((nib >> q) & 1u) ? sc : -sc;
            }
            // the sums were formed from the stage's words and magnitudes: they stand for those loads
            release_stage(&sh->ring, s, dep_bits(d4) ^ (uint32_t)__double_as_longlong(A[0]) ^ (uint32_t)__double_as_longlong(A[3]));
            if (++s == R) { s = 0; phase ^= 1u; }
            const float dd[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                av[t][q] = server_input(A[q], W, dd[q]);
                l1 += fabs((double)av[t][q]);
            }
        }
        const float scale = chunk_scale(consumer_group_sum<WPC>(l1, &sh->ring, flip), st.chunk);
        const float m_pos = f_div(scale, a.gamma_sum);      // momentum approximation: m = +-scale / sum(gamma)

        // ---- second pass: compress again, server error, the post-sync rows ----
#pragma unroll
        for (int t = 0; t < TILES; ++t) {
            const bool ready = mbar_wait(smem_addr(&sh->ring.full[s]), phase, abort_flag, a.error_flag, a.wait_limit_ns);
            const float *stage = reinterpret_cast<const float *>(ring + (size_t)s * lay.stage_bytes);
            const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
            const float4 v4 = ready ? ld4(stage + pos) : zero4, xs4 = ready ? ld4(stage + kTile + pos) : zero4;
            release_stage(&sh->ring, s, dep_bits(v4, xs4));
            if (++s == R) { s = 0; phase ^= 1u; }
            const float vv[4] = {v4.x, v4.y, v4.z, v4.w}, xs[4] = {xs4.x, xs4.y, xs4.z, xs4.w};
            bool b[4];
            float e[4], xo[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                b[q] = av[t][q] >= 0.0f;
                const float hat = b[q] ? scale : -scale;
                e[q] = f_sub(av[t][q], hat);
                xo[q] = f_sub(xs[q], f_div(hat, denom(a.c, vv[q])));           // model sync
            }
            const long long j0 = u0 + (long long)t * kTile;
            const uint32_t word = pack_group(b);
            if (group_leader) st.words_s[(j0 >> 5) + word_in_tile] = word;
            st4_stream(st.ds + j0 + pos, make_float4(e[0], e[1], e[2], e[3]));
            stage_buffer(j0, xo, b, m_pos);
        }
        if (G == 1) {
            if (tid == 0) st.scales_s[unit] = scale;
        } else if (lane == 0 && warp % WPC == 0) {
            st.scales_s[unit * G + my_chunk_in_tile] = scale;
        }
        __syncwarp();   // the next unit overwrites this warp's my_scales
    }
    // tell the store-issuing warp that nothing more comes
    {
        const int buf = (int)(staged_tiles % kStoreBufs);
        mbar_wait(smem_addr(&sh->drained[buf]), (uint32_t)(((staged_tiles / kStoreBufs) & 1) ^ 1), abort_flag, a.error_flag, a.wait_limit_ns);
        if (tid == 0) sh->dst[buf] = -1;
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_addr(&sh->staged[buf]));
    }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
// tiles per unit and chunks per tile for a chunk size the ring kernels take (false: they do not)
static bool unit_shape(int chunk, int *tiles, int *chunks_per_tile)
{
    *tiles = 1;
    *chunks_per_tile = 1;
    if (chunk >= kTile) {
        if (chunk % kTile != 0) return false;
        *tiles = chunk / kTile;
        return *tiles == 1 || *tiles == 2 || *tiles == 4 || *tiles == 8;
    }
    if (chunk < 128 || kTile % chunk != 0) return false;
    *chunks_per_tile = kTile / chunk;      // 2, 4, 8 or 16: whole warps per chunk
    return true;
}

// Ring depth for the server kernel (0: it does not apply to this shape) and the number of units.
int reduce_pipeline_stages(const StateView &st, long long *n_units)
{
    int tiles, g;
    if (!unit_shape(st.chunk, &tiles, &g)) return 0;
    *n_units = st.n / ((long long)tiles * kTile);
    if (*n_units < 1) return 0;
    const ReduceLayout lay = reduce_layout(st.W, g);
    const int budget = 227 * 1024;
    int stages = (budget - lay.ring_off) / lay.stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    return stages >= 4 ? stages : 0;
}

template <int TILES, int G>
static cudaError_t launch_reduce_pipe(const PipeArgs &a, int grid, size_t smem, cudaStream_t s)
{
    auto kern = reduce_pipelined_kernel<TILES, G>;
    static SmemLimitOnce once;
    const cudaError_t e = once.ensure(kern, 227 * 1024);
    if (e != cudaSuccess) return e;
    kern<<<grid, kRingThreads, smem, s>>>(a);
    return cudaGetLastError();
}

static PipeArgs two_call_args(const StateView &st, const Consts &c, float gamma_sum, long long work_items, int stages,
                              ErrorWords error_flag, unsigned long long *sched, unsigned long long wait_limit_ns,
                              long long test_stop_after_tiles)
{
    PipeArgs a{};
    a.st = st; a.c = c; a.gamma = 0.f; a.gamma_sum = gamma_sum;
    a.first_chunk = 0;
    a.n_full_chunks = work_items;
    a.stages = stages;
    a.error_flag = error_flag;
    a.sched = sched;
    a.grad_fmt = kGradAligned;
    a.wait_limit_ns = wait_limit_ns;
    a.test_stop_after_tiles = test_stop_after_tiles;
    return a;
}

#define ZOA_UNIT_DISPATCH(CALL)                          \
    switch (tiles * 100 + g) {                           \
    case 101: return CALL(1, 1);                         \
    case 201: return CALL(2, 1);                         \
    case 401: return CALL(4, 1);                         \
    case 801: return CALL(8, 1);                         \
    case 102: return CALL(1, 2);                         \
    case 104: return CALL(1, 4);                         \
    case 108: return CALL(1, 8);                         \
    case 116: return CALL(1, 16);                        \
    default: return cudaErrorInvalidValue;               \
    }

// Server side for the first n_units units (the caller runs the remaining chunks through reduce_kernel).
cudaError_t launch_reduce_pipelined(const StateView &st, const Consts &c, float gamma_sum, long long n_units,
                                    int stages, int sm_count, ErrorWords error_flag, unsigned long long *sched,
                                    unsigned long long wait_limit_ns, long long test_stop_after_tiles, cudaStream_t s)
{
    int tiles, g;
    if (!unit_shape(st.chunk, &tiles, &g)) return cudaErrorInvalidValue;
    const PipeArgs a = two_call_args(st, c, gamma_sum, n_units, stages, error_flag, sched, wait_limit_ns, test_stop_after_tiles);
    const ReduceLayout lay = reduce_layout(st.W, g);
    const int grid = (int)(n_units < sm_count ? n_units : sm_count);
    const size_t smem = (size_t)lay.ring_off + (size_t)stages * lay.stage_bytes;
#define ZOA_CALL(T, GG) launch_reduce_pipe<T, GG>(a, grid, smem, s)
    ZOA_UNIT_DISPATCH(ZOA_CALL)
#undef ZOA_CALL
}

}  // namespace zoa
