// step_sync_pipelined_kernel: the fused sync step (a whole sync iteration of Algorithm 1 with
// Algorithm 3 inside) as a persistent, warp-specialised kernel for sm_100a.
//
// One block per SM takes chunks from a global counter (SMs do not all get the same
// share of DRAM bandwidth, so a fixed split would leave the fast ones idle at the
// end).  A producer warp streams
// the inputs of each (chunk, worker) - tiles of 2048 coordinates of g, m, u and
// the worker error - through a ring of shared-memory stages with 1-D bulk
// asynchronous copies (cp.async.bulk ... mbarrier::complete_tx), several stages
// ahead of the 512 consumer threads, so DRAM reads stay in flight while the
// consumers sit in the block-wide l1 sums.  After the W workers of a chunk come
// tiles of (server error, v, x_sync) for the server part.  Consumers keep a
// chunk's z in registers (thread t owns coordinates 4t..4t+3 of every tile), so
// shared memory holds only the ring, the packed bits and the magnitudes.
//
// Every wait on an mbarrier is bounded: after the handle's limit (2 s by default) a thread gives
// up, raises the block's abort flag and the handle's device error flag, the
// block stops issuing copies, waits (bounded) for those in flight and leaves.
#include "zoa_internal.h"
#include "zoa_ring.cuh"

namespace zoa {

// A work unit is TILES tiles of 2048 coordinates: one chunk of 2048, 4096 or 8192 coordinates (G = 1), or
// one tile holding G = 2048 / chunk whole chunks of 128 ... 1024 coordinates (TILES = 1), in which
// case a chunk's l1 norm is the sum over the 16 / G consumer warps that own it.
template <int TILES, int G, bool DO_VAR>
__global__ void __launch_bounds__(kThreads, 1) step_sync_pipelined_kernel(const __grid_constant__ PipeArgs a)
{
    constexpr int WPC = kConsumerWarps / G;          // consumer warps per chunk
    constexpr long long kSpan = (long long)TILES * kTile;
    // The server needs a unit's server errors before the l1 sum and its v and x_sync after it: the
    // unit's (at most four) server tiles stay in the ring over the sum.
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    PipeShared *sh = reinterpret_cast<PipeShared *>(smem_raw);
    const StateView &st = a.st;
    const int W = st.W;
    constexpr int words_per_chunk = (int)(kSpan >> 5);                                  // words of a unit
    uint32_t *bits_s = reinterpret_cast<uint32_t *>(smem_raw + 1024);                 // [W][words_per_chunk]
    float *scales_s = reinterpret_cast<float *>(bits_s + W * words_per_chunk);         // [kConsumerWarps][W]
    // On a T_v step with four tiles the binary64 gradient sums of the last two tiles live in shared
    // memory ([tile][k][thread], one column per thread): sixteen of them in registers make the kernel spill.
    constexpr int G_SHARED_TILES = (DO_VAR && TILES == 4) ? 2 : 0;
    constexpr int G_REG_TILES = DO_VAR ? TILES - G_SHARED_TILES : 1;
    const size_t head_bytes = (1024 + (size_t)W * words_per_chunk * 4 + (size_t)kConsumerWarps * W * 4 + 1023) & ~(size_t)1023;
    double *gsum_s = reinterpret_cast<double *>(smem_raw + head_bytes);                 // [G_SHARED_TILES][4][kConsumers]
    unsigned char *ring = smem_raw + head_bytes + (size_t)G_SHARED_TILES * 4 * kConsumers * sizeof(double);
    const int R = a.stages;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int *abort_flag = &sh->abort;

    ring_init(sh, R);

    if (warp == kConsumerWarps) {
        // ------------------------------ producer ------------------------------
        if (lane != 0) return;
        RingProducer p(a, sh, ring, kStageBytes);
        const uint32_t g_elem = (a.grad_fmt & kGradTypeMask) == kGradF32 ? 4u : 2u;
        long long chunk;
        for (long long k = 0; p.ok && p.next_chunk(k, &chunk); ++k) {
            const long long c0 = chunk * kSpan;             // `chunk` numbers the units here
            for (int i = 0; p.ok && i <= W; ++i) {          // i == W: the server's tiles
                for (int t = 0; t < TILES && p.stage_free(); ++t) {
                    const uint32_t full = p.full_barrier(), dst = p.stage_addr();
                    const long long off = c0 + (long long)t * kTile;
                    if (i < W) {
                        const long long row = (long long)i * st.n_pad + off;
                        mbar_arrive_expect_tx(full, 3 * kTileBytes + kTile * g_elem);
                        bulk_load(dst, reinterpret_cast<const char *>(a.g.p[i]) + off * g_elem, kTile * g_elem, full);
                        bulk_load(dst + kTileBytes, st.m + row, kTileBytes, full);
                        bulk_load(dst + 2 * kTileBytes, st.u + row, kTileBytes, full);
                        bulk_load(dst + 3 * kTileBytes, st.dw + row, kTileBytes, full);
                    } else {
                        mbar_arrive_expect_tx(full, 3 * kTileBytes);
                        bulk_load(dst, st.ds + off, kTileBytes, full);
                        bulk_load(dst + kTileBytes, st.v + off, kTileBytes, full);
                        bulk_load(dst + 2 * kTileBytes, st.xs + off, kTileBytes, full);
                    }
                    p.advance();
                }
            }
        }
        p.finish();
        return;
    }

    // -------------------------------- consumers --------------------------------
    int s = 0;
    uint32_t phase = 0;
    int flip = 0;
    const int pos = 4 * tid;                         // this thread's coordinates inside every tile
    const int word_in_tile = pos >> 5;               // = warp * 4 + (lane >> 3)
    const bool group_leader = (lane & 7) == 0;
    float *my_scales = scales_s + warp * W;

    // The post-sync updates of the previous chunk, carried in registers: its 3 W tile stores are
    // spread over the worker iterations of the next chunk (one worker's m, x, u after
    // each worker's compression) instead of leaving in one burst, so that the block's
    // stores and its ring's loads stay evenly mixed.  m is +-m_pos by the server's bit.
    // (Four tiles of x are what fits: 17 warps leave 96 registers per thread, since one SM
    // sub-partition hosts five of them.)
    float x_prev[TILES][4];
    uint32_t bits_prev = 0;
    float m_pos_prev = 0.0f;
    long long c0_prev = -1;
    auto store_prev_worker = [&](int i) {
        const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int t = 0; t < TILES; ++t) {
            const long long row = (long long)i * st.n_pad + c0_prev + t * kTile + pos;
            const uint32_t nib = bits_prev >> (4 * t);
            st4_stream(st.m + row, make_float4((nib & 1u) ? m_pos_prev : -m_pos_prev, (nib & 2u) ? m_pos_prev : -m_pos_prev,
                                               (nib & 4u) ? m_pos_prev : -m_pos_prev, (nib & 8u) ? m_pos_prev : -m_pos_prev));
            st4_stream(st.x + row, make_float4(x_prev[t][0], x_prev[t][1], x_prev[t][2], x_prev[t][3]));
            st4_stream(st.u + row, zero);                                      // buffer reset
        }
    };

    for (long long k = 0;; ++k) {
        // The first tile's barrier also publishes the chunk id (or the end mark).  Leaving the
        // loop must be unanimous (the block sums below count on all 512 consumers), so a
        // wait that ran out is put to the vote.
        const bool gave_up = !mbar_wait(smem_addr(&sh->full[s]), phase, abort_flag, a.error_flag, a.wait_limit_ns);
        if (consumer_any(gave_up)) break;
        const long long chunk = sh->chunk_queue[k % (kMaxStages + 2)];   // the unit
        if (chunk < 0) break;
        const long long c0 = chunk * kSpan;
        const long long scale_idx = G == 1 ? chunk : chunk * G + warp / WPC;       // this thread's chunk
        const bool scale_writer = G == 1 ? tid == 0 : (lane == 0 && warp % WPC == 0);
        double Gs[G_REG_TILES][4];
        if (DO_VAR) {
#pragma unroll
            for (int t = 0; t < G_REG_TILES; ++t) { Gs[t][0] = Gs[t][1] = Gs[t][2] = Gs[t][3] = 0.0; }
#pragma unroll
            for (int q = 0; q < G_SHARED_TILES * 4; ++q) gsum_s[q * kConsumers + tid] = 0.0;
        }
        for (int i = 0; i < W; ++i) {
            float z[TILES][4];
            double l1 = 0.0;
#pragma unroll
            for (int t = 0; t < TILES; ++t) {
                const bool ready = mbar_wait(smem_addr(&sh->full[s]), phase, abort_flag, a.error_flag, a.wait_limit_ns);
                const float *stage = reinterpret_cast<const float *>(ring + (size_t)s * kStageBytes);
                float4 g4 = make_float4(0.f, 0.f, 0.f, 0.f), m4 = g4, u4 = g4, e4 = g4;
                if (ready) {
                    if ((a.grad_fmt & kGradTypeMask) == kGradF32)
                        g4 = ld4(stage + pos);
                    else   // 16-bit gradients fill the first half of the slot
                        g4 = grad16x4_to_float4(*reinterpret_cast<const uint2 *>(reinterpret_cast<const unsigned short *>(stage) + pos), a.grad_fmt);
                    m4 = ld4(stage + kTile + pos);
                    u4 = ld4(stage + 2 * kTile + pos);
                    e4 = ld4(stage + 3 * kTile + pos);
                }
                release_stage(sh, s, dep_bits(g4, m4, u4, e4));
                if (++s == R) { s = 0; phase ^= 1u; }
                const float gg[4] = {g4.x, g4.y, g4.z, g4.w}, mm[4] = {m4.x, m4.y, m4.z, m4.w};
                const float uu[4] = {u4.x, u4.y, u4.z, u4.w}, ee[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float step = f_mul(a.gamma, momentum(a.c, mm[k], gg[k]));   // momentum update, buffer update
                    z[t][k] = f_add(f_add(uu[k], step), ee[k]);                       // u_{t+1/2} + delta
                    l1 += fabs((double)z[t][k]);
                    if (DO_VAR) {
                        if (t < G_REG_TILES) Gs[t][k] += (double)gg[k];
                        else gsum_s[((t - G_REG_TILES) * 4 + k) * kConsumers + tid] += (double)gg[k];
                    }
                }
            }
            const float scale = chunk_scale(consumer_group_sum<WPC>(l1, sh, flip), st.chunk);
            const long long row = (long long)i * st.n_pad + c0;
#pragma unroll
            for (int t = 0; t < TILES; ++t) {
                bool b[4];
                float e[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    b[k] = z[t][k] >= 0.0f;
                    e[k] = f_sub(z[t][k], b[k] ? scale : -scale);
                }
                st4_stream(st.dw + row + t * kTile + pos, make_float4(e[0], e[1], e[2], e[3]));
                const uint32_t word = pack_group(b);
                if (group_leader) {
                    bits_s[i * words_per_chunk + t * (kTile / 32) + word_in_tile] = word;
                    st.words_w[(long long)i * st.words_stride + ((c0 + t * kTile) >> 5) + word_in_tile] = word;
                }
            }
            if (lane == 0) my_scales[i] = scale;
            if (scale_writer) st.scales_w[(long long)i * st.n_chunks + scale_idx] = scale;
            if (c0_prev >= 0) store_prev_worker(i);
        }
        __syncwarp();   // bits_s and my_scales were written by lanes of this warp

        // ---- server: mean of the compressed buffers + server error, compress again ----
        float av[TILES][4];
        int srv_stage[TILES];
        double l1 = 0.0;
#pragma unroll
        for (int t = 0; t < TILES; ++t) {
            const bool ready = mbar_wait(smem_addr(&sh->full[s]), phase, abort_flag, a.error_flag, a.wait_limit_ns);
            srv_stage[t] = s;
            const float *stage = reinterpret_cast<const float *>(ring + (size_t)s * kStageBytes);
            const float4 d4 = ready ? ld4(stage + pos) : make_float4(0.f, 0.f, 0.f, 0.f);
            if (++s == R) { s = 0; phase ^= 1u; }
            const float dd[4] = {d4.x, d4.y, d4.z, d4.w};
            double A[4] = {0.0, 0.0, 0.0, 0.0};
            const int shift = (lane & 7) * 4;
            for (int i = 0; i < W; ++i) {   // worker order
                const uint32_t nib = bits_s[i * words_per_chunk + t * (kTile / 32) + word_in_tile] >> shift;
                const double sc = (double)my_scales[i];
#pragma unroll
                for (int k = 0; k < 4; ++k) A[k] += ((nib >> k) & 1u) ? sc : -sc;
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                av[t][k] = server_input(A[k], W, dd[k]);
                l1 += fabs((double)av[t][k]);
            }
        }
        const float scale = chunk_scale(consumer_group_sum<WPC>(l1, sh, flip), st.chunk);
#pragma unroll
        for (int t = 0; t < TILES; ++t) {
            const float *stage = reinterpret_cast<const float *>(ring + (size_t)srv_stage[t] * kStageBytes);
            const float4 v4 = ld4(stage + kTile + pos), xs4 = ld4(stage + 2 * kTile + pos);
            release_stage(sh, srv_stage[t], dep_bits(v4, xs4));
            const float vv[4] = {v4.x, v4.y, v4.z, v4.w}, xs[4] = {xs4.x, xs4.y, xs4.z, xs4.w};
            bool b[4];
            float e[4], xo[4];
            if (t == 0) bits_prev = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                b[k] = av[t][k] >= 0.0f;
                const float hat = b[k] ? scale : -scale;
                e[k] = f_sub(av[t][k], hat);
                xo[k] = f_sub(xs[k], f_div(hat, denom(a.c, vv[k])));           // model sync
                x_prev[t][k] = xo[k];
                bits_prev |= (b[k] ? 1u : 0u) << (4 * t + k);
            }
            const long long j = c0 + t * kTile + pos;
            const uint32_t word = pack_group(b);
            if (group_leader) st.words_s[((c0 + t * kTile) >> 5) + word_in_tile] = word;
            st4_stream(st.ds + j, make_float4(e[0], e[1], e[2], e[3]));
            st4_stream(st.xs + j, make_float4(xo[0], xo[1], xo[2], xo[3]));
            if (DO_VAR) {
                float vo[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const double g_sum = t < G_REG_TILES ? Gs[t < G_REG_TILES ? t : 0][k] : gsum_s[((t - G_REG_TILES) * 4 + k) * kConsumers + tid];
                    vo[k] = variance(a.c, vv[k], mean_round(g_sum, W));   // variance update
                }
                st4_stream(st.v_next + j, make_float4(vo[0], vo[1], vo[2], vo[3]));
            }
        }
        m_pos_prev = f_div(scale, a.gamma_sum);     // momentum approximation: m = +-scale / sum(gamma); -(s/G) == (-s)/G exactly
        c0_prev = c0;
        if (scale_writer) st.scales_s[scale_idx] = scale;
        __syncwarp();   // the next chunk overwrites bits_s / my_scales of this warp
    }
    if (c0_prev >= 0)
        for (int i = 0; i < W; ++i) store_prev_worker(i);   // the block's last chunk
}

// ---------------------------------------------------------------------------
// Algorithm 2, compressed step, in the same style: per chunk the ring carries W x TILES
// tiles of (g_i, delta_i), TILES tiles of (delta_bar, v), then W x TILES tiles of (m_i, x_i).
// The received gradient g_bar and the denominators sqrt(v + eps) stay in registers
// between the server part and the update of the W workers' momentum and model.
// ---------------------------------------------------------------------------
constexpr int kStage2Bytes = 2 * kTileBytes;

template <int TILES>
__global__ void __launch_bounds__(kThreads, 1) alg2_pipelined_kernel(const __grid_constant__ PipeArgs a)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    PipeShared *sh = reinterpret_cast<PipeShared *>(smem_raw);
    const StateView &st = a.st;
    const int W = st.W;
    const int words_per_chunk = st.chunk >> 5;
    uint32_t *bits_s = reinterpret_cast<uint32_t *>(smem_raw + 1024);
    float *scales_s = reinterpret_cast<float *>(bits_s + W * words_per_chunk);
    unsigned char *ring = smem_raw + ((1024 + (size_t)W * words_per_chunk * 4 + (size_t)kConsumerWarps * W * 4 + 1023) & ~(size_t)1023);
    const int R = a.stages;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int *abort_flag = &sh->abort;

    ring_init(sh, R);

    if (warp == kConsumerWarps) {
        // ------------------------------ producer ------------------------------
        if (lane != 0) return;
        RingProducer p(a, sh, ring, kStage2Bytes);
        const uint32_t g_elem = (a.grad_fmt & kGradTypeMask) == kGradF32 ? 4u : 2u;
        long long chunk;
        for (long long k = 0; p.ok && p.next_chunk(k, &chunk); ++k) {
            const long long c0 = chunk * st.chunk;
            for (int i = 0; p.ok && i <= 2 * W; ++i) {      // i < W: (g, delta); i == W: (delta_bar, v); i > W: (m, x)
                for (int t = 0; t < TILES && p.stage_free(); ++t) {
                    const uint32_t full = p.full_barrier(), dst = p.stage_addr();
                    const long long off = c0 + (long long)t * kTile;
                    if (i < W) {
                        mbar_arrive_expect_tx(full, kTileBytes + kTile * g_elem);
                        bulk_load(dst, reinterpret_cast<const char *>(a.g.p[i]) + off * g_elem, kTile * g_elem, full);
                        bulk_load(dst + kTileBytes, st.dw + (long long)i * st.n_pad + off, kTileBytes, full);
                    } else if (i == W) {
                        mbar_arrive_expect_tx(full, 2 * kTileBytes);
                        bulk_load(dst, st.ds + off, kTileBytes, full);
                        bulk_load(dst + kTileBytes, st.v + off, kTileBytes, full);
                    } else {
                        const long long row = (long long)(i - W - 1) * st.n_pad + off;
                        mbar_arrive_expect_tx(full, 2 * kTileBytes);
                        bulk_load(dst, st.m + row, kTileBytes, full);
                        bulk_load(dst + kTileBytes, st.x + row, kTileBytes, full);
                    }
                    p.advance();
                }
            }
        }
        p.finish();
        return;
    }

    // -------------------------------- consumers --------------------------------
    int s = 0;
    uint32_t phase = 0;
    int flip = 0;
    const int pos = 4 * tid;
    const int word_in_tile = pos >> 5;
    const bool group_leader = (lane & 7) == 0;
    float *my_scales = scales_s + warp * W;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);

    // Waits for the next stage, hands back its two slots, and releases it once the warp has read them.
    auto next_tile = [&](float4 &slot0, float4 &slot1, bool slot0_is_grad) {
        const bool ready = mbar_wait(smem_addr(&sh->full[s]), phase, abort_flag, a.error_flag, a.wait_limit_ns);
        const float *stage = reinterpret_cast<const float *>(ring + (size_t)s * kStage2Bytes);
        slot0 = zero4;
        slot1 = zero4;
        if (ready) {
            if (slot0_is_grad && (a.grad_fmt & kGradTypeMask) != kGradF32)
                slot0 = grad16x4_to_float4(*reinterpret_cast<const uint2 *>(reinterpret_cast<const unsigned short *>(stage) + pos), a.grad_fmt);
            else
                slot0 = ld4(stage + pos);
            slot1 = ld4(stage + kTile + pos);
        }
        release_stage(sh, s, dep_bits(slot0, slot1));
        if (++s == R) { s = 0; phase ^= 1u; }
    };

    for (long long k = 0;; ++k) {
        const bool gave_up = !mbar_wait(smem_addr(&sh->full[s]), phase, abort_flag, a.error_flag, a.wait_limit_ns);
        if (consumer_any(gave_up)) break;
        const long long chunk = sh->chunk_queue[k % (kMaxStages + 2)];
        if (chunk < 0) break;
        const long long c0 = chunk * st.chunk;

        // ---- workers: compress g + delta (Algorithm 3, worker side) ----
        for (int i = 0; i < W; ++i) {
            float z[TILES][4];
            double l1 = 0.0;
#pragma unroll
            for (int t = 0; t < TILES; ++t) {
                float4 g4, e4;
                next_tile(g4, e4, true);
                z[t][0] = f_add(g4.x, e4.x); z[t][1] = f_add(g4.y, e4.y);
                z[t][2] = f_add(g4.z, e4.z); z[t][3] = f_add(g4.w, e4.w);
                l1 += fabs((double)z[t][0]) + fabs((double)z[t][1]) + fabs((double)z[t][2]) + fabs((double)z[t][3]);
            }
            const float scale = chunk_scale(consumer_sum(l1, sh, flip), st.chunk);
            const long long row = (long long)i * st.n_pad + c0;
#pragma unroll
            for (int t = 0; t < TILES; ++t) {
                bool b[4];
                float e[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    b[q] = z[t][q] >= 0.0f;
                    e[q] = f_sub(z[t][q], b[q] ? scale : -scale);
                }
                st4_stream(st.dw + row + t * kTile + pos, make_float4(e[0], e[1], e[2], e[3]));
                const uint32_t word = pack_group(b);
                if (group_leader) {
                    bits_s[i * words_per_chunk + t * (kTile / 32) + word_in_tile] = word;
                    st.words_w[(long long)i * st.words_stride + ((c0 + t * kTile) >> 5) + word_in_tile] = word;
                }
            }
            if (lane == 0) my_scales[i] = scale;
            if (tid == 0) st.scales_w[(long long)i * st.n_chunks + chunk] = scale;
        }
        __syncwarp();

        // ---- server: mean + server error, compress again; keep g_bar and the denominators ----
        float gbar[TILES][4], dn[TILES][4];
        double l1 = 0.0;
#pragma unroll
        for (int t = 0; t < TILES; ++t) {
            float4 d4, v4;
            next_tile(d4, v4, false);
            const float dd[4] = {d4.x, d4.y, d4.z, d4.w}, vv[4] = {v4.x, v4.y, v4.z, v4.w};
            double A[4] = {0.0, 0.0, 0.0, 0.0};
            const int shift = (lane & 7) * 4;
            for (int i = 0; i < W; ++i) {
                const uint32_t nib = bits_s[i * words_per_chunk + t * (kTile / 32) + word_in_tile] >> shift;
                const double sc = (double)my_scales[i];
#pragma unroll
                for (int q = 0; q < 4; ++q) A[q] += ((nib >> q) & 1u) ? sc : -sc;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                gbar[t][q] = server_input(A[q], W, dd[q]);       // the server's input for now
                dn[t][q] = denom(a.c, vv[q]);
                l1 += fabs((double)gbar[t][q]);
            }
        }
        const float scale = chunk_scale(consumer_sum(l1, sh, flip), st.chunk);
#pragma unroll
        for (int t = 0; t < TILES; ++t) {
            bool b[4];
            float e[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                b[q] = gbar[t][q] >= 0.0f;
                const float hat = b[q] ? scale : -scale;
                e[q] = f_sub(gbar[t][q], hat);
                gbar[t][q] = hat;                                // what every worker receives from the Compressed-AllReduce
            }
            const uint32_t word = pack_group(b);
            if (group_leader) st.words_s[((c0 + t * kTile) >> 5) + word_in_tile] = word;
            st4_stream(st.ds + c0 + t * kTile + pos, make_float4(e[0], e[1], e[2], e[3]));
        }
        if (tid == 0) st.scales_s[chunk] = scale;

        // ---- every worker: momentum update and model update of Algorithm 2 ----
        for (int i = 0; i < W; ++i) {
#pragma unroll
            for (int t = 0; t < TILES; ++t) {
                float4 m4, x4;
                next_tile(m4, x4, false);
                const float mm[4] = {m4.x, m4.y, m4.z, m4.w}, xx[4] = {x4.x, x4.y, x4.z, x4.w};
                float mo[4], xo[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    mo[q] = momentum(a.c, mm[q], gbar[t][q]);
                    xo[q] = f_sub(xx[q], f_div(f_mul(a.gamma, mo[q]), dn[t][q]));
                }
                const long long row = (long long)i * st.n_pad + c0 + t * kTile + pos;
                st4_stream(st.m + row, make_float4(mo[0], mo[1], mo[2], mo[3]));
                st4_stream(st.x + row, make_float4(xo[0], xo[1], xo[2], xo[3]));
            }
        }
        __syncwarp();
    }
}

// ---------------------------------------------------------------------------
// The local step of Algorithm 1 (momentum, model and buffer updates; the variance update on T_v
// steps) in the same style: a unit is one tile of 2048 coordinates of all W workers; the ring
// carries per worker a stage of (g, m, x, u) and, with the first worker, the tile of v.  The
// consumers need no barrier among themselves (the step is elementwise); the ring only keeps
// more loads in flight than resident blocks of an elementwise kernel can.
// ---------------------------------------------------------------------------
constexpr int kLocalStageBytes = 5 * kTileBytes;      // g, m, x, u, v

template <bool DO_VAR>
__global__ void __launch_bounds__(kThreads, 1) local_step_pipelined_kernel(const __grid_constant__ PipeArgs a)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    PipeShared *sh = reinterpret_cast<PipeShared *>(smem_raw);
    const StateView &st = a.st;
    const int W = st.W;
    unsigned char *ring = smem_raw + 1024;
    const int R = a.stages;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int *abort_flag = &sh->abort;

    ring_init(sh, R);

    if (warp == kConsumerWarps) {
        if (lane != 0) return;
        RingProducer p(a, sh, ring, kLocalStageBytes);
        const uint32_t g_elem = (a.grad_fmt & kGradTypeMask) == kGradF32 ? 4u : 2u;
        long long unit;
        for (long long k = 0; p.ok && p.next_chunk(k, &unit); ++k) {
            const long long off = unit * kTile;
            for (int i = 0; i < W && p.stage_free(); ++i) {
                const uint32_t full = p.full_barrier(), dst = p.stage_addr();
                const long long row = (long long)i * st.n_pad + off;
                mbar_arrive_expect_tx(full, 3 * kTileBytes + kTile * g_elem + (i == 0 ? kTileBytes : 0));
                bulk_load(dst, reinterpret_cast<const char *>(a.g.p[i]) + off * g_elem, kTile * g_elem, full);
                bulk_load(dst + kTileBytes, st.m + row, kTileBytes, full);
                bulk_load(dst + 2 * kTileBytes, st.x + row, kTileBytes, full);
                bulk_load(dst + 3 * kTileBytes, st.u + row, kTileBytes, full);
                if (i == 0) bulk_load(dst + 4 * kTileBytes, st.v + off, kTileBytes, full);
                p.advance();
            }
        }
        p.finish();
        return;
    }

    int s = 0;
    uint32_t phase = 0;
    const int pos = 4 * tid;
    for (long long k = 0;; ++k) {
        const bool gave_up = !mbar_wait(smem_addr(&sh->full[s]), phase, abort_flag, a.error_flag, a.wait_limit_ns);
        if (consumer_any(gave_up)) break;
        const long long unit = sh->chunk_queue[k % (kMaxStages + 2)];
        if (unit < 0) break;
        const long long j = unit * kTile + pos;
        float d[4] = {1.f, 1.f, 1.f, 1.f}, vv[4] = {0.f, 0.f, 0.f, 0.f};
        double Gs[4] = {0.0, 0.0, 0.0, 0.0};
        for (int i = 0; i < W; ++i) {
            const bool ready = mbar_wait(smem_addr(&sh->full[s]), phase, abort_flag, a.error_flag, a.wait_limit_ns);
            const float *stage = reinterpret_cast<const float *>(ring + (size_t)s * kLocalStageBytes);
            float4 g4 = make_float4(0.f, 0.f, 0.f, 0.f), m4 = g4, x4 = g4, u4 = g4;
            if (ready) {
                if ((a.grad_fmt & kGradTypeMask) == kGradF32)
                    g4 = ld4(stage + pos);
                else   // 16-bit gradients fill the first half of the slot
                    g4 = grad16x4_to_float4(*reinterpret_cast<const uint2 *>(reinterpret_cast<const unsigned short *>(stage) + pos), a.grad_fmt);
                m4 = ld4(stage + kTile + pos);
                x4 = ld4(stage + 2 * kTile + pos);
                u4 = ld4(stage + 3 * kTile + pos);
                if (i == 0) {
                    const float4 v4 = ld4(stage + 4 * kTile + pos);
                    vv[0] = v4.x; vv[1] = v4.y; vv[2] = v4.z; vv[3] = v4.w;
#pragma unroll
                    for (int q = 0; q < 4; ++q) d[q] = denom(a.c, vv[q]);
                }
            }
            release_stage(sh, s, dep_bits(g4, m4, x4, u4) ^ __float_as_uint(d[0]));
            if (++s == R) { s = 0; phase ^= 1u; }
            const float gg[4] = {g4.x, g4.y, g4.z, g4.w}, mm[4] = {m4.x, m4.y, m4.z, m4.w};
            const float xx[4] = {x4.x, x4.y, x4.z, x4.w}, uu[4] = {u4.x, u4.y, u4.z, u4.w};
            float mo[4], xo[4], uo[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                mo[q] = momentum(a.c, mm[q], gg[q]);            // momentum update
                const float step = f_mul(a.gamma, mo[q]);
                xo[q] = f_sub(xx[q], f_div(step, d[q]));        // model update
                uo[q] = f_add(uu[q], step);                     // buffer update
                if (DO_VAR) Gs[q] += (double)gg[q];
            }
            const long long row = (long long)i * st.n_pad + j;
            st4_stream(st.m + row, make_float4(mo[0], mo[1], mo[2], mo[3]));
            st4_stream(st.x + row, make_float4(xo[0], xo[1], xo[2], xo[3]));
            st4_stream(st.u + row, make_float4(uo[0], uo[1], uo[2], uo[3]));
        }
        if (DO_VAR) {
            float vo[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) vo[q] = variance(a.c, vv[q], mean_round(Gs[q], W));   // variance update
            st4_stream(st.v_next + j, make_float4(vo[0], vo[1], vo[2], vo[3]));
        }
    }
}

// ---------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------
// Tiles per unit and chunks per tile for a chunk size the ring kernels take (false: they do not).
static bool unit_shape(int chunk, int *tiles, int *chunks_per_tile)
{
    *tiles = 1;
    *chunks_per_tile = 1;
    if (chunk >= kTile) {
        if (chunk % kTile != 0) return false;
        *tiles = chunk / kTile;
        // eight tiles (chunk 16384) would fill the ring and leave no registers for the deferred
        // stores: the chunk-per-block kernel is the faster one there
        return *tiles == 1 || *tiles == 2 || *tiles == 4;
    }
    if (chunk < 128 || kTile % chunk != 0) return false;
    *chunks_per_tile = kTile / chunk;      // 2, 4, 8 or 16: whole warps per chunk
    return true;
}

static size_t pipeline_fixed_smem(int W, int chunk)
{
    const int span = chunk < kTile ? kTile : chunk;
    const size_t head = 1024 + (size_t)W * (span / 32) * 4 + (size_t)kConsumerWarps * W * 4;
    return (head + 1023) & ~(size_t)1023;
}

// How many ring stages fit (0 = the pipelined kernel does not apply to this shape).
int pipeline_stages(const StateView &st, int grad_fmt)
{
    if (!(grad_fmt & kGradAligned)) return 0;
    int tiles, g;
    if (!unit_shape(st.chunk, &tiles, &g)) return 0;
    if (st.n / ((long long)tiles * kTile) < 1) return 0;
    const size_t budget = 227 * 1024;
    const size_t fixed = pipeline_fixed_smem(st.W, st.chunk);
    // the server tiles of a unit stay in the ring over the l1 sum: tiles + 1 stages at least
    const int least = tiles + 1;
    if (fixed + (size_t)least * kStageBytes > budget) return 0;
    int stages = (int)((budget - fixed) / kStageBytes);
    if (stages > kSyncStages) stages = kSyncStages;
    return stages >= least ? stages : 0;
}

// Chunks per work unit of the ring kernels (1 for chunks of 2048 coordinates and more).
int pipeline_chunks_per_unit(const StateView &st) { return st.chunk < kTile ? kTile / st.chunk : 1; }

template <int TILES, int G, bool DO_VAR>
static cudaError_t launch_pipe(const PipeArgs &a, int grid, size_t smem, cudaStream_t s)
{
    auto kern = step_sync_pipelined_kernel<TILES, G, DO_VAR>;
    static SmemLimitOnce once;   // per instantiation
    const cudaError_t e = once.ensure(kern, 227 * 1024);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, smem, s>>>(a);
    return cudaGetLastError();
}

// Runs the units [first_unit, first_unit + n_units) of a sync step (a unit is one chunk of 2048 coordinates or
// more, or the 2048 / chunk smaller chunks of one tile); what is left over is the caller's.
// *var_fused tells whether the variance update was done here too.
cudaError_t launch_step_sync_pipelined(const StateView &st, const GradPtrs &g, const Consts &c, float gamma,
                                       float gamma_sum, bool do_var, int grad_fmt, long long first_unit, long long n_units, int stages,
                                       int sm_count, ErrorWords error_flag, unsigned long long *sched, unsigned long long wait_limit_ns,
                                       long long test_stop_after_tiles, bool *var_fused, cudaStream_t s)
{
    PipeArgs a;
    a.st = st; a.g = g; a.c = c; a.gamma = gamma; a.gamma_sum = gamma_sum;
    a.first_chunk = first_unit;
    a.n_full_chunks = n_units;
    a.stages = stages;
    a.error_flag = error_flag;
    a.sched = sched;
    a.grad_fmt = grad_fmt;
    a.wait_limit_ns = wait_limit_ns;
    a.test_stop_after_tiles = test_stop_after_tiles;
    const int grid = (int)(n_units < sm_count ? n_units : sm_count);
    int tiles, cpt;
    if (!unit_shape(st.chunk, &tiles, &cpt)) return cudaErrorInvalidValue;
    size_t fixed = pipeline_fixed_smem(st.W, st.chunk);
    if (tiles == 4 && do_var) {           // two tiles of gradient sums in shared memory; the ring gives up a stage for them
        fixed += 2 * 4 * kConsumers * sizeof(double);
        const int fit = (int)((227 * 1024 - fixed) / kStageBytes);
        if (fit < tiles + 1) do_var = false;
        else if (stages > fit) a.stages = stages = fit;
    }
    if (!do_var) fixed = pipeline_fixed_smem(st.W, st.chunk);
    const size_t smem = fixed + (size_t)stages * kStageBytes;
    *var_fused = do_var;
#define ZOA_PIPE(T, GG) (do_var ? launch_pipe<T, GG, true>(a, grid, smem, s) : launch_pipe<T, GG, false>(a, grid, smem, s))
    switch (tiles * 100 + cpt) {
    case 101: return ZOA_PIPE(1, 1);
    case 201: return ZOA_PIPE(2, 1);
    case 401: return ZOA_PIPE(4, 1);
    case 102: return ZOA_PIPE(1, 2);
    case 104: return ZOA_PIPE(1, 4);
    case 108: return ZOA_PIPE(1, 8);
    case 116: return ZOA_PIPE(1, 16);
    default: return cudaErrorInvalidValue;
    }
#undef ZOA_PIPE
}

// The local step for the whole tiles [first_unit, first_unit + n_units) (tiles of 2048 coordinates); what is left
// over is the caller's.  Needs 16-byte aligned gradients.
cudaError_t launch_local_step_pipelined(const StateView &st, const GradPtrs &g, const Consts &c, float gamma, bool do_var,
                                        int grad_fmt, long long first_unit, long long n_units, int sm_count, ErrorWords error_flag,
                                        unsigned long long *sched, unsigned long long wait_limit_ns,
                                        long long test_stop_after_tiles, cudaStream_t s)
{
    PipeArgs a;
    a.st = st; a.g = g; a.c = c; a.gamma = gamma; a.gamma_sum = 0.f;
    a.first_chunk = first_unit;
    a.n_full_chunks = n_units;
    a.stages = (227 * 1024 - 1024) / kLocalStageBytes;        // five stages of 40 KB
    a.error_flag = error_flag;
    a.sched = sched;
    a.grad_fmt = grad_fmt;
    a.wait_limit_ns = wait_limit_ns;
    a.test_stop_after_tiles = test_stop_after_tiles;
    const int grid = (int)(n_units < sm_count ? n_units : sm_count);
    const size_t smem = 1024 + (size_t)a.stages * kLocalStageBytes;
    static SmemLimitOnce once[2];
    cudaError_t e = once[0].ensure(local_step_pipelined_kernel<false>, 227 * 1024);
    if (e == cudaSuccess) e = once[1].ensure(local_step_pipelined_kernel<true>, 227 * 1024);
    if (e != cudaSuccess) return e;
    if (do_var) local_step_pipelined_kernel<true><<<grid, kThreads, smem, s>>>(a);
    else local_step_pipelined_kernel<false><<<grid, kThreads, smem, s>>>(a);
    return cudaGetLastError();
}

}  // namespace zoa

namespace zoa {

int alg2_pipeline_stages(const StateView &st, int grad_fmt)
{
    if (!(grad_fmt & kGradAligned)) return 0;
    if (st.chunk != kTile && st.chunk != 2 * kTile && st.chunk != 4 * kTile) return 0;
    if (st.n / st.chunk < 1) return 0;
    const size_t budget = 227 * 1024;
    const size_t fixed = pipeline_fixed_smem(st.W, st.chunk);
    if (fixed + 2 * (size_t)kStage2Bytes > budget) return 0;
    int stages = (int)((budget - fixed) / kStage2Bytes);
    return stages > kMaxStages ? kMaxStages : stages;
}

template <int TILES>
static cudaError_t launch_alg2_pipe(const PipeArgs &a, int grid, size_t smem, cudaStream_t s)
{
    auto kern = alg2_pipelined_kernel<TILES>;
    static SmemLimitOnce once;
    const cudaError_t e = once.ensure(kern, 227 * 1024);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, smem, s>>>(a);
    return cudaGetLastError();
}

// The full chunks of a compressed step of Algorithm 2; a ragged last chunk is the caller's.
cudaError_t launch_alg2_pipelined(const StateView &st, const GradPtrs &g, const Consts &c, float gamma, int grad_fmt,
                                  int stages, int sm_count, ErrorWords error_flag, unsigned long long *sched,
                                  unsigned long long wait_limit_ns, long long test_stop_after_tiles, cudaStream_t s)
{
    PipeArgs a;
    a.st = st; a.g = g; a.c = c; a.gamma = gamma; a.gamma_sum = 0.f;
    a.first_chunk = 0;
    a.n_full_chunks = st.n / st.chunk;
    a.stages = stages;
    a.error_flag = error_flag;
    a.sched = sched;
    a.grad_fmt = grad_fmt;
    a.wait_limit_ns = wait_limit_ns;
    a.test_stop_after_tiles = test_stop_after_tiles;
    const int grid = (int)(a.n_full_chunks < sm_count ? a.n_full_chunks : sm_count);
    const size_t smem = pipeline_fixed_smem(st.W, st.chunk) + (size_t)stages * kStage2Bytes;
    switch (st.chunk / kTile) {
    case 1: return launch_alg2_pipe<1>(a, grid, smem, s);
    case 2: return launch_alg2_pipe<2>(a, grid, smem, s);
    case 4: return launch_alg2_pipe<4>(a, grid, smem, s);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace zoa
