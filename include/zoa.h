/*
 * zoa - the per-parameter optimizer step of 0/1 Adam (arXiv 2202.06009) for W
 * data-parallel workers held as separate state buffers on one NVIDIA B200.
 *
 * Plain C ABI.  Pointers are marked (device) or (host).  The library owns all
 * optimizer state; gradients are borrowed, read-only, and must stay valid until
 * the stream has finished the call's work.  Every call that takes a stream
 * enqueues its work on that stream and returns after host-side validation
 * only; nothing synchronises unless stated.  A handle is not thread-safe
 * (different handles may be used from different threads).
 *
 * Errors.  ZOA_ERR_ARG and ZOA_ERR_STATE are found before anything is enqueued:
 * the handle and its state are unchanged.  After ZOA_ERR_CUDA, ZOA_ERR_ALLOC or
 * ZOA_ERR_DEVICE from a call that enqueues work (a step, reduce, copy or
 * import call) part of the call's work may have run and the host scalars may
 * not have advanced: the optimizer state is undefined and should be restored
 * from a checkpoint (zoa_import_state) or rebuilt.  Once a kernel has given up on
 * a bounded wait, every step, reduce, compress, allreduce and server entry point
 * returns ZOA_ERR_DEVICE (without synchronising; the news travels through a word of
 * pinned host memory) until zoa_check_device has reported and cleared it.
 *
 * Arithmetic contract (what "the same result" means for every entry point):
 * all state is IEEE binary32; each elementwise operation is one
 * round-to-nearest binary32 operation (no fused multiply-add, subnormals
 * kept); the three reductions of the method - the l1 norm of a chunk, the mean
 * over workers of the compressed buffers, the mean over workers of the
 * gradients - accumulate in binary64 and are rounded to binary32 once.
 *
 * State layout in device memory (n = n_params, row stride n_pad = n rounded up
 * to 128 elements, padding always zero):
 *   x, m, u, delta_w   float [W][n_pad]     per-worker model, momentum, buffer, error
 *   v, delta_s, x_sync float [n_pad]        variance, server error, model at the last sync
 *   words_w            uint32 [W][n_pad/32] sign bits each worker sent
 *   scales_w           float  [W][n_chunks] one magnitude per chunk and worker
 *   words_s, scales_s  uint32 [n_pad/32], float [n_chunks]   what the server sent back
 * Coordinate j is bit (j mod 32), least significant first, of word j / 32;
 * unused bits are zero.  Chunk c covers coordinates [c*chunk, min((c+1)*chunk, n)).
 */
#ifndef ZOA_H
#define ZOA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct zoa_handle_s *zoa_handle;

typedef enum {
    ZOA_OK = 0,
    ZOA_ERR_ARG = 1,    /* a bad argument; nothing was changed */
    ZOA_ERR_ALLOC = 2,  /* device or host memory could not be had */
    ZOA_ERR_CUDA = 3,   /* a CUDA call or an earlier kernel failed; see zoa_last_error */
    ZOA_ERR_STATE = 4,  /* calls out of order: t not increasing, reduce with nothing accumulated */
    ZOA_ERR_DEVICE = 5, /* a kernel gave up on a bounded wait or wrote out of bounds; state is undefined */
    ZOA_ERR_NONFINITE = 6 /* zoa_check_finite found NaN or infinite values */
} zoa_status;

typedef enum {
    ZOA_BUF_X = 0, ZOA_BUF_M = 1, ZOA_BUF_U = 2, ZOA_BUF_DELTA_W = 3,
    ZOA_BUF_V = 4, ZOA_BUF_DELTA_S = 5, ZOA_BUF_X_SYNC = 6,
    ZOA_BUF_WORDS_W = 7, ZOA_BUF_SCALES_W = 8, ZOA_BUF_WORDS_S = 9, ZOA_BUF_SCALES_S = 10
} zoa_buffer;

typedef struct {
    int64_t n_steps;        /* optimizer steps taken (Algorithm 1 iterations) */
    int64_t n_syncs;        /* 1-bit AllReduce rounds */
    int64_t n_var_updates;  /* variance updates (steps in T_v) */
    int64_t n_launches;     /* kernels this handle has launched */
    int64_t bits_per_worker;/* bits a worker would have sent so far: n_syncs * (n + 32 n_chunks) */
    int64_t t_last;         /* last step index seen, -1 before the first */
    int64_t t_sync;         /* t' of Algorithm 1 */
    double gamma_sum;       /* learning rates accumulated into u since the last sync */
} zoa_stats;

/* The inputs of Algorithm 1 (its "Require" clause): creates the state for a d = n_params
 * dimensional model on W workers with m_0 = v_0 = u_0 = 0, both compression
 * errors 0 (Algorithm 3), x_0 = 0 until zoa_set_params, t' = 0, on the current
 * CUDA device.  chunk is the number of consecutive coordinates that share one
 * magnitude in the compressor of Eq. 3 (chunk >= n_params gives Eq. 3 as printed).
 * Requires n_params >= 1, 1 <= W <= 64, 0 <= beta < 1, eps > 0, chunk a
 * multiple of 32 in [32, 2^30].  Chunks up to 16384 are handled by one thread
 * block each (the fast kernels); larger ones, up to the whole vector, by
 * multi-pass kernels that take each l1 norm in two steps.  Allocates device
 * memory (cudaMalloc). */
zoa_status zoa_create(zoa_handle *out, size_t n_params, int W, float beta1, float beta2,
                      float eps, int chunk);

/* Frees everything the handle owns.  Synchronises the device first. */
zoa_status zoa_destroy(zoa_handle h);

/* x_0 of Algorithm 1: copies x0 (device, n_params floats) into every worker's
 * model and into x_sync.  All workers start from the same model, as the
 * analysis of the method assumes. */
zoa_status zoa_set_params(zoa_handle h, const float *x0, void *stream);

/* T_v of Algorithm 1 as an explicit list of step indices (host, any order).
 * Default: empty (the variance is never updated). */
zoa_status zoa_set_var_steps(zoa_handle h, const int64_t *steps, size_t count);

/* The same call under the name zoa_set_var_policy. */
zoa_status zoa_set_var_policy(zoa_handle h, const int64_t *steps, size_t count);

/* T_v by the rule of the paragraph "Policy for T_v and T_u": the j-th update is
 * at k_j with k_0 = 0 and k_{j+1} - k_j = 2^floor(j / kappa), for k_j < freeze_at. */
zoa_status zoa_set_var_policy_doubling(zoa_handle h, int kappa, int64_t freeze_at);

/* The two schedules of the paragraph "Policy for T_v and T_u" as plain host
 * functions (no handle, no GPU).  Both return the number of entries the full
 * answer has and write at most `capacity` of them (pass NULL, 0 to size).
 * zoa_policy_var_steps: k_0 = 0, k_{j+1} - k_j = 2^floor(j / kappa) while
 * k_j < freeze_at (the paper uses kappa = 16).
 * zoa_policy_sync_pieces: the interval between syncs is 1 through the learning
 * rate warm-up and then doubles every `double_every` steps (the steps in which
 * the learning rate halves), never above max_interval (the paper: warm-up 12.5K
 * steps, 32678, 16 for BERT); returned as pieces for zoa_set_sync_policy. */
size_t zoa_policy_var_steps(int kappa, int64_t freeze_at, int64_t *out, size_t capacity);
size_t zoa_policy_sync_pieces(int64_t warmup, int64_t double_every, int32_t max_interval,
                              int64_t *boundaries, int32_t *intervals, size_t capacity);

/* Installs zoa_policy_sync_pieces on the handle.  With freeze_variance != 0 it
 * also drops every T_v step from the first step whose sync interval exceeds 1
 * (the paper stops updating the variance there); call it after the T_v setter. */
zoa_status zoa_set_sync_policy_doubling(zoa_handle h, int64_t warmup, int64_t double_every,
                                        int32_t max_interval, int freeze_variance);

/* T_u of Algorithm 1 as a piecewise-constant interval: piece r starts at step
 * boundaries[r] (host, strictly increasing, boundaries[0] = 0) and has a sync
 * at every step t with (t - boundaries[r]) % intervals[r] == 0.  Default: one
 * piece with interval 1 (sync at every step). */
zoa_status zoa_set_sync_policy(zoa_handle h, const int64_t *boundaries, const int32_t *intervals,
                               size_t count);

/* Membership tests, 1 or 0 (negative on a bad handle). */
int zoa_sync_due(zoa_handle h, int64_t t);
int zoa_var_due(zoa_handle h, int64_t t);

/* Algorithm 1: the momentum, model and buffer updates for every worker, and the
 * variance update (full-precision mean of the gradients, then v) when t is in T_v
 * (the new variance takes effect from the next step on, so that a following
 * zoa_onebit_reduce still uses v_t as the algorithm's model sync does).
 * grads: (host) array of W (device) pointers, n_params elements each (binary32
 * unless ZOA_OPT_GRAD_TYPE says otherwise), worker i's gradient at step t;
 * 16-byte aligned pointers take the vector path.
 * lr is gamma_t; t must be larger than at the previous step. */
zoa_status zoa_step(zoa_handle h, const void *const *grads, float lr, int64_t t, void *stream);

/* Algorithm 1's sync branch (t in T_u) with Algorithm 3 inside: compresses u + delta per
 * worker (Eq. 3 per chunk), averages, compresses again on the "server" with its
 * own error, then m = u_bar / sum(gamma), x = x_sync - u_bar / sqrt(v_t + eps),
 * u = 0 on every worker.  ZOA_ERR_STATE if nothing was accumulated since the
 * last sync (the divisor of the momentum approximation would be zero). */
zoa_status zoa_onebit_reduce(zoa_handle h, void *stream);

/* The two halves of zoa_onebit_reduce, for callers that want to time or
 * interleave them: zoa_onebit_compress is the worker side of Algorithm 3 (packs
 * u + delta of every worker into words_w / scales_w, keeps the errors);
 * zoa_onebit_average is the server side and the rest of Algorithm 1's sync branch (reads
 * words_w / scales_w).  compress then average == zoa_onebit_reduce. */
zoa_status zoa_onebit_compress(zoa_handle h, void *stream);
zoa_status zoa_onebit_average(zoa_handle h, void *stream);

/* Algorithm 3 by itself, z_bar = 1bit-AllReduce(z; delta, delta_bar), on buffers the
 * caller owns: z is a (host) array of W (device) pointers of n_params floats (read
 * only, any alignment; 16-byte aligned ones take the vector path), z_bar (device)
 * receives the n_params floats every worker would get back.  The worker errors, the
 * server error and the wire buffers are the handle's (ZOA_BUF_DELTA_W, ZOA_BUF_DELTA_S,
 * ZOA_BUF_WORDS_*, ZOA_BUF_SCALES_*); x, m, u, v are not touched.  Works on any handle
 * with chunk <= 16384.  zoa_allreduce_compress is the worker side alone (packs z + delta
 * into words_w / scales_w, keeps the errors), zoa_allreduce_average the server side alone
 * (reads words_w / scales_w and the server error, writes the server error, words_s /
 * scales_s and, if z_bar is not NULL, z_bar); compress then average == zoa_onebit_allreduce.
 * zoa_create_allreduce makes a handle that holds only this state - W + 1 error rows
 * and the packed buffers, about a fifth of a full handle - on which only these three
 * calls, buffer access, the checks and zoa_destroy work (the others: ZOA_ERR_STATE). */
zoa_status zoa_create_allreduce(zoa_handle *out, size_t n_params, int W, int chunk);
zoa_status zoa_onebit_allreduce(zoa_handle h, const float *const *z, float *z_bar, void *stream);
zoa_status zoa_allreduce_compress(zoa_handle h, const float *const *z, void *stream);
zoa_status zoa_allreduce_average(zoa_handle h, float *z_bar, void *stream);

/* Building blocks for the paper's own mapping, one worker per GPU (Algorithm 3:
 * every worker sends its packed buffer to the server, the server sends its
 * packed result to every worker).  Each GPU holds a handle for its own
 * worker(s) and is the server for a contiguous range of chunks; the
 * collectives run between these calls (paper_2202_06009_b200/distributed.py
 * drives them with torch.distributed):
 *   zoa_step, zoa_onebit_compress          local step, pack u + delta (words_w, scales_w)
 *   -- all-to-all of each range's words and scales --
 *   zoa_dist_server_range                  server side for this GPU's chunk range
 *   -- all-gather of words_s / scales_s into every handle's own buffers --
 *   zoa_dist_apply                         rest of Algorithm 1's sync branch from words_s / scales_s
 * zoa_dist_server_range: words_all / scales_all (device) hold, for each of the
 * W_total workers in worker order, the packed words and the magnitudes of the
 * chunks [first_chunk, first_chunk + n_chunks), rows words_stride / scales_stride
 * elements apart, starting at the range's first word / chunk.  It updates the
 * server error of that range and writes that range of words_s / scales_s.
 * Chunks above 16384 are not supported here.
 * zoa_dist_variance: the variance update of Algorithm 1 when the mean gradient g_bar
 * (device, n_params floats) comes from a collective; call it after zoa_step on a
 * step in T_v for which the handle's own T_v list is empty.  A collective's
 * binary32 sum is not the binary64 worker-order sum of the single-GPU path, so v
 * (and through it x) can differ from it in the last bits. */
zoa_status zoa_dist_server_range(zoa_handle h, const uint32_t *words_all, size_t words_stride,
                                 const float *scales_all, size_t scales_stride, int W_total,
                                 int64_t first_chunk, int64_t n_chunks, void *stream);
zoa_status zoa_dist_apply(zoa_handle h, void *stream);
zoa_status zoa_dist_variance(zoa_handle h, const float *g_bar, void *stream);

/* The same round with the two exchanges done by the kernels themselves, as stores
 * through peer pointers (NVLink), for handles that hold one worker each:
 *   zoa_dist_step_pack_push   local updates of a sync step + worker side of Algorithm 3,
 *                             the packed words and magnitudes of each chunk stored into
 *                             the receive buffer of the rank that serves it
 *   -- every rank waits until all ranks have finished that call --
 *   zoa_dist_server_push      server side for this rank's chunk range, its packed result
 *                             stored into every rank's whole-vector words_s / scales_s
 *   -- every rank waits again --
 *   zoa_dist_apply
 * No kernel waits for another rank: the two waits belong to the caller (a
 * stream-ordered barrier between the ranks).  world ranks; rank s serves the
 * chunks [chunk_begin[s], chunk_begin[s+1]) (host array of world + 1 entries, from
 * 0 to the number of chunks, not decreasing).  peer_words[s] / peer_scales[s]
 * (host arrays of world device pointers) point at the first word / magnitude of
 * that range inside the row that rank s keeps for the calling rank, i.e. inside
 * the words_all / scales_all it will pass to zoa_dist_server_push; they may be
 * NULL for ranks that serve no chunk.  zoa_dist_pack_push is the worker side
 * alone, after zoa_step.  zoa_dist_step_pack_push takes the rank's gradient
 * (device, n_params elements in the handle's gradient type) and stands for
 * zoa_step on a sync step: the half-step momentum, model and buffer are formed
 * in registers and not stored, since zoa_dist_apply overwrites all three; the
 * variance update of a T_v step still goes through zoa_dist_variance.  The
 * handle's own words_w / scales_w are written as well.  peer_words_s[r] /
 * peer_scales_s[r] point at the first element of rank r's whole-vector buffers
 * (n_pad/32 words, n_chunks magnitudes; the calling rank's own entry may be its
 * own buffers or any other buffer of that size).  Errors: ZOA_ERR_ARG for a
 * handle with more than one worker, chunks above 16384, a malformed table or a
 * NULL pointer; ZOA_ERR_STATE as for zoa_step.  Nothing is allocated.  (The
 * paper ships these buffers over the network; it describes no such kernels.) */
zoa_status zoa_dist_pack_push(zoa_handle h, int world, const int64_t *chunk_begin,
                              void *const *peer_words, void *const *peer_scales, void *stream);
zoa_status zoa_dist_step_pack_push(zoa_handle h, const void *grad, float lr, int64_t t, int world,
                                   const int64_t *chunk_begin, void *const *peer_words,
                                   void *const *peer_scales, void *stream);
zoa_status zoa_dist_server_push(zoa_handle h, const uint32_t *words_all, size_t words_stride,
                                const float *scales_all, size_t scales_stride, int W_total,
                                int64_t first_chunk, int64_t n_chunks, int world,
                                void *const *peer_words_s, void *const *peer_scales_s, void *stream);

/* zoa_step followed by zoa_onebit_reduce, same results bit for bit, in one
 * pass over memory that never writes the half-step values. */
zoa_status zoa_step_sync(zoa_handle h, const void *const *grads, float lr, int64_t t,
                         void *stream);

/* One iteration of Algorithm 2 (the frozen-variance framework that exchanges
 * gradients, not accumulated updates; 1-bit Adam when T_v is an initial run of
 * steps).  If t is in T_v: g_bar = mean of the W gradients (Algorithm 4) and the
 * variance moves (effective from the next step); otherwise g_bar is the output
 * of the error-feedback 1-bit AllReduce of the gradients (Algorithm 3, same
 * error buffers and wire buffers as zoa_onebit_reduce).  Then on every worker
 * m = beta1 m + (1 - beta1) g_bar and x = x - lr m / sqrt(v_t + eps), m being the
 * momentum just computed (the convention that makes this the no-local-step case
 * of Algorithm 1).  u, x_sync and the sum of learning rates are not touched.
 * Arguments and errors as zoa_step. */
zoa_status zoa_alg2_step(zoa_handle h, const void *const *grads, float lr, int64_t t, void *stream);

/* One iteration of Algorithm 1 under the handle's own policies: zoa_step_sync
 * if t is in T_u, else zoa_step. */
zoa_status zoa_step_auto(zoa_handle h, const void *const *grads, float lr, int64_t t,
                         void *stream);

/* The same iteration with gradients in (host) memory: host_grads is an array
 * of W (host) pointers of n_params floats (pinned memory copies fastest).
 * Copies them to a device staging area the handle allocates on first use,
 * runs zoa_step_auto, and, if host_x_out is not NULL, copies worker 0's model
 * back (n_params floats).  Large problems are cut into eight chunk ranges so
 * that the copies of one range (on a stream of the handle's own) overlap the
 * kernels and the result copy of the previous one (on `stream`); everything is
 * ordered with `stream`, which therefore tells when the step and host_x_out are
 * done.  Does not synchronise. */
zoa_status zoa_step_host(zoa_handle h, const void *const *host_grads, float lr, int64_t t,
                         float *host_x_out, void *stream);

/* Borrowed (device) pointer to one row of a state buffer and its length in
 * elements (n_pad, n_pad/32 or n_chunks).  worker is ignored for shared buffers.
 * With chunks above 16384 the library keeps the two error buffers between syncs
 * as "what was compressed", the magnitude still to be subtracted; asking for
 * ZOA_BUF_DELTA_W or ZOA_BUF_DELTA_S (here, in zoa_copy_out / zoa_copy_in and in
 * zoa_export_state) first brings them to their plain form, which waits for the
 * device and runs one short kernel. */
zoa_status zoa_get_buffer(zoa_handle h, zoa_buffer which, int worker, void **dev_ptr,
                          size_t *n_elems);

/* The same call under the name zoa_get_ptr (`what` takes the zoa_buffer values). */
zoa_status zoa_get_ptr(zoa_handle h, int what, int worker, void **dev_ptr, size_t *stride_elems);

/* Checkpoint of everything Algorithm 1 carries from one iteration to the next
 * (its "Require" clause and the two errors of Algorithm 3): x, m, u and the
 * worker error of every worker, v_t and - when a T_v step's update is still
 * pending, i.e. between zoa_step and the next step call - v_{t+1} with the
 * pending mark, the server error, x_sync, the sum of learning rates since the
 * last sync, t', the last step index, beta1, beta2, eps, both policies and the
 * step / sync / variance-update counters.  The packed wire buffers are outputs
 * of a sync, not state, and are not saved; options (zoa_set_option) are not either.
 * zoa_state_size: bytes the blob takes for the handle as it stands (it grows
 * with the policy tables).  zoa_export_state: waits for the device, then writes
 * the blob to host_blob (host, at least zoa_state_size bytes).
 * zoa_import_state: restores a blob into a handle created with the same
 * n_params, W and chunk (ZOA_ERR_ARG otherwise, or if the blob is malformed or
 * truncated; nothing is changed then); waits for the device first.  A run that
 * exports, imports into a fresh handle and continues gives the same bits as
 * the run that was never interrupted, also when the export falls between
 * zoa_step on a T_v step and zoa_onebit_reduce. */
zoa_status zoa_state_size(zoa_handle h, size_t *bytes);
zoa_status zoa_export_state(zoa_handle h, void *host_blob, size_t bytes);
zoa_status zoa_import_state(zoa_handle h, const void *host_blob, size_t bytes);

/* Synchronous copies between a state row and (host) memory, in elements of the
 * buffer's type from element `offset`; for tests and inspection.  ZOA_BUF_V is
 * the newest variance (v_{t+1} while an update is pending); a checkpoint
 * needs both, which zoa_export_state saves. */
zoa_status zoa_copy_out(zoa_handle h, zoa_buffer which, int worker, size_t offset, size_t count,
                        void *host_dst);
zoa_status zoa_copy_in(zoa_handle h, zoa_buffer which, int worker, size_t offset, size_t count,
                       const void *host_src);

/* Host scalars of Algorithm 1 (sum of gammas since the last sync, t', last t);
 * lets tests and benchmarks rewind the step counter. */
zoa_status zoa_set_scalars(zoa_handle h, double gamma_sum, int64_t t_sync, int64_t t_last);

zoa_status zoa_get_stats(zoa_handle h, zoa_stats *out);

/* Waits for the device and reports ZOA_ERR_CUDA if a CUDA error is pending,
 * ZOA_ERR_DEVICE if a kernel of this handle gave up on a bounded wait since the
 * last check (which also clears that condition, so that step calls are accepted
 * again), or if one of the guard areas that surround every device buffer of
 * the handle no longer holds its pattern (a kernel wrote out of bounds). */
zoa_status zoa_check_device(zoa_handle h);

/* Debug scan (synchronous, reads every float state buffer once): counts the NaN
 * and infinite values in x, m, u, both errors, v and x_sync; returns
 * ZOA_ERR_NONFINITE if there are any.  n_nonfinite may be NULL.  A non-finite
 * gradient spreads through the l1 norm to its whole chunk at the next sync. */
zoa_status zoa_check_finite(zoa_handle h, int64_t *n_nonfinite);

/* Tuning switches.  ZOA_OPT_PIPELINE (default 1): run the fused sync step and the
 * compressed step of Algorithm 2 as the persistent bulk-copy-ring kernels where
 * the shape allows (chunk 2048, 4096 or 8192, 16-byte aligned gradients) and the
 * problem has at least four chunks per SM; 2: wherever the shape allows; 0: always
 * the chunk-per-block kernels.  The results are the same bit for bit.
 * ZOA_OPT_WAIT_LIMIT_MS (default 2000): how long a kernel thread waits for an
 * asynchronous copy before it gives up; the kernel then ends early, the state is
 * undefined and zoa_check_device reports ZOA_ERR_DEVICE.
 * ZOA_OPT_TEST_STOP_AFTER_TILES (default 0 = off): for testing that error path
 * only - the copy-issuing lane of every block stops after this many tiles (in the
 * server kernel of zoa_allreduce_average the copies are never started), so the
 * waits of the other threads run out after the limit.
 * ZOA_OPT_GRAD_TYPE (default ZOA_GRAD_F32): element type of the buffers passed as
 * `grads` / `host_grads` from now on: binary32, binary16 (IEEE half) or bfloat16.
 * 16-bit gradients are converted to binary32 exactly when they are loaded; all
 * arithmetic and all state stay binary32, so the results equal those of the same
 * values passed as binary32.  (The paper trains in FP16; its communication buffer
 * u is still formed in the optimizer's precision.) */
enum { ZOA_OPT_PIPELINE = 1, ZOA_OPT_WAIT_LIMIT_MS = 2, ZOA_OPT_TEST_STOP_AFTER_TILES = 3, ZOA_OPT_GRAD_TYPE = 4 };
enum { ZOA_GRAD_F32 = 0, ZOA_GRAD_F16 = 1, ZOA_GRAD_BF16 = 2 };
zoa_status zoa_set_option(zoa_handle h, int option, int value);

/* Text of the last error on this handle (or of the last failed zoa_create if h
 * is NULL).  Never NULL. */
const char *zoa_last_error(zoa_handle h);

/* (The paper has no counterpart to this entry point; it exists for callers that
 * must not allocate device memory.)
 * The error-feedback 1-bit AllReduce of Algorithm 3 on buffers the caller owns,
 * without a handle and without allocating anything: no cudaMalloc, cudaFree or
 * allocating library call is made.  It is meant for code that runs where
 * device allocation is forbidden or harmful - inside a region whose memory a
 * framework's allocator has already handed out, in a latency-critical loop that
 * cannot afford cudaMalloc's implicit synchronisation, in a process whose
 * memory is pre-partitioned between tenants, or in a clean-up path that runs
 * when the device is already full.
 *   z        (host) array of W (device) pointers, n floats each: the buffers to reduce, read-only
 *   delta_w  (host) array of W (device) pointers, n floats each: worker errors, updated in place
 *   delta_s  (device) n floats: server error, updated in place
 *   z_bar    (device) n floats: the result, +-magnitude of the server's chunk
 * The packed sign words and magnitudes that travel between the two kernels of
 * a call live in an array built into the library (1,048,576 32-bit slots, 4 MiB,
 * held by every GPU that loads the library until the process exits).  The call
 * needs W * (ceil(n/32) + ceil(n/chunk)) slots and returns ZOA_ERR_ARG, with a
 * text in zoa_static_last_error(), if that is more.  All calls on a device share
 * the array: calls whose GPU work may overlap (different streams without
 * ordering) race on it and must be serialised by the caller.  The array keeps
 * the last call's contents; a call reads only what it wrote itself, so nothing
 * needs clearing.  The first call on each device looks up the array's device
 * address and raises two kernels' shared-memory limit: make that first call
 * before any stream capture starts.  Pointers that are all 16-byte aligned take
 * the 128-bit path, others a scalar one.  Work is enqueued on `stream`; the
 * call does not synchronise. */
zoa_status zoa_onebit_allreduce_static(const float *const *z, float *const *delta_w, float *delta_s,
                                       float *z_bar, size_t n, int W, int chunk, void *stream);

/* Capacity of that built-in array in 32-bit slots, and the text of the last
 * error zoa_onebit_allreduce_static returned on this thread (never NULL). */
size_t zoa_static_scratch_slots(void);
const char *zoa_static_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ZOA_H */
