// The C ABI of include/zoa.h: handle, validation, policies, host scalars of
// Algorithm 1 (sum of gammas, t', pending variance) and kernel dispatch.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "../../include/zoa.h"
#include "zoa_internal.h"

using namespace zoa;

struct zoa_handle_s {
    int device = 0, sm_count = 148;
    long long n = 0, n_pad = 0, n_chunks = 0, words_stride = 0;
    int W = 0, chunk = 0;
    Consts c{};
    float *x = nullptr, *m = nullptr, *u = nullptr, *dw = nullptr;
    float *v_cur = nullptr, *v_nxt = nullptr, *ds = nullptr, *xs = nullptr;
    uint32_t *words_w = nullptr, *words_s = nullptr;
    float *scales_w = nullptr, *scales_s = nullptr;
    float *staging = nullptr;      // [W][n_pad], device copy of host gradients (zoa_step_host)
    cudaStream_t copy_stream = nullptr;                 // host-to-device copies of zoa_step_host run here ...
    std::vector<cudaEvent_t> copy_events;               // ... and these order them with the caller's stream
    int *error_flag = nullptr;     // device int: a kernel gave up on a bounded wait
    int *error_host = nullptr;     // the same news in pinned, mapped host memory: the step entry points test it without synchronising
    int *error_host_dev = nullptr; // its device-side address
    unsigned long long *sched = nullptr;   // device [2]: chunk counter of the persistent kernel, finished blocks
    double *partials = nullptr;    // device [W + 1][n_chunks * segments]: per-segment l1 sums, chunk > 16384 only
    bool large_chunk = false;
    bool allreduce_only = false;   // zoa_create_allreduce: no x, m, u, v, x_sync; only Algorithm 3's own state
    // Large chunks only: the worker-error rows / the server-error row hold what was compressed at the last
    // sync, the magnitude still to be subtracted (the large-chunk kernels read that form directly).
    bool dw_pending = false, ds_pending = false;
    int grad_type = 0;             // 0 binary32, 1 binary16, 2 bfloat16: how `grads` buffers are read
    int use_pipeline = 1;          // ring kernels: 0 never, 1 where the shape allows and the problem is large enough, 2 wherever the shape allows
    int wait_limit_ms = 2000;      // bound on every device-side wait
    long long test_stop_after_tiles = 0;   // error-path test hook, see zoa_set_option
    bool v_pending = false;        // v_nxt holds v_{t+1}; it becomes v at the next step
    std::vector<int64_t> var_steps;                    // T_v, sorted
    std::vector<int64_t> sync_bounds{0};               // T_u pieces
    std::vector<int32_t> sync_intervals{1};
    double gamma_sum = 0.0;
    int64_t t_sync = 0, t_last = -1;
    int64_t n_steps = 0, n_syncs = 0, n_var_updates = 0, n_launches = 0;
    struct Guarded { char *ptr; size_t bytes, padded; };
    std::vector<Guarded> guarded;  // every device buffer: user pointer, payload bytes, payload rounded up to 256
    std::string err;
};

// Named range around an entry point, for profilers (costs a pointer test when none is attached).
struct TraceRange {
    explicit TraceRange(const char *name) { nvtxRangePushA(name); }
    ~TraceRange() { nvtxRangePop(); }
};

static thread_local std::string g_create_error;   // text of this thread's last failed zoa_create

static zoa_status fail(zoa_handle h, zoa_status s, const std::string &msg)
{
    if (h) h->err = msg; else g_create_error = msg;
    return s;
}
static zoa_status fail_cuda(zoa_handle h, cudaError_t e, const char *what)
{
    return fail(h, e == cudaErrorMemoryAllocation ? ZOA_ERR_ALLOC : ZOA_ERR_CUDA,
                std::string(what) + ": " + cudaGetErrorString(e));
}
#define ZOA_CUDA(h, call)                                        \
    do {                                                         \
        cudaError_t e_ = (call);                                 \
        if (e_ != cudaSuccess) return fail_cuda(h, e_, #call);   \
    } while (0)

static bool on_own_device(zoa_handle h);

static StateView view(zoa_handle h)
{
    StateView st{};
    st.x = h->x; st.m = h->m; st.u = h->u; st.dw = h->dw;
    st.v = h->v_cur; st.v_next = h->v_nxt; st.ds = h->ds; st.xs = h->xs;
    st.words_w = h->words_w; st.scales_w = h->scales_w; st.words_s = h->words_s; st.scales_s = h->scales_s;
    st.n = h->n; st.n_pad = h->n_pad; st.n_chunks = h->n_chunks; st.words_stride = h->words_stride;
    st.W = h->W; st.chunk = h->chunk;
    return st;
}

// Every device buffer sits between two guard areas filled with a fixed pattern; zoa_check_device
// verifies them, so a kernel that writes outside a buffer is caught without a memory checker.
static const size_t kGuardBytes = 256;
static const unsigned char kGuardByte = 0xA5;

static void free_all(zoa_handle h)
{
    for (auto &b : h->guarded) cudaFree(b.ptr - kGuardBytes);
    h->guarded.clear();
    if (h->staging) cudaFree(h->staging);
    for (cudaEvent_t e : h->copy_events) cudaEventDestroy(e);
    h->copy_events.clear();
    if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
    h->copy_stream = nullptr;
    if (h->error_host) cudaFreeHost(h->error_host);
    h->error_host = h->error_host_dev = nullptr;
}

static ErrorWords error_words(zoa_handle h) { return ErrorWords{h->error_flag, h->error_host_dev}; }

// A kernel of an earlier call gave up on a bounded wait: every later step would run on undefined
// state, so the step entry points refuse until zoa_check_device has reported and cleared it.
static bool device_gave_up(zoa_handle h) { return h->error_host && *static_cast<volatile int *>(h->error_host) != 0; }
#define ZOA_REFUSE_AFTER_DEVICE_ERROR(h, who)                                                                      \
    do {                                                                                                            \
        if (device_gave_up(h))                                                                                      \
            return fail(h, ZOA_ERR_DEVICE, std::string(who) + ": an earlier kernel gave up waiting for its "        \
                                           "asynchronous copies; the optimizer state is undefined (zoa_check_device clears the flag)"); \
    } while (0)

static cudaError_t alloc_guarded(zoa_handle h, void **p, size_t bytes)
{
    char *base = nullptr;
    const size_t payload = (bytes + 255) / 256 * 256;
    cudaError_t e = cudaMalloc(reinterpret_cast<void **>(&base), payload + 2 * kGuardBytes);
    if (e != cudaSuccess) { *p = nullptr; return e; }
    e = cudaMemset(base, kGuardByte, payload + 2 * kGuardBytes);          // guards and the rounding slack
    if (e == cudaSuccess && bytes) e = cudaMemset(base + kGuardBytes, 0, bytes);   // the payload itself starts at zero
    if (e != cudaSuccess) { cudaFree(base); *p = nullptr; return e; }
    *p = base + kGuardBytes;
    h->guarded.push_back({base + kGuardBytes, bytes, payload});
    return cudaSuccess;
}

// True if every guard area still holds its pattern.
static cudaError_t guards_intact(zoa_handle h, bool *intact)
{
    unsigned char host[3 * 256];
    *intact = true;
    for (auto &b : h->guarded) {
        const size_t tail = b.padded - b.bytes + kGuardBytes;   // rounding slack + the guard after it
        cudaError_t e = cudaMemcpy(host, b.ptr - kGuardBytes, kGuardBytes, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess) e = cudaMemcpy(host + kGuardBytes, b.ptr + b.bytes, tail, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return e;
        for (size_t k = 0; k < kGuardBytes + tail; ++k)
            if (host[k] != kGuardByte) *intact = false;
    }
    return cudaSuccess;
}

template <typename T>
static cudaError_t alloc_zero(zoa_handle h, T **p, size_t count)
{
    return alloc_guarded(h, reinterpret_cast<void **>(p), count * sizeof(T));
}

static zoa_status create_handle(zoa_handle *out, size_t n_params, int W, float beta1, float beta2, float eps, int chunk,
                                bool allreduce_only)
{
    if (!out) return fail(nullptr, ZOA_ERR_ARG, "zoa_create: out is NULL");
    *out = nullptr;
    if (n_params < 1 || n_params > (size_t)1 << 40) return fail(nullptr, ZOA_ERR_ARG, "zoa_create: n_params out of range");
    if (W < 1 || W > kMaxWorkers) return fail(nullptr, ZOA_ERR_ARG, "zoa_create: W must be in [1, 64]");
    if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f))
        return fail(nullptr, ZOA_ERR_ARG, "zoa_create: beta1 and beta2 must be in [0, 1)");
    if (!(eps > 0.f) || !std::isfinite(eps)) return fail(nullptr, ZOA_ERR_ARG, "zoa_create: eps must be positive");
    if (chunk < 32 || chunk > (1 << 30) || chunk % 32 != 0)
        return fail(nullptr, ZOA_ERR_ARG, "zoa_create: chunk must be a multiple of 32 in [32, 2^30]");

    zoa_handle h = new (std::nothrow) zoa_handle_s;
    if (!h) return fail(nullptr, ZOA_ERR_ALLOC, "zoa_create: out of host memory");
    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
    if (e == cudaSuccess) e = configure_kernels();
    if (e != cudaSuccess) { delete h; return fail_cuda(nullptr, e, "zoa_create: device set-up"); }

    h->n = (long long)n_params;
    h->n_pad = (h->n + kRowAlign - 1) / kRowAlign * kRowAlign;
    h->W = W;
    h->chunk = chunk;
    h->n_chunks = (h->n + chunk - 1) / chunk;
    h->words_stride = h->n_pad / 32;
    h->c.b1 = beta1; h->c.ob1 = 1.0f - beta1;
    h->c.b2 = beta2; h->c.ob2 = 1.0f - beta2;
    h->c.eps = eps;

    const size_t rows = (size_t)W * (size_t)h->n_pad, row = (size_t)h->n_pad;
    h->allreduce_only = allreduce_only;
    const size_t full_rows = allreduce_only ? 0 : rows, full_row = allreduce_only ? 0 : row;   // what Algorithm 1 adds to Algorithm 3
    if ((e = alloc_zero(h, &h->x, full_rows)) == cudaSuccess && (e = alloc_zero(h, &h->m, full_rows)) == cudaSuccess &&
        (e = alloc_zero(h, &h->u, full_rows)) == cudaSuccess && (e = alloc_zero(h, &h->dw, rows)) == cudaSuccess &&
        (e = alloc_zero(h, &h->v_cur, full_row)) == cudaSuccess && (e = alloc_zero(h, &h->v_nxt, full_row)) == cudaSuccess &&
        (e = alloc_zero(h, &h->ds, row)) == cudaSuccess && (e = alloc_zero(h, &h->xs, full_row)) == cudaSuccess &&
        (e = alloc_zero(h, &h->words_w, (size_t)W * h->words_stride)) == cudaSuccess &&
        (e = alloc_zero(h, &h->words_s, (size_t)h->words_stride)) == cudaSuccess &&
        (e = alloc_zero(h, &h->scales_w, (size_t)W * h->n_chunks)) == cudaSuccess &&
        (e = alloc_zero(h, &h->scales_s, (size_t)h->n_chunks)) == cudaSuccess &&
        (e = alloc_zero(h, &h->error_flag, 1)) == cudaSuccess && (e = alloc_zero(h, &h->sched, 2)) == cudaSuccess) {
        h->large_chunk = chunk > kMaxChunk;
        if (h->large_chunk)
            e = alloc_zero(h, &h->partials, (size_t)(W + 1) * (size_t)h->n_chunks * (size_t)large_chunk_segments(view(h)));
        if (e == cudaSuccess) e = cudaHostAlloc(reinterpret_cast<void **>(&h->error_host), sizeof(int), cudaHostAllocMapped);
        if (e == cudaSuccess) {
            *h->error_host = 0;
            e = cudaHostGetDevicePointer(reinterpret_cast<void **>(&h->error_host_dev), h->error_host, 0);
        } else {
            h->error_host = nullptr;
        }
        if (e == cudaSuccess) e = cudaDeviceSynchronize();
    }
    if (e != cudaSuccess) {
        free_all(h);
        delete h;
        cudaGetLastError();
        return fail_cuda(nullptr, e, "zoa_create: allocating state");
    }
    *out = h;
    return ZOA_OK;
}

extern "C" zoa_status zoa_create(zoa_handle *out, size_t n_params, int W, float beta1, float beta2,
                                 float eps, int chunk)
{
    return create_handle(out, n_params, W, beta1, beta2, eps, chunk, false);
}

extern "C" zoa_status zoa_create_allreduce(zoa_handle *out, size_t n, int W, int chunk)
{
    if (chunk > kMaxChunk) return fail(nullptr, ZOA_ERR_ARG, "zoa_create_allreduce: chunk must be at most 16384");
    return create_handle(out, n, W, 0.f, 0.f, 1.f, chunk, true);
}

// Entry points of Algorithm 1 / Algorithm 2 need the full state.
#define ZOA_NEEDS_FULL_STATE(h, who)                                                                                    \
    do {                                                                                                                \
        if ((h)->allreduce_only)                                                                                        \
            return fail(h, ZOA_ERR_STATE, std::string(who) + ": the handle was made by zoa_create_allreduce and holds "  \
                                                             "only the state of Algorithm 3");                           \
    } while (0)

extern "C" zoa_status zoa_destroy(zoa_handle h)
{
    if (!h) return ZOA_ERR_ARG;
    int current = -1;
    const bool restore = cudaGetDevice(&current) == cudaSuccess && current != h->device;
    cudaSetDevice(h->device);
    cudaDeviceSynchronize();
    free_all(h);
    delete h;
    if (restore) cudaSetDevice(current);      // the caller's current device stays what it was
    return ZOA_OK;
}

extern "C" zoa_status zoa_set_params(zoa_handle h, const float *x0, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    ZOA_NEEDS_FULL_STATE(h, "zoa_set_params");
    if (!x0) return fail(h, ZOA_ERR_ARG, "zoa_set_params: x0 is NULL");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_set_params: the handle's device is not the current CUDA device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t bytes = (size_t)h->n * sizeof(float);
    for (int i = 0; i < h->W; ++i)
        ZOA_CUDA(h, cudaMemcpyAsync(h->x + (size_t)i * h->n_pad, x0, bytes, cudaMemcpyDeviceToDevice, s));
    ZOA_CUDA(h, cudaMemcpyAsync(h->xs, x0, bytes, cudaMemcpyDeviceToDevice, s));
    return ZOA_OK;
}

extern "C" zoa_status zoa_set_var_steps(zoa_handle h, const int64_t *steps, size_t count)
{
    if (!h) return ZOA_ERR_ARG;
    if (count && !steps) return fail(h, ZOA_ERR_ARG, "zoa_set_var_steps: steps is NULL");
    for (size_t k = 0; k < count; ++k)
        if (steps[k] < 0) return fail(h, ZOA_ERR_ARG, "zoa_set_var_steps: negative step index");
    h->var_steps.assign(steps, steps + count);
    std::sort(h->var_steps.begin(), h->var_steps.end());
    h->var_steps.erase(std::unique(h->var_steps.begin(), h->var_steps.end()), h->var_steps.end());
    return ZOA_OK;
}

// ---- the paper's schedules as plain host functions (no handle, no GPU) ----------------------

// T_v: k_0 = 0, k_{j+1} - k_j = 2^floor(j / kappa), for k_j < freeze_at.
extern "C" size_t zoa_policy_var_steps(int kappa, int64_t freeze_at, int64_t *out, size_t capacity)
{
    if (kappa < 1 || freeze_at < 0) return 0;
    size_t count = 0;
    int64_t k = 0;
    for (int64_t j = 0; k < freeze_at; ++j) {
        if (out && count < capacity) out[count] = k;
        ++count;
        const int64_t e = j / kappa;
        if (e >= 62) break;
        k += (int64_t)1 << e;
    }
    return count;
}

// T_u: the interval between syncs is 1 through the warm-up and then doubles every `double_every`
// steps, as the learning rate halves: interval(t) = min(2^floor((t - warmup) / double_every), max_interval)
// for t >= warmup.  Written as pieces (boundary, interval).
extern "C" size_t zoa_policy_sync_pieces(int64_t warmup, int64_t double_every, int32_t max_interval,
                                         int64_t *boundaries, int32_t *intervals, size_t capacity)
{
    if (warmup < 0 || double_every < 1 || max_interval < 1) return 0;
    size_t count = 0;
    auto push = [&](int64_t b, int32_t k) {
        if (boundaries && intervals && count < capacity) { boundaries[count] = b; intervals[count] = k; }
        ++count;
    };
    push(0, 1);
    int32_t interval = 1;
    for (int64_t r = 1; interval < max_interval; ++r) {
        interval = interval > max_interval / 2 ? max_interval : interval * 2;
        push(warmup + r * double_every, interval);
    }
    return count;
}

extern "C" zoa_status zoa_set_var_policy_doubling(zoa_handle h, int kappa, int64_t freeze_at)
{
    if (!h) return ZOA_ERR_ARG;
    if (kappa < 1 || freeze_at < 0) return fail(h, ZOA_ERR_ARG, "zoa_set_var_policy_doubling: kappa >= 1, freeze_at >= 0");
    const size_t count = zoa_policy_var_steps(kappa, freeze_at, nullptr, 0);
    h->var_steps.assign(count, 0);
    zoa_policy_var_steps(kappa, freeze_at, h->var_steps.data(), count);
    return ZOA_OK;
}

extern "C" zoa_status zoa_set_sync_policy_doubling(zoa_handle h, int64_t warmup, int64_t double_every,
                                                   int32_t max_interval, int freeze_variance)
{
    if (!h) return ZOA_ERR_ARG;
    const size_t count = zoa_policy_sync_pieces(warmup, double_every, max_interval, nullptr, nullptr, 0);
    if (count == 0) return fail(h, ZOA_ERR_ARG, "zoa_set_sync_policy_doubling: warmup >= 0, double_every >= 1, max_interval >= 1");
    h->sync_bounds.assign(count, 0);
    h->sync_intervals.assign(count, 1);
    zoa_policy_sync_pieces(warmup, double_every, max_interval, h->sync_bounds.data(), h->sync_intervals.data(), count);
    if (freeze_variance) {
        // no variance updates once the interval between syncs exceeds 1
        int64_t first_sparse = -1;
        for (size_t r = 0; r < count; ++r)
            if (h->sync_intervals[r] > 1) { first_sparse = h->sync_bounds[r]; break; }
        if (first_sparse >= 0)
            h->var_steps.erase(std::lower_bound(h->var_steps.begin(), h->var_steps.end(), first_sparse), h->var_steps.end());
    }
    return ZOA_OK;
}

extern "C" zoa_status zoa_set_sync_policy(zoa_handle h, const int64_t *boundaries, const int32_t *intervals,
                                          size_t count)
{
    if (!h) return ZOA_ERR_ARG;
    if (count < 1 || !boundaries || !intervals) return fail(h, ZOA_ERR_ARG, "zoa_set_sync_policy: need at least one piece");
    if (boundaries[0] != 0) return fail(h, ZOA_ERR_ARG, "zoa_set_sync_policy: boundaries[0] must be 0");
    for (size_t r = 0; r < count; ++r) {
        if (intervals[r] < 1) return fail(h, ZOA_ERR_ARG, "zoa_set_sync_policy: intervals must be >= 1");
        if (r && boundaries[r] <= boundaries[r - 1]) return fail(h, ZOA_ERR_ARG, "zoa_set_sync_policy: boundaries must increase");
    }
    h->sync_bounds.assign(boundaries, boundaries + count);
    h->sync_intervals.assign(intervals, intervals + count);
    return ZOA_OK;
}

extern "C" int zoa_sync_due(zoa_handle h, int64_t t)
{
    if (!h || t < 0) return -1;
    size_t r = std::upper_bound(h->sync_bounds.begin(), h->sync_bounds.end(), t) - h->sync_bounds.begin() - 1;
    return (t - h->sync_bounds[r]) % h->sync_intervals[r] == 0 ? 1 : 0;
}

extern "C" int zoa_var_due(zoa_handle h, int64_t t)
{
    if (!h || t < 0) return -1;
    return std::binary_search(h->var_steps.begin(), h->var_steps.end(), t) ? 1 : 0;
}

// Checks shared by the step entry points; fills the pointer pack.
static zoa_status check_step_args(zoa_handle h, const void *const *grads, float lr, int64_t t, GradPtrs *gp,
                                  int *aligned, const char *who)
{
    if (!h) return ZOA_ERR_ARG;
    ZOA_REFUSE_AFTER_DEVICE_ERROR(h, who);
    ZOA_NEEDS_FULL_STATE(h, who);
    if (!grads) return fail(h, ZOA_ERR_ARG, std::string(who) + ": grads is NULL");
    if (!std::isfinite(lr)) return fail(h, ZOA_ERR_ARG, std::string(who) + ": lr is not finite");
    if (t < 0) return fail(h, ZOA_ERR_ARG, std::string(who) + ": t is negative");
    if (t <= h->t_last) return fail(h, ZOA_ERR_STATE, std::string(who) + ": t must increase from step to step");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, std::string(who) + ": the handle's device is not the current CUDA device");
    bool all_aligned = true;
    for (int i = 0; i < h->W; ++i) {
        if (!grads[i]) return fail(h, ZOA_ERR_ARG, std::string(who) + ": a gradient pointer is NULL");
        gp->p[i] = static_cast<const float *>(grads[i]);
        if (reinterpret_cast<uintptr_t>(grads[i]) & 15u) all_aligned = false;
    }
    for (int i = h->W; i < kMaxWorkers; ++i) gp->p[i] = nullptr;
    *aligned = (all_aligned ? kGradAligned : 0) | (h->grad_type << 1);   // the format code ld_grad4 takes
    return ZOA_OK;
}

static bool on_own_device(zoa_handle h)
{
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == h->device;
}

static void commit_variance(zoa_handle h)
{
    if (h->v_pending) {
        std::swap(h->v_cur, h->v_nxt);
        h->v_pending = false;
    }
}

// Brings the error rows of a large-chunk handle to their plain form before anything outside the
// large-chunk kernels reads or writes them.  Synchronises.
static cudaError_t plain_errors(zoa_handle h)
{
    if (!h->dw_pending && !h->ds_pending) return cudaSuccess;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = launch_plain_errors(view(h), h->dw_pending, h->ds_pending, nullptr);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e == cudaSuccess) {
        h->n_launches += (h->dw_pending ? 1 : 0) + (h->ds_pending ? 1 : 0);
        h->dw_pending = h->ds_pending = false;
    }
    return e;
}

// Worker side / server side of the 1-bit AllReduce of u, by the kernels that fit the chunk size.
static cudaError_t run_compress(zoa_handle h, cudaStream_t s)
{
    int launches = 0;
    cudaError_t e;
    if (h->large_chunk) {
        GradPtrs none{};
        e = launch_large_compress(view(h), none, h->c, 0.f, 0, kGradAligned, h->dw_pending, h->partials, &launches, s);
        h->dw_pending = true;
    } else {
        e = launch_compress(view(h), 0, h->n_chunks, s);
        launches = 1;
    }
    h->n_launches += launches;
    return e;
}
static cudaError_t run_server(zoa_handle h, float gamma_sum, cudaStream_t s)
{
    int launches = 0;
    cudaError_t e;
    if (h->large_chunk) {
        e = launch_large_server(view(h), h->c, 1, gamma_sum, h->ds_pending, h->partials, &launches, s);
        h->ds_pending = true;
    } else {
        const StateView st = view(h);
        long long n_units = 0, first = 0;
        const int stages = h->use_pipeline ? reduce_pipeline_stages(st, &n_units) : 0;
        e = cudaSuccess;
        if (stages > 0 && (h->use_pipeline == 2 || n_units >= 4ll * h->sm_count)) {
            e = launch_reduce_pipelined(st, h->c, gamma_sum, n_units, stages, h->sm_count, error_words(h), h->sched,
                                        (unsigned long long)h->wait_limit_ms * 1000000ull, h->test_stop_after_tiles, s);
            ++launches;
            first = n_units * std::max<long long>(h->chunk, 2048) / h->chunk;
        }
        if (e == cudaSuccess && first < h->n_chunks) {
            e = launch_reduce(st, h->c, gamma_sum, first, h->n_chunks - first, s);
            ++launches;
        }
    }
    h->n_launches += launches;
    return e;
}

// The local updates of Algorithm 1 (+ the variance update) for the chunks [c0, c1).
static zoa_status run_local_range(zoa_handle h, const StateView &st, const GradPtrs &gp, float lr, bool do_var, int fmt,
                                  long long c0, long long c1, cudaStream_t s)
{
    long long e0 = c0 * h->chunk;
    const long long e1 = std::min<long long>(c1 * (long long)h->chunk, h->n);
    // whole tiles of 2048 coordinates through the ring kernel (aligned gradients, a tile-aligned start,
    // enough tiles to feed every SM), the rest one float4 per thread
    const long long n_units = (e0 % 2048 == 0 && (fmt & kGradAligned)) ? (e1 - e0) / 2048 : 0;
    if (h->use_pipeline && (h->use_pipeline == 2 || n_units >= 4ll * h->sm_count) && n_units > 0) {
        ZOA_CUDA(h, launch_local_step_pipelined(st, gp, h->c, lr, do_var, fmt, e0 / 2048, n_units, h->sm_count, error_words(h), h->sched,
                                                (unsigned long long)h->wait_limit_ms * 1000000ull, h->test_stop_after_tiles, s));
        h->n_launches += 1;
        e0 += n_units * 2048;
    }
    if (e0 < e1) {
        ZOA_CUDA(h, launch_local_step(st, gp, h->c, lr, do_var, fmt, e0, e1, s));
        h->n_launches += 1;
    }
    return ZOA_OK;
}

// A whole sync step (chunks up to 16384) for the chunks [c0, c1): the bulk-copy ring for the
// full chunks where it applies, the chunk-per-block kernel for the rest, the variance update
// fused or beside it.
static zoa_status run_sync_range(zoa_handle h, const StateView &st, const GradPtrs &gp, float lr, float gamma_sum,
                                 bool do_var, int fmt, long long c0, long long c1, cudaStream_t s)
{
    const long long e0 = c0 * h->chunk, e1 = std::min<long long>(c1 * (long long)h->chunk, h->n);
    const bool ragged = c1 == h->n_chunks && h->n % h->chunk != 0;
    // The ring kernel takes whole units (one chunk of 2048 coordinates or more, or the G smaller chunks of
    // a tile) from a unit boundary; the chunks left over go to the chunk-per-block kernel.
    const int G = pipeline_chunks_per_unit(st);
    const long long n_units = c0 % G == 0 ? (c1 - c0 - (ragged ? 1 : 0)) / G : 0;
    // The persistent kernel pays off once every SM has a few units to stream; below that the
    // one-block-per-chunk kernel starts faster (measured on a 512-chunk problem).
    const bool enough = h->use_pipeline == 2 || n_units >= 4ll * h->sm_count;
    const int stages = h->use_pipeline && enough && n_units > 0 ? pipeline_stages(st, fmt) : 0;
    long long var_first = e0;     // coordinates from here to e1 still need the variance update
    if (stages > 0) {
        bool var_fused = false;
        ZOA_CUDA(h, launch_step_sync_pipelined(st, gp, h->c, lr, gamma_sum, do_var, fmt, c0 / G, n_units, stages, h->sm_count,
                                               error_words(h), h->sched, (unsigned long long)h->wait_limit_ms * 1000000ull,
                                               h->test_stop_after_tiles, &var_fused, s));
        h->n_launches += 1;
        const long long done = c0 + n_units * G;      // first chunk the ring kernel did not take
        if (done < c1) {
            ZOA_CUDA(h, launch_step_sync(st, gp, h->c, lr, gamma_sum, fmt, done, c1 - done, s));
            h->n_launches += 1;
        }
        if (var_fused) var_first = done * h->chunk;
    } else {
        ZOA_CUDA(h, launch_step_sync(st, gp, h->c, lr, gamma_sum, fmt, c0, c1 - c0, s));
        h->n_launches += 1;
    }
    if (do_var && var_first < e1) {
        ZOA_CUDA(h, launch_variance(st, gp, h->c, fmt, var_first, e1, s));
        h->n_launches += 1;
    }
    return ZOA_OK;
}

extern "C" zoa_status zoa_step(zoa_handle h, const void *const *grads, float lr, int64_t t, void *stream)
{
    TraceRange trace("zoa_step");
    GradPtrs gp;
    int aligned;   // gradient format code: alignment bit and element type
    zoa_status rc = check_step_args(h, grads, lr, t, &gp, &aligned, "zoa_step");
    if (rc != ZOA_OK) return rc;
    commit_variance(h);
    const bool do_var = zoa_var_due(h, t) == 1;
    rc = run_local_range(h, view(h), gp, lr, do_var, aligned, 0, h->n_chunks, static_cast<cudaStream_t>(stream));
    if (rc != ZOA_OK) return rc;
    h->gamma_sum += (double)lr;
    if (do_var) { h->v_pending = true; h->n_var_updates += 1; }
    h->t_last = t;
    h->n_steps += 1;
    return ZOA_OK;
}

extern "C" zoa_status zoa_onebit_reduce(zoa_handle h, void *stream)
{
    TraceRange trace("zoa_onebit_reduce");
    if (!h) return ZOA_ERR_ARG;
    ZOA_REFUSE_AFTER_DEVICE_ERROR(h, "zoa_onebit_reduce");
    ZOA_NEEDS_FULL_STATE(h, "zoa_onebit_reduce");
    const float gamma_sum = (float)h->gamma_sum;
    if (!(h->gamma_sum > 0.0) || !(gamma_sum > 0.f) || !std::isfinite(gamma_sum))
        return fail(h, ZOA_ERR_STATE, "zoa_onebit_reduce: nothing accumulated since the last sync (sum of learning rates is not positive)");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_onebit_reduce: the handle's device is not the current CUDA device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    ZOA_CUDA(h, run_compress(h, s));
    ZOA_CUDA(h, run_server(h, gamma_sum, s));
    h->gamma_sum = 0.0;
    h->t_sync = h->t_last;
    h->n_syncs += 1;
    return ZOA_OK;
}

extern "C" zoa_status zoa_onebit_compress(zoa_handle h, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    ZOA_REFUSE_AFTER_DEVICE_ERROR(h, "zoa_onebit_compress");
    ZOA_NEEDS_FULL_STATE(h, "zoa_onebit_compress");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_onebit_compress: the handle's device is not the current CUDA device");
    ZOA_CUDA(h, run_compress(h, static_cast<cudaStream_t>(stream)));
    return ZOA_OK;
}

extern "C" zoa_status zoa_onebit_average(zoa_handle h, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    const float gamma_sum = (float)h->gamma_sum;
    if (!(h->gamma_sum > 0.0) || !(gamma_sum > 0.f) || !std::isfinite(gamma_sum))
        return fail(h, ZOA_ERR_STATE, "zoa_onebit_average: nothing accumulated since the last sync (sum of learning rates is not positive)");
    ZOA_REFUSE_AFTER_DEVICE_ERROR(h, "zoa_onebit_average");
    ZOA_NEEDS_FULL_STATE(h, "zoa_onebit_average");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_onebit_average: the handle's device is not the current CUDA device");
    ZOA_CUDA(h, run_server(h, gamma_sum, static_cast<cudaStream_t>(stream)));
    h->gamma_sum = 0.0;
    h->t_sync = h->t_last;
    h->n_syncs += 1;
    return ZOA_OK;
}

// Server side of Algorithm 3 alone for the chunks [first, first + count) of packed buffers that start at
// chunk `first`: the prefetching kernel for the whole chunks where the buffers allow it, the plain
// one-block-per-chunk kernel for a ragged last chunk and every other case.
static zoa_status run_server_alone(zoa_handle h, const uint32_t *words_in, long long words_stride, const float *scales_in,
                                   long long scales_stride, int W_total, long long first, long long count, const PeerOut &out,
                                   float *z_bar, cudaStream_t s)
{
    const StateView st = view(h);
    const bool ragged = first + count == h->n_chunks && h->n % h->chunk != 0;
    long long whole = 0;
    if (h->use_pipeline && server_prefetch_applies(st, words_in, words_stride, W_total, z_bar)) whole = count - (ragged ? 1 : 0);
    if (whole > 0) {
        ZOA_CUDA(h, launch_server_prefetch(st, words_in, words_stride, scales_in, scales_stride, W_total, first, whole, out, z_bar,
                                           error_words(h), (unsigned long long)h->wait_limit_ms * 1000000ull,
                                           h->test_stop_after_tiles > 0, s));
        h->n_launches += 1;
    }
    if (whole < count) {
        ZOA_CUDA(h, launch_dist_server(st, words_in + (whole * h->chunk >> 5), words_stride, scales_in + whole, scales_stride, W_total,
                                       first + whole, count - whole, out, z_bar, s));
        h->n_launches += 1;
    }
    return ZOA_OK;
}

// ---- Algorithm 3 on caller-owned buffers, with the handle's errors and wire buffers ---------------

static zoa_status allreduce_compress(zoa_handle h, const float *const *z, cudaStream_t s, const char *who)
{
    ZOA_REFUSE_AFTER_DEVICE_ERROR(h, who);
    if (h->large_chunk) return fail(h, ZOA_ERR_ARG, std::string(who) + ": chunk must be at most 16384");
    if (!z) return fail(h, ZOA_ERR_ARG, std::string(who) + ": z is NULL");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, std::string(who) + ": the handle's device is not the current CUDA device");
    GradPtrs zp{};
    bool aligned = true;
    for (int i = 0; i < h->W; ++i) {
        if (!z[i]) return fail(h, ZOA_ERR_ARG, std::string(who) + ": a buffer pointer is NULL");
        zp.p[i] = z[i];
        if (reinterpret_cast<uintptr_t>(z[i]) & 15u) aligned = false;
    }
    ZOA_CUDA(h, launch_compress_external(view(h), zp, aligned ? kGradAligned : 0, s));
    h->n_launches += 1;
    return ZOA_OK;
}

static zoa_status allreduce_average(zoa_handle h, float *z_bar, cudaStream_t s, const char *who)
{
    ZOA_REFUSE_AFTER_DEVICE_ERROR(h, who);
    if (h->large_chunk) return fail(h, ZOA_ERR_ARG, std::string(who) + ": chunk must be at most 16384");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, std::string(who) + ": the handle's device is not the current CUDA device");
    PeerOut none{};
    return run_server_alone(h, h->words_w, h->words_stride, h->scales_w, h->n_chunks, h->W, 0, h->n_chunks, none, z_bar, s);
}

extern "C" zoa_status zoa_allreduce_compress(zoa_handle h, const float *const *z, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    return allreduce_compress(h, z, static_cast<cudaStream_t>(stream), "zoa_allreduce_compress");
}

extern "C" zoa_status zoa_allreduce_average(zoa_handle h, float *z_bar, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    return allreduce_average(h, z_bar, static_cast<cudaStream_t>(stream), "zoa_allreduce_average");
}

extern "C" zoa_status zoa_onebit_allreduce(zoa_handle h, const float *const *z, float *z_bar, void *stream)
{
    TraceRange trace("zoa_onebit_allreduce");
    if (!h) return ZOA_ERR_ARG;
    if (!z_bar) return fail(h, ZOA_ERR_ARG, "zoa_onebit_allreduce: z_bar is NULL");
    zoa_status rc = allreduce_compress(h, z, static_cast<cudaStream_t>(stream), "zoa_onebit_allreduce");
    if (rc != ZOA_OK) return rc;
    rc = allreduce_average(h, z_bar, static_cast<cudaStream_t>(stream), "zoa_onebit_allreduce");
    if (rc == ZOA_OK) h->n_syncs += 1;
    return rc;
}

// ---- one worker per GPU: the pieces between the collectives ------------------------------------

extern "C" zoa_status zoa_dist_server_range(zoa_handle h, const uint32_t *words_all, size_t words_stride,
                                            const float *scales_all, size_t scales_stride, int W_total,
                                            int64_t first_chunk, int64_t n_chunks, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    if (h->large_chunk) return fail(h, ZOA_ERR_ARG, "zoa_dist_server_range: chunk must be at most 16384");
    if (W_total < 1 || W_total > kMaxWorkers) return fail(h, ZOA_ERR_ARG, "zoa_dist_server_range: W_total must be in [1, 64]");
    if (first_chunk < 0 || n_chunks < 0 || first_chunk + n_chunks > h->n_chunks)
        return fail(h, ZOA_ERR_ARG, "zoa_dist_server_range: chunk range outside the vector");
    if (n_chunks == 0) return ZOA_OK;
    if (!words_all || !scales_all) return fail(h, ZOA_ERR_ARG, "zoa_dist_server_range: NULL buffer");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_dist_server_range: the handle's device is not the current CUDA device");
    ZOA_REFUSE_AFTER_DEVICE_ERROR(h, "zoa_dist_server_range");
    PeerOut none{};
    return run_server_alone(h, words_all, (long long)words_stride, scales_all, (long long)scales_stride, W_total, first_chunk, n_chunks,
                            none, nullptr, static_cast<cudaStream_t>(stream));
}

extern "C" zoa_status zoa_dist_server_push(zoa_handle h, const uint32_t *words_all, size_t words_stride,
                                           const float *scales_all, size_t scales_stride, int W_total,
                                           int64_t first_chunk, int64_t n_chunks, int world,
                                           void *const *peer_words_s, void *const *peer_scales_s, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    if (h->large_chunk) return fail(h, ZOA_ERR_ARG, "zoa_dist_server_push: chunk must be at most 16384");
    if (W_total < 1 || W_total > kMaxWorkers) return fail(h, ZOA_ERR_ARG, "zoa_dist_server_push: W_total must be in [1, 64]");
    if (world < 1 || world > kMaxWorkers) return fail(h, ZOA_ERR_ARG, "zoa_dist_server_push: world must be in [1, 64]");
    if (first_chunk < 0 || n_chunks < 0 || first_chunk + n_chunks > h->n_chunks)
        return fail(h, ZOA_ERR_ARG, "zoa_dist_server_push: chunk range outside the vector");
    if (!peer_words_s || !peer_scales_s) return fail(h, ZOA_ERR_ARG, "zoa_dist_server_push: NULL pointer table");
    PeerOut out{};
    out.world = world;
    for (int r = 0; r < world; ++r) {
        if (!peer_words_s[r] || !peer_scales_s[r]) return fail(h, ZOA_ERR_ARG, "zoa_dist_server_push: a peer pointer is NULL");
        out.words_s[r] = static_cast<uint32_t *>(peer_words_s[r]);
        out.scales_s[r] = static_cast<float *>(peer_scales_s[r]);
    }
    if (n_chunks == 0) return ZOA_OK;
    if (!words_all || !scales_all) return fail(h, ZOA_ERR_ARG, "zoa_dist_server_push: NULL buffer");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_dist_server_push: the handle's device is not the current CUDA device");
    ZOA_REFUSE_AFTER_DEVICE_ERROR(h, "zoa_dist_server_push");
    return run_server_alone(h, words_all, (long long)words_stride, scales_all, (long long)scales_stride, W_total, first_chunk, n_chunks,
                            out, nullptr, static_cast<cudaStream_t>(stream));
}

// The table of a rank's destinations, checked: the ranges tile the chunks in rank order and
// every rank that serves a chunk has both pointers.
static zoa_status make_push_plan(zoa_handle h, int world, const int64_t *chunk_begin, void *const *peer_words,
                                 void *const *peer_scales, PushPlan *plan, const char *who)
{
    ZOA_NEEDS_FULL_STATE(h, who);
    if (h->W != 1) return fail(h, ZOA_ERR_ARG, std::string(who) + ": the handle must hold exactly one worker");
    if (h->large_chunk) return fail(h, ZOA_ERR_ARG, std::string(who) + ": chunk must be at most 16384");
    if (world < 1 || world > kMaxWorkers) return fail(h, ZOA_ERR_ARG, std::string(who) + ": world must be in [1, 64]");
    if (!chunk_begin || !peer_words || !peer_scales) return fail(h, ZOA_ERR_ARG, std::string(who) + ": NULL table");
    if (chunk_begin[0] != 0 || chunk_begin[world] != h->n_chunks)
        return fail(h, ZOA_ERR_ARG, std::string(who) + ": chunk_begin must run from 0 to the number of chunks");
    *plan = PushPlan{};
    plan->world = world;
    for (int r = 0; r < world; ++r) {
        if (chunk_begin[r + 1] < chunk_begin[r]) return fail(h, ZOA_ERR_ARG, std::string(who) + ": chunk_begin must not decrease");
        if (chunk_begin[r + 1] > chunk_begin[r] && (!peer_words[r] || !peer_scales[r]))
            return fail(h, ZOA_ERR_ARG, std::string(who) + ": a rank that serves chunks has a NULL pointer");
        plan->chunk_begin[r] = chunk_begin[r];
        plan->words[r] = static_cast<uint32_t *>(peer_words[r]);
        plan->scales[r] = static_cast<float *>(peer_scales[r]);
    }
    plan->chunk_begin[world] = chunk_begin[world];
    return ZOA_OK;
}

extern "C" zoa_status zoa_dist_pack_push(zoa_handle h, int world, const int64_t *chunk_begin,
                                         void *const *peer_words, void *const *peer_scales, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    PushPlan plan;
    zoa_status rc = make_push_plan(h, world, chunk_begin, peer_words, peer_scales, &plan, "zoa_dist_pack_push");
    if (rc != ZOA_OK) return rc;
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_dist_pack_push: the handle's device is not the current CUDA device");
    ZOA_CUDA(h, launch_dist_pack_push(view(h), nullptr, h->c, 0.f, 0, plan, static_cast<cudaStream_t>(stream)));
    h->n_launches += 1;
    return ZOA_OK;
}

extern "C" zoa_status zoa_dist_step_pack_push(zoa_handle h, const void *grad, float lr, int64_t t, int world,
                                              const int64_t *chunk_begin, void *const *peer_words,
                                              void *const *peer_scales, void *stream)
{
    TraceRange trace("zoa_dist_step_pack_push");
    if (!h) return ZOA_ERR_ARG;
    PushPlan plan;
    zoa_status rc = make_push_plan(h, world, chunk_begin, peer_words, peer_scales, &plan, "zoa_dist_step_pack_push");
    if (rc != ZOA_OK) return rc;
    GradPtrs gp;
    int fmt;
    const void *grads[1] = {grad};
    rc = check_step_args(h, grads, lr, t, &gp, &fmt, "zoa_dist_step_pack_push");
    if (rc != ZOA_OK) return rc;
    const double total = h->gamma_sum + (double)lr;
    if (!(total > 0.0) || !((float)total > 0.f) || !std::isfinite((float)total))
        return fail(h, ZOA_ERR_STATE, "zoa_dist_step_pack_push: sum of learning rates since the last sync is not positive");
    commit_variance(h);
    ZOA_CUDA(h, launch_dist_pack_push(view(h), gp.p[0], h->c, lr, fmt, plan, static_cast<cudaStream_t>(stream)));
    h->n_launches += 1;
    h->gamma_sum = total;
    h->t_last = t;
    h->n_steps += 1;
    return ZOA_OK;
}

extern "C" zoa_status zoa_dist_apply(zoa_handle h, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    ZOA_NEEDS_FULL_STATE(h, "zoa_dist_apply");
    const float gamma_sum = (float)h->gamma_sum;
    if (!(h->gamma_sum > 0.0) || !(gamma_sum > 0.f) || !std::isfinite(gamma_sum))
        return fail(h, ZOA_ERR_STATE, "zoa_dist_apply: nothing accumulated since the last sync (sum of learning rates is not positive)");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_dist_apply: the handle's device is not the current CUDA device");
    ZOA_CUDA(h, launch_dist_apply(view(h), h->c, gamma_sum, static_cast<cudaStream_t>(stream)));
    h->n_launches += 1;
    h->gamma_sum = 0.0;
    h->t_sync = h->t_last;
    h->n_syncs += 1;
    return ZOA_OK;
}

extern "C" zoa_status zoa_dist_variance(zoa_handle h, const float *g_bar, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    ZOA_NEEDS_FULL_STATE(h, "zoa_dist_variance");
    if (!g_bar) return fail(h, ZOA_ERR_ARG, "zoa_dist_variance: g_bar is NULL");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_dist_variance: the handle's device is not the current CUDA device");
    if (h->v_pending) return fail(h, ZOA_ERR_STATE, "zoa_dist_variance: a variance update is already pending for this step");
    ZOA_CUDA(h, launch_dist_variance(view(h), h->c, g_bar, static_cast<cudaStream_t>(stream)));
    h->n_launches += 1;
    h->v_pending = true;
    h->n_var_updates += 1;
    return ZOA_OK;
}

extern "C" zoa_status zoa_step_sync(zoa_handle h, const void *const *grads, float lr, int64_t t, void *stream)
{
    TraceRange trace("zoa_step_sync");
    GradPtrs gp;
    int aligned;   // gradient format code: alignment bit and element type
    zoa_status rc = check_step_args(h, grads, lr, t, &gp, &aligned, "zoa_step_sync");
    if (rc != ZOA_OK) return rc;
    const double total = h->gamma_sum + (double)lr;
    const float gamma_sum = (float)total;
    if (!(total > 0.0) || !(gamma_sum > 0.f) || !std::isfinite(gamma_sum))
        return fail(h, ZOA_ERR_STATE, "zoa_step_sync: sum of learning rates since the last sync is not positive");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    commit_variance(h);
    const bool do_var = zoa_var_due(h, t) == 1;
    const StateView st = view(h);
    if (h->large_chunk) {
        // No single block can hold a chunk: the multi-pass kernels form the half-step buffer on the
        // fly (twice), so m, x, u are written once, by the server pass.
        int launches = 0;
        ZOA_CUDA(h, launch_large_compress(st, gp, h->c, lr, 2, aligned, h->dw_pending, h->partials, &launches, s));
        h->dw_pending = true;
        h->n_launches += launches;
        ZOA_CUDA(h, run_server(h, gamma_sum, s));
        if (do_var) {
            ZOA_CUDA(h, launch_variance(st, gp, h->c, aligned, 0, h->n, s));
            h->n_launches += 1;
            h->v_pending = true;
            h->n_var_updates += 1;
        }
        h->gamma_sum = 0.0;
        h->t_last = t;
        h->t_sync = t;
        h->n_steps += 1;
        h->n_syncs += 1;
        return ZOA_OK;
    }
    rc = run_sync_range(h, st, gp, lr, gamma_sum, do_var, aligned, 0, h->n_chunks, s);
    if (rc != ZOA_OK) return rc;
    if (do_var) {
        h->v_pending = true;
        h->n_var_updates += 1;
    }
    h->gamma_sum = 0.0;
    h->t_last = t;
    h->t_sync = t;
    h->n_steps += 1;
    h->n_syncs += 1;
    return ZOA_OK;
}

extern "C" zoa_status zoa_alg2_step(zoa_handle h, const void *const *grads, float lr, int64_t t, void *stream)
{
    TraceRange trace("zoa_alg2_step");
    GradPtrs gp;
    int aligned;   // gradient format code: alignment bit and element type
    zoa_status rc = check_step_args(h, grads, lr, t, &gp, &aligned, "zoa_alg2_step");
    if (rc != ZOA_OK) return rc;
    commit_variance(h);
    const bool full = zoa_var_due(h, t) == 1;
    if (h->large_chunk && !full) {
        int launches = 0;
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        ZOA_CUDA(h, launch_large_compress(view(h), gp, h->c, lr, 1, aligned, h->dw_pending, h->partials, &launches, s));
        h->dw_pending = true;
        ZOA_CUDA(h, launch_large_server(view(h), h->c, 2, lr, h->ds_pending, h->partials, &launches, s));
        h->ds_pending = true;
        h->n_launches += launches;
    } else {
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        const StateView st = view(h);
        const bool enough_chunks = h->use_pipeline == 2 || h->n / h->chunk >= 4ll * h->sm_count;
        const int stages = (!full && h->use_pipeline && enough_chunks) ? alg2_pipeline_stages(st, aligned) : 0;
        long long first = 0;
        if (stages > 0) {   // full chunks through the bulk-copy ring, a ragged last chunk through the block kernel
            ZOA_CUDA(h, launch_alg2_pipelined(st, gp, h->c, lr, aligned, stages, h->sm_count, error_words(h), h->sched,
                                              (unsigned long long)h->wait_limit_ms * 1000000ull, h->test_stop_after_tiles, s));
            h->n_launches += 1;
            first = h->n / h->chunk;
        }
        if (full || first < h->n_chunks) {
            ZOA_CUDA(h, launch_alg2(st, gp, h->c, lr, full, aligned, first, h->n_chunks - first, s));
            h->n_launches += 1;
        }
    }
    if (full) { h->v_pending = true; h->n_var_updates += 1; } else h->n_syncs += 1;
    h->t_last = t;
    h->n_steps += 1;
    return ZOA_OK;
}

extern "C" zoa_status zoa_step_auto(zoa_handle h, const void *const *grads, float lr, int64_t t, void *stream)
{
    if (!h) return ZOA_ERR_ARG;
    return zoa_sync_due(h, t) == 1 ? zoa_step_sync(h, grads, lr, t, stream) : zoa_step(h, grads, lr, t, stream);
}

extern "C" zoa_status zoa_step_host(zoa_handle h, const void *const *host_grads, float lr, int64_t t,
                                    float *host_x_out, void *stream)
{
    TraceRange trace("zoa_step_host");
    if (!h) return ZOA_ERR_ARG;
    if (!host_grads) return fail(h, ZOA_ERR_ARG, "zoa_step_host: host_grads is NULL");
    for (int i = 0; i < h->W; ++i)
        if (!host_grads[i]) return fail(h, ZOA_ERR_ARG, "zoa_step_host: a gradient pointer is NULL");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_step_host: the handle's device is not the current CUDA device");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!h->staging) {
        cudaError_t e = cudaMalloc(reinterpret_cast<void **>(&h->staging), (size_t)h->W * h->n_pad * sizeof(float));
        if (e != cudaSuccess) { h->staging = nullptr; cudaGetLastError(); return fail_cuda(h, e, "zoa_step_host: staging area"); }
    }
    const void *dev[kMaxWorkers];
    for (int i = 0; i < h->W; ++i) dev[i] = h->staging + (size_t)i * h->n_pad;
    const size_t g_bytes = h->grad_type ? 2 : 4;

    // Everything is validated before the first copy is enqueued.
    GradPtrs gp;
    int fmt;
    zoa_status rc = check_step_args(h, dev, lr, t, &gp, &fmt, "zoa_step_host");
    if (rc != ZOA_OK) return rc;
    const bool do_sync = zoa_sync_due(h, t) == 1;
    const double total = h->gamma_sum + (double)lr;
    const float gamma_sum = (float)total;
    if (do_sync && (!(total > 0.0) || !(gamma_sum > 0.f) || !std::isfinite(gamma_sum)))
        return fail(h, ZOA_ERR_STATE, "zoa_step_host: sum of learning rates since the last sync is not positive");

    // Large chunks are not cut into ranges, and small problems are not worth it: copy, then step.
    const int kSegments = 8;
    if (h->large_chunk || h->n_chunks < 64 * kSegments) {
        for (int i = 0; i < h->W; ++i)
            ZOA_CUDA(h, cudaMemcpyAsync(const_cast<void *>(dev[i]), host_grads[i], (size_t)h->n * g_bytes, cudaMemcpyHostToDevice, s));
        rc = zoa_step_auto(h, dev, lr, t, stream);
        if (rc != ZOA_OK) return rc;
        if (host_x_out)
            ZOA_CUDA(h, cudaMemcpyAsync(host_x_out, h->x, (size_t)h->n * sizeof(float), cudaMemcpyDeviceToHost, s));
        return ZOA_OK;
    }

    // Otherwise the vector is cut into chunk ranges: the copies of range k+1 (on the handle's own copy
    // stream) run while the kernels of range k and the copy of its part of the result (on the
    // caller's stream) do, so the step costs little more than moving the gradients over the bus.
    if (!h->copy_stream) ZOA_CUDA(h, cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
    while ((int)h->copy_events.size() < kSegments + 1) {
        cudaEvent_t e;
        ZOA_CUDA(h, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        h->copy_events.push_back(e);
    }
    // the staging area may still be read by the caller's stream (the previous step)
    ZOA_CUDA(h, cudaEventRecord(h->copy_events[kSegments], s));
    ZOA_CUDA(h, cudaStreamWaitEvent(h->copy_stream, h->copy_events[kSegments], 0));
    commit_variance(h);
    const bool do_var = zoa_var_due(h, t) == 1;
    const StateView st = view(h);
    for (int k = 0; k < kSegments; ++k) {
        // range boundaries on multiples of 16 chunks, so that every range starts on a unit of the ring kernels
        const long long c0 = h->n_chunks * k / kSegments / 16 * 16;
        const long long c1 = k + 1 == kSegments ? h->n_chunks : h->n_chunks * (k + 1) / kSegments / 16 * 16;
        const long long e0 = c0 * h->chunk, e1 = std::min<long long>(c1 * (long long)h->chunk, h->n);
        for (int i = 0; i < h->W; ++i)
            ZOA_CUDA(h, cudaMemcpyAsync(reinterpret_cast<char *>(const_cast<void *>(dev[i])) + (size_t)e0 * g_bytes,
                                        static_cast<const char *>(host_grads[i]) + (size_t)e0 * g_bytes,
                                        (size_t)(e1 - e0) * g_bytes, cudaMemcpyHostToDevice, h->copy_stream));
        ZOA_CUDA(h, cudaEventRecord(h->copy_events[k], h->copy_stream));
        ZOA_CUDA(h, cudaStreamWaitEvent(s, h->copy_events[k], 0));
        rc = do_sync ? run_sync_range(h, st, gp, lr, gamma_sum, do_var, fmt, c0, c1, s)
                     : run_local_range(h, st, gp, lr, do_var, fmt, c0, c1, s);
        if (rc != ZOA_OK) return rc;
        if (host_x_out)
            ZOA_CUDA(h, cudaMemcpyAsync(host_x_out + e0, h->x + e0, (size_t)(e1 - e0) * sizeof(float), cudaMemcpyDeviceToHost, s));
    }
    if (do_var) { h->v_pending = true; h->n_var_updates += 1; }
    h->gamma_sum = do_sync ? 0.0 : total;
    h->t_last = t;
    if (do_sync) { h->t_sync = t; h->n_syncs += 1; }
    h->n_steps += 1;
    return ZOA_OK;
}

// Row base, element size and row length of a state buffer.
static zoa_status locate(zoa_handle h, zoa_buffer which, int worker, char **base, size_t *elem, size_t *len)
{
    const bool per_worker = which == ZOA_BUF_X || which == ZOA_BUF_M || which == ZOA_BUF_U ||
                            which == ZOA_BUF_DELTA_W || which == ZOA_BUF_WORDS_W || which == ZOA_BUF_SCALES_W;
    if (per_worker && (worker < 0 || worker >= h->W)) return fail(h, ZOA_ERR_ARG, "worker index out of range");
    if (h->allreduce_only && (which == ZOA_BUF_X || which == ZOA_BUF_M || which == ZOA_BUF_U || which == ZOA_BUF_V || which == ZOA_BUF_X_SYNC))
        return fail(h, ZOA_ERR_ARG, "the handle was made by zoa_create_allreduce and has no such buffer");
    const size_t i = per_worker ? (size_t)worker : 0;
    *elem = 4;
    switch (which) {
    case ZOA_BUF_X: *base = (char *)(h->x + i * h->n_pad); *len = h->n_pad; break;
    case ZOA_BUF_M: *base = (char *)(h->m + i * h->n_pad); *len = h->n_pad; break;
    case ZOA_BUF_U: *base = (char *)(h->u + i * h->n_pad); *len = h->n_pad; break;
    case ZOA_BUF_DELTA_W: *base = (char *)(h->dw + i * h->n_pad); *len = h->n_pad; break;
    case ZOA_BUF_V: *base = (char *)(h->v_pending ? h->v_nxt : h->v_cur); *len = h->n_pad; break;
    case ZOA_BUF_DELTA_S: *base = (char *)h->ds; *len = h->n_pad; break;
    case ZOA_BUF_X_SYNC: *base = (char *)h->xs; *len = h->n_pad; break;
    case ZOA_BUF_WORDS_W: *base = (char *)(h->words_w + i * h->words_stride); *len = h->words_stride; break;
    case ZOA_BUF_SCALES_W: *base = (char *)(h->scales_w + i * h->n_chunks); *len = h->n_chunks; break;
    case ZOA_BUF_WORDS_S: *base = (char *)h->words_s; *len = h->words_stride; break;
    case ZOA_BUF_SCALES_S: *base = (char *)h->scales_s; *len = h->n_chunks; break;
    default: return fail(h, ZOA_ERR_ARG, "unknown buffer");
    }
    return ZOA_OK;
}

extern "C" zoa_status zoa_get_buffer(zoa_handle h, zoa_buffer which, int worker, void **dev_ptr, size_t *n_elems)
{
    if (!h) return ZOA_ERR_ARG;
    if (!dev_ptr) return fail(h, ZOA_ERR_ARG, "zoa_get_buffer: dev_ptr is NULL");
    if (which == ZOA_BUF_DELTA_W || which == ZOA_BUF_DELTA_S) ZOA_CUDA(h, plain_errors(h));
    char *base; size_t elem, len;
    zoa_status rc = locate(h, which, worker, &base, &elem, &len);
    if (rc != ZOA_OK) return rc;
    *dev_ptr = base;
    if (n_elems) *n_elems = len;
    return ZOA_OK;
}

extern "C" zoa_status zoa_copy_out(zoa_handle h, zoa_buffer which, int worker, size_t offset, size_t count, void *host_dst)
{
    if (!h) return ZOA_ERR_ARG;
    char *base; size_t elem, len;
    zoa_status rc = locate(h, which, worker, &base, &elem, &len);
    if (rc != ZOA_OK) return rc;
    if (!host_dst || offset > len || count > len - offset) return fail(h, ZOA_ERR_ARG, "zoa_copy_out: range outside the row");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_copy_out: the handle's device is not the current CUDA device");
    if (which == ZOA_BUF_DELTA_W || which == ZOA_BUF_DELTA_S) ZOA_CUDA(h, plain_errors(h));
    ZOA_CUDA(h, cudaDeviceSynchronize());
    ZOA_CUDA(h, cudaMemcpy(host_dst, base + offset * elem, count * elem, cudaMemcpyDeviceToHost));
    return ZOA_OK;
}

extern "C" zoa_status zoa_copy_in(zoa_handle h, zoa_buffer which, int worker, size_t offset, size_t count, const void *host_src)
{
    if (!h) return ZOA_ERR_ARG;
    char *base; size_t elem, len;
    zoa_status rc = locate(h, which, worker, &base, &elem, &len);
    if (rc != ZOA_OK) return rc;
    if (!host_src || offset > len || count > len - offset) return fail(h, ZOA_ERR_ARG, "zoa_copy_in: range outside the row");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_copy_in: the handle's device is not the current CUDA device");
    if (which == ZOA_BUF_DELTA_W || which == ZOA_BUF_DELTA_S) ZOA_CUDA(h, plain_errors(h));
    ZOA_CUDA(h, cudaDeviceSynchronize());
    ZOA_CUDA(h, cudaMemcpy(base + offset * elem, host_src, count * elem, cudaMemcpyHostToDevice));
    return ZOA_OK;
}

extern "C" zoa_status zoa_set_scalars(zoa_handle h, double gamma_sum, int64_t t_sync, int64_t t_last)
{
    if (!h) return ZOA_ERR_ARG;
    if (!std::isfinite(gamma_sum) || gamma_sum < 0.0 || t_last < -1) return fail(h, ZOA_ERR_ARG, "zoa_set_scalars: bad value");
    h->gamma_sum = gamma_sum;
    h->t_sync = t_sync;
    h->t_last = t_last;
    return ZOA_OK;
}

// The names the optimizer's C interface was first drafted with; same calls.
extern "C" zoa_status zoa_set_var_policy(zoa_handle h, const int64_t *steps, size_t count)
{
    return zoa_set_var_steps(h, steps, count);
}
extern "C" zoa_status zoa_get_ptr(zoa_handle h, int what, int worker, void **dev_ptr, size_t *stride_elems)
{
    return zoa_get_buffer(h, static_cast<zoa_buffer>(what), worker, dev_ptr, stride_elems);
}

// ---- checkpoint: the whole state of Algorithm 1 / Algorithm 3 as one host blob ------------------
//
// Layout: BlobHeader, then T_v (int64 each), the T_u pieces (int64 boundaries, then int32
// intervals, padded to 8 bytes), then n floats per row: x, m, u, delta_w (W rows each),
// v_t, v_{t+1} (meaningful only when v_pending), delta_s, x_sync.
namespace {
struct BlobHeader {
    char magic[8];                 // "ZOASTATE"
    uint32_t version, header_bytes;
    int64_t n, n_chunks;
    int32_t W, chunk;
    float beta1, beta2, eps;
    int32_t v_pending;
    double gamma_sum;
    int64_t t_sync, t_last;
    int64_t n_steps, n_syncs, n_var_updates;
    uint64_t n_var_steps, n_sync_pieces;
    uint64_t total_bytes;
};
const char kBlobMagic[8] = {'Z', 'O', 'A', 'S', 'T', 'A', 'T', 'E'};
const uint32_t kBlobVersion = 1;

size_t blob_policy_bytes(size_t n_var, size_t n_pieces)
{
    return n_var * sizeof(int64_t) + n_pieces * sizeof(int64_t) + (n_pieces * sizeof(int32_t) + 7) / 8 * 8;
}
size_t blob_rows(int W) { return 4 * (size_t)W + 4; }
}  // namespace

extern "C" zoa_status zoa_state_size(zoa_handle h, size_t *bytes)
{
    if (!h) return ZOA_ERR_ARG;
    if (!bytes) return fail(h, ZOA_ERR_ARG, "zoa_state_size: bytes is NULL");
    *bytes = sizeof(BlobHeader) + blob_policy_bytes(h->var_steps.size(), h->sync_bounds.size()) +
             blob_rows(h->W) * (size_t)h->n * sizeof(float);
    return ZOA_OK;
}

extern "C" zoa_status zoa_export_state(zoa_handle h, void *host_blob, size_t bytes)
{
    if (!h) return ZOA_ERR_ARG;
    ZOA_NEEDS_FULL_STATE(h, "zoa_export_state");
    size_t need = 0;
    zoa_state_size(h, &need);
    if (!host_blob) return fail(h, ZOA_ERR_ARG, "zoa_export_state: host_blob is NULL");
    if (bytes < need) return fail(h, ZOA_ERR_ARG, "zoa_export_state: the buffer is smaller than zoa_state_size");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_export_state: the handle's device is not the current CUDA device");
    ZOA_CUDA(h, plain_errors(h));
    ZOA_CUDA(h, cudaDeviceSynchronize());
    BlobHeader hd{};
    std::memcpy(hd.magic, kBlobMagic, 8);
    hd.version = kBlobVersion;
    hd.header_bytes = (uint32_t)sizeof(BlobHeader);
    hd.n = h->n; hd.n_chunks = h->n_chunks; hd.W = h->W; hd.chunk = h->chunk;
    hd.beta1 = h->c.b1; hd.beta2 = h->c.b2; hd.eps = h->c.eps;
    hd.v_pending = h->v_pending ? 1 : 0;
    hd.gamma_sum = h->gamma_sum;
    hd.t_sync = h->t_sync; hd.t_last = h->t_last;
    hd.n_steps = h->n_steps; hd.n_syncs = h->n_syncs; hd.n_var_updates = h->n_var_updates;
    hd.n_var_steps = h->var_steps.size();
    hd.n_sync_pieces = h->sync_bounds.size();
    hd.total_bytes = need;
    char *p = static_cast<char *>(host_blob);
    std::memcpy(p, &hd, sizeof(hd));
    p += sizeof(hd);
    std::memset(p, 0, blob_policy_bytes(hd.n_var_steps, hd.n_sync_pieces));
    std::memcpy(p, h->var_steps.data(), hd.n_var_steps * sizeof(int64_t));
    p += hd.n_var_steps * sizeof(int64_t);
    std::memcpy(p, h->sync_bounds.data(), hd.n_sync_pieces * sizeof(int64_t));
    p += hd.n_sync_pieces * sizeof(int64_t);
    std::memcpy(p, h->sync_intervals.data(), hd.n_sync_pieces * sizeof(int32_t));
    p += (hd.n_sync_pieces * sizeof(int32_t) + 7) / 8 * 8;
    const size_t row_bytes = (size_t)h->n * sizeof(float);
    float *const per_worker[4] = {h->x, h->m, h->u, h->dw};
    for (float *buf : per_worker)
        for (int i = 0; i < h->W; ++i, p += row_bytes)
            ZOA_CUDA(h, cudaMemcpy(p, buf + (size_t)i * h->n_pad, row_bytes, cudaMemcpyDeviceToHost));
    float *const shared[4] = {h->v_cur, h->v_nxt, h->ds, h->xs};
    for (float *buf : shared) {
        ZOA_CUDA(h, cudaMemcpy(p, buf, row_bytes, cudaMemcpyDeviceToHost));
        p += row_bytes;
    }
    return ZOA_OK;
}

extern "C" zoa_status zoa_import_state(zoa_handle h, const void *host_blob, size_t bytes)
{
    if (!h) return ZOA_ERR_ARG;
    ZOA_NEEDS_FULL_STATE(h, "zoa_import_state");
    if (!host_blob) return fail(h, ZOA_ERR_ARG, "zoa_import_state: host_blob is NULL");
    if (bytes < sizeof(BlobHeader)) return fail(h, ZOA_ERR_ARG, "zoa_import_state: the blob is shorter than its header");
    BlobHeader hd;
    std::memcpy(&hd, host_blob, sizeof(hd));
    if (std::memcmp(hd.magic, kBlobMagic, 8) != 0 || hd.version != kBlobVersion || hd.header_bytes != sizeof(BlobHeader))
        return fail(h, ZOA_ERR_ARG, "zoa_import_state: not a state blob of this library version");
    if (hd.n != h->n || hd.W != h->W || hd.chunk != h->chunk)
        return fail(h, ZOA_ERR_ARG, "zoa_import_state: the blob was exported from a handle with another n_params, W or chunk");
    if (hd.n_var_steps > ((uint64_t)1 << 40) || hd.n_sync_pieces < 1 || hd.n_sync_pieces > ((uint64_t)1 << 40))
        return fail(h, ZOA_ERR_ARG, "zoa_import_state: malformed policy tables");
    const size_t need = sizeof(BlobHeader) + blob_policy_bytes(hd.n_var_steps, hd.n_sync_pieces) +
                        blob_rows(h->W) * (size_t)h->n * sizeof(float);
    if (hd.total_bytes != need || bytes < need) return fail(h, ZOA_ERR_ARG, "zoa_import_state: the blob is truncated");
    if (!(hd.beta1 >= 0.f && hd.beta1 < 1.f) || !(hd.beta2 >= 0.f && hd.beta2 < 1.f) || !(hd.eps > 0.f) ||
        !std::isfinite(hd.gamma_sum) || hd.gamma_sum < 0.0 || hd.t_last < -1)
        return fail(h, ZOA_ERR_ARG, "zoa_import_state: a scalar of the blob is out of range");
    const char *p = static_cast<const char *>(host_blob) + sizeof(BlobHeader);
    std::vector<int64_t> var_steps(hd.n_var_steps), bounds(hd.n_sync_pieces);
    std::vector<int32_t> intervals(hd.n_sync_pieces);
    std::memcpy(var_steps.data(), p, hd.n_var_steps * sizeof(int64_t));
    p += hd.n_var_steps * sizeof(int64_t);
    std::memcpy(bounds.data(), p, hd.n_sync_pieces * sizeof(int64_t));
    p += hd.n_sync_pieces * sizeof(int64_t);
    std::memcpy(intervals.data(), p, hd.n_sync_pieces * sizeof(int32_t));
    p += (hd.n_sync_pieces * sizeof(int32_t) + 7) / 8 * 8;
    if (bounds[0] != 0) return fail(h, ZOA_ERR_ARG, "zoa_import_state: malformed policy tables");
    for (size_t r = 0; r < bounds.size(); ++r)
        if (intervals[r] < 1 || (r && bounds[r] <= bounds[r - 1])) return fail(h, ZOA_ERR_ARG, "zoa_import_state: malformed policy tables");
    if (!std::is_sorted(var_steps.begin(), var_steps.end())) return fail(h, ZOA_ERR_ARG, "zoa_import_state: malformed policy tables");
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_import_state: the handle's device is not the current CUDA device");
    ZOA_CUDA(h, cudaDeviceSynchronize());
    // From here on the handle changes; a failing copy leaves it undefined (ZOA_ERR_CUDA).
    commit_variance(h);        // v_cur / v_nxt take their plain roles before they are overwritten
    h->dw_pending = h->ds_pending = false;      // the blob's error rows are plain
    const size_t row_bytes = (size_t)h->n * sizeof(float);
    float *const per_worker[4] = {h->x, h->m, h->u, h->dw};
    for (float *buf : per_worker)
        for (int i = 0; i < h->W; ++i, p += row_bytes)
            ZOA_CUDA(h, cudaMemcpy(buf + (size_t)i * h->n_pad, p, row_bytes, cudaMemcpyHostToDevice));
    float *const shared[4] = {h->v_cur, h->v_nxt, h->ds, h->xs};
    for (float *buf : shared) {
        ZOA_CUDA(h, cudaMemcpy(buf, p, row_bytes, cudaMemcpyHostToDevice));
        p += row_bytes;
    }
    h->c.b1 = hd.beta1; h->c.ob1 = 1.0f - hd.beta1;
    h->c.b2 = hd.beta2; h->c.ob2 = 1.0f - hd.beta2;
    h->c.eps = hd.eps;
    h->v_pending = hd.v_pending != 0;
    h->gamma_sum = hd.gamma_sum;
    h->t_sync = hd.t_sync; h->t_last = hd.t_last;
    h->n_steps = hd.n_steps; h->n_syncs = hd.n_syncs; h->n_var_updates = hd.n_var_updates;
    h->var_steps.swap(var_steps);
    h->sync_bounds.swap(bounds);
    h->sync_intervals.swap(intervals);
    return ZOA_OK;
}

extern "C" zoa_status zoa_get_stats(zoa_handle h, zoa_stats *out)
{
    if (!h || !out) return ZOA_ERR_ARG;
    out->n_steps = h->n_steps;
    out->n_syncs = h->n_syncs;
    out->n_var_updates = h->n_var_updates;
    out->n_launches = h->n_launches;
    out->bits_per_worker = h->n_syncs * (h->n + 32 * h->n_chunks);
    out->t_last = h->t_last;
    out->t_sync = h->t_sync;
    out->gamma_sum = h->gamma_sum;
    return ZOA_OK;
}

extern "C" zoa_status zoa_check_device(zoa_handle h)
{
    if (!h) return ZOA_ERR_ARG;
    ZOA_CUDA(h, cudaDeviceSynchronize());
    ZOA_CUDA(h, cudaGetLastError());
    bool intact = true;
    ZOA_CUDA(h, guards_intact(h, &intact));
    if (!intact) return fail(h, ZOA_ERR_DEVICE, "a kernel wrote outside one of the handle's buffers (guard area overwritten)");
    int flag = 0;
    ZOA_CUDA(h, cudaMemcpy(&flag, h->error_flag, sizeof(int), cudaMemcpyDeviceToHost));
    if (flag || device_gave_up(h)) {
        cudaMemset(h->error_flag, 0, sizeof(int));
        *static_cast<volatile int *>(h->error_host) = 0;
        cudaMemset(h->sched, 0, 2 * sizeof(unsigned long long));
        return fail(h, ZOA_ERR_DEVICE, "a kernel gave up waiting for its asynchronous copies; the optimizer state is undefined");
    }
    return ZOA_OK;
}

extern "C" zoa_status zoa_check_finite(zoa_handle h, int64_t *n_nonfinite)
{
    if (!h) return ZOA_ERR_ARG;
    if (!on_own_device(h)) return fail(h, ZOA_ERR_STATE, "zoa_check_finite: the handle's device is not the current CUDA device");
    ZOA_CUDA(h, plain_errors(h));
    ZOA_CUDA(h, cudaDeviceSynchronize());
    ZOA_CUDA(h, cudaMemset(h->sched, 0, 2 * sizeof(unsigned long long)));      // borrowed as the counter; it is 0 between launches
    const long long rows = (long long)h->W * h->n_pad;
    const float *bufs[] = {h->x, h->m, h->u, h->dw, h->v_pending ? h->v_nxt : h->v_cur, h->ds, h->xs};
    const long long counts[] = {rows, rows, rows, rows, h->n_pad, h->n_pad, h->n_pad};
    for (int k = 0; k < 7; ++k)
        if (!h->allreduce_only || bufs[k] == h->dw || bufs[k] == h->ds)
            ZOA_CUDA(h, launch_count_nonfinite(bufs[k], counts[k], h->sched, h->sm_count, nullptr));
    unsigned long long bad = 0;
    ZOA_CUDA(h, cudaMemcpy(&bad, h->sched, sizeof(bad), cudaMemcpyDeviceToHost));
    ZOA_CUDA(h, cudaMemset(h->sched, 0, 2 * sizeof(unsigned long long)));
    if (n_nonfinite) *n_nonfinite = (int64_t)bad;
    if (bad) return fail(h, ZOA_ERR_NONFINITE, "the optimizer state holds NaN or infinite values");
    return ZOA_OK;
}

extern "C" zoa_status zoa_set_option(zoa_handle h, int option, int value)
{
    if (!h) return ZOA_ERR_ARG;
    switch (option) {
    case ZOA_OPT_PIPELINE:
        if (value < 0 || value > 2) return fail(h, ZOA_ERR_ARG, "zoa_set_option: ZOA_OPT_PIPELINE takes 0, 1 or 2");
        h->use_pipeline = value;
        return ZOA_OK;
    case ZOA_OPT_GRAD_TYPE:
        if (value < ZOA_GRAD_F32 || value > ZOA_GRAD_BF16) return fail(h, ZOA_ERR_ARG, "zoa_set_option: unknown gradient type");
        h->grad_type = value;
        return ZOA_OK;
    case ZOA_OPT_WAIT_LIMIT_MS:
        if (value < 1 || value > 60000) return fail(h, ZOA_ERR_ARG, "zoa_set_option: wait limit must be 1..60000 ms");
        h->wait_limit_ms = value;
        return ZOA_OK;
    case ZOA_OPT_TEST_STOP_AFTER_TILES:
        if (value < 0) return fail(h, ZOA_ERR_ARG, "zoa_set_option: negative tile count");
        h->test_stop_after_tiles = value;
        return ZOA_OK;
    default: return fail(h, ZOA_ERR_ARG, "zoa_set_option: unknown option");
    }
}

extern "C" const char *zoa_last_error(zoa_handle h)
{
    return h ? h->err.c_str() : g_create_error.c_str();
}
