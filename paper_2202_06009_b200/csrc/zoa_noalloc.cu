// zoa_onebit_allreduce_static: the error-feedback 1-bit AllReduce on caller-owned
// buffers, for callers that must not allocate device memory.
//
// Who cannot allocate: code that runs where cudaMalloc is forbidden or harmful -
// inside a framework's caching-allocator region whose memory budget is already
// handed out, in a latency-critical loop where cudaMalloc's implicit device
// synchronisation would stall every stream, in a process whose memory is fully
// pre-partitioned between tenants, or in an error/clean-up path that runs when
// the device is already out of memory.  Such callers own every byte they pass
// in; the only extra memory this entry point touches is the fixed array below,
// which is part of the loaded library image.
//
// The packed sign words and per-chunk magnitudes that the workers "send" to
// the server live between the two kernels of a call.  Here they sit in a
// file-scope __device__ array of a fixed size, so a call allocates nothing:
// no cudaMalloc, no cudaFree, no library routine that allocates.
//
// Consequences the caller must know:
//  * every GPU that loads the library holds the array (4 MiB) until exit;
//  * sizes whose packed form does not fit are rejected (ZOA_ERR_ARG);
//  * all calls on a device share the array: two calls whose work overlaps on
//    the GPU (different streams, no ordering between them) race on it;
//  * the array keeps the previous call's contents; every word and magnitude a
//    call reads was written earlier in the same call, so nothing has to be
//    cleared in between;
//  * the first call on a device looks up the array's device address
//    (cudaGetSymbolAddress) and raises two kernels' shared-memory limit; make
//    that first call before any stream capture begins.
#include <cstdint>
#include <mutex>

#include "../../include/zoa.h"
#include "zoa_device.cuh"

namespace zoa {

// 1 Mi 32-bit slots = 4 MiB: [W][words_stride] sign words, then [W][n_chunks] magnitudes.
constexpr size_t kStaticScratchSlots = (size_t)1 << 20;
static __device__ __align__(256) uint32_t g_static_scratch[kStaticScratchSlots];

struct StaticArgs {
    const float *z[kMaxWorkers];   // buffers to reduce, n floats each
    float *delta_w[kMaxWorkers];   // worker errors, in/out
    float *delta_s;                // server error, in/out
    float *z_bar;                  // result
    uint32_t *words;               // scratch: [W][words_stride]
    float *scales;                 // scratch: [W][n_chunks]
    long long n, n_chunks, words_stride;
    int W, chunk, aligned;
};

__device__ __forceinline__ void st_guard4(float *p, long long j, long long n, bool aligned, const float v[4])
{
    if (aligned && j + 4 <= n) {
        st4(p + j, make_float4(v[0], v[1], v[2], v[3]));
        return;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k)
        if (j + k < n) p[j + k] = v[k];
}

// Worker side of Algorithm 3 for (chunk blockIdx.x, worker blockIdx.y): the
// packed result goes to the static scratch.
__global__ void static_compress_kernel(StaticArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *scratch = reinterpret_cast<double *>(smem_raw);
    float *z_s = reinterpret_cast<float *>(smem_raw + 34 * sizeof(double));
    const int i = blockIdx.y;
    const long long c0 = (long long)blockIdx.x * a.chunk;
    const int len = (int)(a.n - c0 < a.chunk ? a.n - c0 : a.chunk);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;

    double l1 = 0.0;
    for (int base = warp * 128; base < len; base += n_warps * 128) {
        const int idx = base + 4 * lane;
        if (idx < len) {
            const float4 z4 = ld_grad4(a.z[i], c0 + idx, a.n, a.aligned);
            const float4 e4 = ld_grad4(a.delta_w[i], c0 + idx, a.n, a.aligned);
            const float4 s4 = make_float4(f_add(z4.x, e4.x), f_add(z4.y, e4.y), f_add(z4.z, e4.z), f_add(z4.w, e4.w));
            st4(z_s + idx, s4);
            l1 += fabs((double)s4.x) + fabs((double)s4.y) + fabs((double)s4.z) + fabs((double)s4.w);
        }
    }
    const float scale = chunk_scale(block_sum(l1, scratch), len);
    for (int base = warp * 128; base < len; base += n_warps * 128) {
        const int idx = base + 4 * lane;
        float z[4] = {0.f, 0.f, 0.f, 0.f};
        bool b[4];
        if (idx < len) {
            const float4 z4 = ld4(z_s + idx);
            z[0] = z4.x; z[1] = z4.y; z[2] = z4.z; z[3] = z4.w;
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool valid = idx + k < len;
            b[k] = valid && (z[k] >= 0.0f);
            z[k] = valid ? f_sub(z[k], b[k] ? scale : -scale) : 0.0f;
        }
        const uint32_t word = pack_tile(b);
        if (idx < len) st_guard4(a.delta_w[i], c0 + idx, a.n, a.aligned, z);
        if (lane < 4 && base + 32 * lane < len)
            a.words[(long long)i * a.words_stride + ((c0 + base) >> 5) + lane] = word;
    }
    if (threadIdx.x == 0) a.scales[(long long)i * a.n_chunks + blockIdx.x] = scale;
}

// Server side of Algorithm 3 for chunk blockIdx.x, reading the static scratch.
__global__ void static_average_kernel(StaticArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *scratch = reinterpret_cast<double *>(smem_raw);
    float *scales = reinterpret_cast<float *>(smem_raw + 34 * sizeof(double));
    float *a_s = scales + kMaxWorkers;
    const long long c0 = (long long)blockIdx.x * a.chunk;
    const int len = (int)(a.n - c0 < a.chunk ? a.n - c0 : a.chunk);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;

    for (int i = threadIdx.x; i < a.W; i += blockDim.x) scales[i] = a.scales[(long long)i * a.n_chunks + blockIdx.x];
    __syncthreads();
    double l1 = 0.0;
    for (int base = warp * 128; base < len; base += n_warps * 128) {
        const int idx = base + 4 * lane;
        if (idx < len) {
            double A[4] = {0.0, 0.0, 0.0, 0.0};
            const long long word_idx = (c0 + idx) >> 5;
            const int shift = idx & 31;
            for (int i = 0; i < a.W; ++i) {
                const uint32_t nib = a.words[(long long)i * a.words_stride + word_idx] >> shift;
                const double s = (double)scales[i];
#pragma unroll
                for (int k = 0; k < 4; ++k) A[k] += ((nib >> k) & 1u) ? s : -s;
            }
            const float4 e4 = ld_grad4(a.delta_s, c0 + idx, a.n, a.aligned);
            const float ee[4] = {e4.x, e4.y, e4.z, e4.w};
            float v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                v[k] = idx + k < len ? server_input(A[k], a.W, ee[k]) : 0.0f;
                l1 += fabs((double)v[k]);
            }
            st4(a_s + idx, make_float4(v[0], v[1], v[2], v[3]));
        }
    }
    const float scale = chunk_scale(block_sum(l1, scratch), len);
    for (int base = warp * 128; base < len; base += n_warps * 128) {
        const int idx = base + 4 * lane;
        if (idx < len) {
            const float4 a4 = ld4(a_s + idx);
            const float v[4] = {a4.x, a4.y, a4.z, a4.w};
            float hat[4], err[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                hat[k] = v[k] >= 0.0f ? scale : -scale;
                err[k] = f_sub(v[k], hat[k]);
            }
            st_guard4(a.z_bar, c0 + idx, a.n, a.aligned, hat);
            st_guard4(a.delta_s, c0 + idx, a.n, a.aligned, err);
        }
    }
}

// Per-device set-up, done once with that device current.
static std::mutex g_setup_mutex;
static uint32_t *g_scratch_addr[64] = {nullptr};

static cudaError_t static_setup(int device, uint32_t **addr)
{
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[device]) {
        uint32_t *p = nullptr;
        // In host code the array's name is only a stand-in; its device address must be asked for.
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_static_scratch);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(static_compress_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(34 * sizeof(double) + kMaxChunk * sizeof(float)));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(static_average_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(34 * sizeof(double) + (kMaxWorkers + kMaxChunk) * sizeof(float)));
        if (e != cudaSuccess) return e;
        g_scratch_addr[device] = p;
    }
    *addr = g_scratch_addr[device];
    return cudaSuccess;
}

}  // namespace zoa

using namespace zoa;

static thread_local const char *g_static_error = "";
static zoa_status static_fail(zoa_status s, const char *msg)
{
    g_static_error = msg;
    return s;
}

extern "C" size_t zoa_static_scratch_slots(void) { return kStaticScratchSlots; }
extern "C" const char *zoa_static_last_error(void) { return g_static_error; }

extern "C" zoa_status zoa_onebit_allreduce_static(const float *const *z, float *const *delta_w, float *delta_s,
                                                  float *z_bar, size_t n, int W, int chunk, void *stream)
{
    if (!z || !delta_w || !delta_s || !z_bar) return static_fail(ZOA_ERR_ARG, "zoa_onebit_allreduce_static: a NULL pointer");
    if (n < 1 || W < 1 || W > kMaxWorkers) return static_fail(ZOA_ERR_ARG, "zoa_onebit_allreduce_static: need n >= 1 and 1 <= W <= 64");
    if (chunk < 32 || chunk > kMaxChunk || chunk % 32 != 0)
        return static_fail(ZOA_ERR_ARG, "zoa_onebit_allreduce_static: chunk must be a multiple of 32 in [32, 16384]");
    // One worker's sign words alone must fit, which also keeps the 64-bit size arithmetic below from wrapping.
    if (n > (size_t)32 * kStaticScratchSlots)
        return static_fail(ZOA_ERR_ARG, "zoa_onebit_allreduce_static: n exceeds what the 1,048,576 slots of the built-in scratch "
                                        "array can hold for a single worker; use a handle (zoa_create) for this size");
    StaticArgs a{};
    a.n = (long long)n;
    a.W = W;
    a.chunk = chunk;
    a.n_chunks = (a.n + chunk - 1) / chunk;
    a.words_stride = (a.n + 31) / 32;
    // Does the packed form of this call fit the fixed array?
    const unsigned long long need = (unsigned long long)W * (unsigned long long)(a.words_stride + a.n_chunks);
    if (need > kStaticScratchSlots)
        return static_fail(ZOA_ERR_ARG, "zoa_onebit_allreduce_static: W * (ceil(n/32) + ceil(n/chunk)) exceeds the "
                                        "1,048,576 slots of the built-in scratch array; use a handle (zoa_create) for this size");
    a.aligned = 1;
    for (int i = 0; i < W; ++i) {
        if (!z[i] || !delta_w[i]) return static_fail(ZOA_ERR_ARG, "zoa_onebit_allreduce_static: a NULL buffer pointer");
        a.z[i] = z[i];
        a.delta_w[i] = delta_w[i];
        if ((reinterpret_cast<uintptr_t>(z[i]) | reinterpret_cast<uintptr_t>(delta_w[i])) & 15u) a.aligned = 0;
    }
    if ((reinterpret_cast<uintptr_t>(delta_s) | reinterpret_cast<uintptr_t>(z_bar)) & 15u) a.aligned = 0;
    a.delta_s = delta_s;
    a.z_bar = z_bar;

    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64)
        return static_fail(ZOA_ERR_CUDA, "zoa_onebit_allreduce_static: no usable current device");
    uint32_t *scratch = nullptr;
    if (static_setup(device, &scratch) != cudaSuccess)
        return static_fail(ZOA_ERR_CUDA, "zoa_onebit_allreduce_static: looking up the scratch array's device address failed");
    a.words = scratch;
    a.scales = reinterpret_cast<float *>(scratch + (size_t)W * a.words_stride);

    int threads = chunk / 8;
    threads = threads < 128 ? 128 : threads > 1024 ? 1024 : threads;
    int p = 128;
    while (p < threads) p <<= 1;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    static_compress_kernel<<<dim3((unsigned)a.n_chunks, (unsigned)W), p,
                             34 * sizeof(double) + (size_t)chunk * sizeof(float), s>>>(a);
    if (cudaGetLastError() != cudaSuccess) return static_fail(ZOA_ERR_CUDA, "zoa_onebit_allreduce_static: kernel launch failed");
    static_average_kernel<<<(unsigned)a.n_chunks, p,
                            34 * sizeof(double) + (kMaxWorkers + (size_t)chunk) * sizeof(float), s>>>(a);
    if (cudaGetLastError() != cudaSuccess) return static_fail(ZOA_ERR_CUDA, "zoa_onebit_allreduce_static: kernel launch failed");
    return ZOA_OK;
}
