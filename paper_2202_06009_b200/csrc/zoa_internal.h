// Declarations shared between the kernels' translation unit and the C-ABI one.
#pragma once

#include <mutex>

#include "zoa_device.cuh"

namespace zoa {

// Where a kernel that gives up on a bounded wait says so: a device word (zoa_check_device reads
// and clears it) and the device-side address of a word in pinned, mapped host memory, which the
// step entry points test without synchronising.
struct ErrorWords {
    int *device;
    int *host_mapped;
};

// Raises a kernel's dynamic shared-memory limit the first time the kernel is launched on a
// device; one object per kernel (template instantiation).  Safe to call from several threads.
struct SmemLimitOnce {
    std::mutex mu;
    bool done[64] = {false};
    template <typename Kernel>
    cudaError_t ensure(Kernel kern, int bytes)
    {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        std::lock_guard<std::mutex> lock(mu);
        if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
        return e;
    }
};

cudaError_t configure_kernels();

cudaError_t launch_local_step(const StateView &st, const GradPtrs &g, const Consts &c, float gamma,
                              bool do_var, int g_aligned, long long first, long long end, cudaStream_t s);
cudaError_t launch_variance(const StateView &st, const GradPtrs &g, const Consts &c, int g_aligned,
                            long long first, long long end, cudaStream_t s);
cudaError_t launch_compress(const StateView &st, long long first_chunk, long long count, cudaStream_t s);
cudaError_t launch_reduce(const StateView &st, const Consts &c, float gamma_sum, long long first_chunk, long long count, cudaStream_t s);

// Ring form of the server half of zoa_onebit_reduce, zoa_reduce_pipeline.cu.  reduce_pipeline_stages:
// ring depth (0 = the kernel does not take this shape) and how many whole units of max(chunk, 2048)
// coordinates the vector holds; the chunks after them go through launch_reduce.
int reduce_pipeline_stages(const StateView &st, long long *n_units);
cudaError_t launch_reduce_pipelined(const StateView &st, const Consts &c, float gamma_sum, long long n_units,
                                    int stages, int sm_count, ErrorWords error_flag, unsigned long long *sched,
                                    unsigned long long wait_limit_ns, long long test_stop_after_tiles, cudaStream_t s);
// Server side of Algorithm 3 alone with its inputs prefetched into shared memory (zoa_server_pipeline.cu):
// whether the buffers allow it, and the launch for the whole chunks [first_chunk, first_chunk + count).
bool server_prefetch_applies(const StateView &st, const uint32_t *words_in, long long words_in_stride, int W_total, const float *z_bar);
cudaError_t launch_server_prefetch(const StateView &st, const uint32_t *words_in, long long words_in_stride,
                                   const float *scales_in, long long scales_in_stride, int W_total, long long first_chunk,
                                   long long count, const PeerOut &out, float *z_bar, ErrorWords error_flag,
                                   unsigned long long wait_limit_ns, bool skip_copies, cudaStream_t s);
cudaError_t launch_step_sync(const StateView &st, const GradPtrs &g, const Consts &c, float gamma,
                             float gamma_sum, int g_aligned, long long first_chunk, long long count, cudaStream_t s);

cudaError_t launch_alg2(const StateView &st, const GradPtrs &g, const Consts &c, float gamma, bool full_precision,
                        int g_aligned, long long first_chunk, long long count, cudaStream_t s);

// Chunks larger than kMaxChunk (up to the whole vector): multi-pass kernels, zoa_kernels.cu.
long long large_chunk_segments(const StateView &st);
cudaError_t launch_large_compress(const StateView &st, const GradPtrs &g, const Consts &c, float gamma, int src,
                                  int g_aligned, bool pending, double *partials, int *launches, cudaStream_t s);
cudaError_t launch_large_server(const StateView &st, const Consts &c, int mode, float scalar, bool pending, double *partials,
                                int *launches, cudaStream_t s);
cudaError_t launch_plain_errors(const StateView &st, bool workers, bool server, cudaStream_t s);

// Pipelined (bulk-copy ring) form of the fused sync step, zoa_pipeline.cu.
int pipeline_stages(const StateView &st, int grad_fmt);
int pipeline_chunks_per_unit(const StateView &st);
cudaError_t launch_step_sync_pipelined(const StateView &st, const GradPtrs &g, const Consts &c, float gamma,
                                       float gamma_sum, bool do_var, int grad_fmt, long long first_unit, long long n_units, int stages,
                                       int sm_count, ErrorWords error_flag,
                                       unsigned long long *sched, unsigned long long wait_limit_ns,
                                       long long test_stop_after_tiles, bool *var_fused, cudaStream_t s);

cudaError_t launch_local_step_pipelined(const StateView &st, const GradPtrs &g, const Consts &c, float gamma, bool do_var,
                                        int grad_fmt, long long first_unit, long long n_units, int sm_count, ErrorWords error_flag,
                                        unsigned long long *sched, unsigned long long wait_limit_ns,
                                        long long test_stop_after_tiles, cudaStream_t s);

// One worker per GPU: the kernels between the collectives.
cudaError_t launch_dist_server(const StateView &st, const uint32_t *words_in, long long words_in_stride,
                               const float *scales_in, long long scales_in_stride, int W_total,
                               long long first_chunk, long long count, const PeerOut &out, float *z_bar, cudaStream_t s);
cudaError_t launch_compress_external(const StateView &st, const GradPtrs &z, int z_fmt, cudaStream_t s);
cudaError_t launch_dist_pack_push(const StateView &st, const float *g, const Consts &c, float gamma, int g_fmt,
                                  const PushPlan &plan, cudaStream_t s);
cudaError_t launch_dist_apply(const StateView &st, const Consts &c, float gamma_sum, cudaStream_t s);
cudaError_t launch_dist_variance(const StateView &st, const Consts &c, const float *g_bar, cudaStream_t s);

cudaError_t launch_count_nonfinite(const float *p, long long count, unsigned long long *out, int sm_count, cudaStream_t s);

int alg2_pipeline_stages(const StateView &st, int grad_fmt);
cudaError_t launch_alg2_pipelined(const StateView &st, const GradPtrs &g, const Consts &c, float gamma, int grad_fmt,
                                  int stages, int sm_count, ErrorWords error_flag, unsigned long long *sched,
                                  unsigned long long wait_limit_ns, long long test_stop_after_tiles, cudaStream_t s);

}  // namespace zoa
