// Declarations shared between the kernels' translation unit and the C-ABI one.
#pragma once

#include "zoa_device.cuh"

namespace zoa {

cudaError_t configure_kernels();

cudaError_t launch_local_step(const StateView &st, const GradPtrs &g, const Consts &c, float gamma,
                              bool do_var, bool g_aligned, int sm_count, cudaStream_t s);
cudaError_t launch_variance(const StateView &st, const GradPtrs &g, const Consts &c, bool g_aligned,
                            int sm_count, cudaStream_t s);
cudaError_t launch_compress(const StateView &st, cudaStream_t s);
cudaError_t launch_reduce(const StateView &st, const Consts &c, float gamma_sum, cudaStream_t s);
cudaError_t launch_step_sync(const StateView &st, const GradPtrs &g, const Consts &c, float gamma,
                             float gamma_sum, bool g_aligned, cudaStream_t s);

}  // namespace zoa
