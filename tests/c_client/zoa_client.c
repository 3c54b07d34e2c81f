/* A plain C user of include/zoa.h: no Python, no torch.  Reads a problem from a binary file
 * (header of six int64: n, W, chunk, steps, sync interval, number of T_v steps; then the T_v
 * steps as int64, x0 as n floats and steps x W x n gradient floats), runs Algorithm 1 through
 * the fused entry point on even steps and the two-call form on odd steps, and writes worker
 * 0's x, m, u followed by v to the output file.  Exit code 0 on success. */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include <cuda_runtime_api.h>

#include "zoa.h"

#define CHECK_ZOA(h, call)                                                              \
    do {                                                                                \
        zoa_status s_ = (call);                                                         \
        if (s_ != ZOA_OK) {                                                             \
            fprintf(stderr, "%s -> %d: %s\n", #call, (int)s_, zoa_last_error(h));       \
            return 2;                                                                   \
        }                                                                               \
    } while (0)
#define CHECK_CUDA(call)                                                                \
    do {                                                                                \
        cudaError_t e_ = (call);                                                        \
        if (e_ != cudaSuccess) {                                                        \
            fprintf(stderr, "%s: %s\n", #call, cudaGetErrorString(e_));                 \
            return 3;                                                                   \
        }                                                                               \
    } while (0)

int main(int argc, char **argv)
{
    if (argc != 3) return 1;
    FILE *in = fopen(argv[1], "rb");
    if (!in) return 1;
    int64_t hdr[6];
    if (fread(hdr, sizeof(int64_t), 6, in) != 6) return 1;
    const int64_t n = hdr[0], W = hdr[1], chunk = hdr[2], steps = hdr[3], interval = hdr[4], n_var = hdr[5];
    int64_t *var_steps = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n_var > 0 ? n_var : 1));
    float *host = (float *)malloc(sizeof(float) * (size_t)n);
    if (!var_steps || !host) return 1;
    if (fread(var_steps, sizeof(int64_t), (size_t)n_var, in) != (size_t)n_var) return 1;

    zoa_handle h = NULL;
    CHECK_ZOA(NULL, zoa_create(&h, (size_t)n, (int)W, 0.9f, 0.999f, 1e-8f, (int)chunk));
    cudaStream_t stream;
    CHECK_CUDA(cudaStreamCreate(&stream));
    float *d_x0 = NULL, *d_g = NULL;
    CHECK_CUDA(cudaMalloc((void **)&d_x0, sizeof(float) * (size_t)n));
    CHECK_CUDA(cudaMalloc((void **)&d_g, sizeof(float) * (size_t)(n * W)));
    if (fread(host, sizeof(float), (size_t)n, in) != (size_t)n) return 1;
    CHECK_CUDA(cudaMemcpyAsync(d_x0, host, sizeof(float) * (size_t)n, cudaMemcpyHostToDevice, stream));
    CHECK_ZOA(h, zoa_set_params(h, d_x0, stream));
    CHECK_ZOA(h, zoa_set_var_steps(h, var_steps, (size_t)n_var));
    const int64_t bounds[1] = {0};
    const int32_t intervals[1] = {(int32_t)interval};
    CHECK_ZOA(h, zoa_set_sync_policy(h, bounds, intervals, 1));

    const void *grads[64];
    for (int64_t i = 0; i < W; ++i) grads[i] = d_g + i * n;
    for (int64_t t = 0; t < steps; ++t) {
        for (int64_t i = 0; i < W; ++i) {
            if (fread(host, sizeof(float), (size_t)n, in) != (size_t)n) return 1;
            CHECK_CUDA(cudaMemcpyAsync(d_g + i * n, host, sizeof(float) * (size_t)n, cudaMemcpyHostToDevice, stream));
            CHECK_CUDA(cudaStreamSynchronize(stream));      /* `host` is reused for the next worker */
        }
        if (t % 2 == 0) {
            CHECK_ZOA(h, zoa_step_auto(h, grads, 1e-3f, t, stream));
        } else {
            CHECK_ZOA(h, zoa_step(h, grads, 1e-3f, t, stream));
            if (zoa_sync_due(h, t)) CHECK_ZOA(h, zoa_onebit_reduce(h, stream));
        }
    }
    CHECK_CUDA(cudaStreamSynchronize(stream));
    CHECK_ZOA(h, zoa_check_device(h));

    FILE *out = fopen(argv[2], "wb");
    if (!out) return 1;
    const zoa_buffer which[4] = {ZOA_BUF_X, ZOA_BUF_M, ZOA_BUF_U, ZOA_BUF_V};
    for (int k = 0; k < 4; ++k) {
        CHECK_ZOA(h, zoa_copy_out(h, which[k], 0, 0, (size_t)n, host));
        if (fwrite(host, sizeof(float), (size_t)n, out) != (size_t)n) return 1;
    }
    fclose(out);
    fclose(in);
    zoa_stats st;
    CHECK_ZOA(h, zoa_get_stats(h, &st));
    printf("steps %lld syncs %lld launches %lld\n", (long long)st.n_steps, (long long)st.n_syncs, (long long)st.n_launches);
    CHECK_ZOA(h, zoa_destroy(h));
    cudaFree(d_x0);
    cudaFree(d_g);
    cudaStreamDestroy(stream);
    free(host);
    free(var_steps);
    return 0;
}
