// Synthetic memory-bound "simulation" co-runner for the SM-quota experiments: a bounded number
// of read-modify-write passes over a device buffer by a persistent grid of a chosen size.
#include "../../include/ebrl_actgen.h"
#include <cuda_runtime.h>

namespace {
__global__ void __launch_bounds__(512) sim_stream_kernel(float4 *buf, uint64_t n4, int n_steps, float alpha, float beta)
{
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (int s = 0; s < n_steps; ++s)
        for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
            float4 v = buf[i];
            v.x = fmaf(v.x, alpha, beta); v.y = fmaf(v.y, alpha, beta);
            v.z = fmaf(v.z, alpha, beta); v.w = fmaf(v.w, alpha, beta);
            buf[i] = v;
        }
}
}  // namespace

extern "C" ebrl_status_t ebrl_sim_corunner_launch(float *buf, uint64_t n_floats, int32_t n_steps, int32_t n_ctas, void *stream)
{
    if (!buf || (n_floats & 3) || (((uintptr_t)buf) & 15) || n_steps < 0 || n_ctas < 1) return EBRL_ERR_INVALID_ARG;
    if (n_floats == 0 || n_steps == 0) return EBRL_OK;
    sim_stream_kernel<<<n_ctas, 512, 0, (cudaStream_t)stream>>>((float4 *)buf, n_floats / 4, n_steps, 0.999f, 0.001f);
    return cudaGetLastError() == cudaSuccess ? EBRL_OK : EBRL_ERR_CUDA;
}
