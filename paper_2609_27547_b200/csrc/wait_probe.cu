// A harmless exercise of the bounded device-side wait every kernel of this library uses: one
// warp waits on an mbarrier that nothing ever signals; when the limit runs out the wait returns,
// the kernel records EBRL_ERR_TIMEOUT in a status word and exits normally -- no trap, no hang,
// the context stays usable.  This is how a lost producer shows up in the real kernels.
#include "../../include/ebrl_actgen.h"
#include "ptx_helpers.cuh"

#include <cuda_runtime.h>

namespace {
__global__ void wait_probe_kernel(unsigned long long limit_ns, int signal_it, int *status, unsigned long long *waited_ns)
{
    __shared__ unsigned long long bar;
    __shared__ int abort_flag;
    using namespace ebrl::ptx;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (signal_it && threadIdx.x == 0) mbar_arrive(b);   // the healthy case: the producer arrives
    const unsigned long long t0 = gtimer();
    const bool ok = mbar_wait(b, 0, limit_ns, &abort_flag);
    if (threadIdx.x == 0) {
        *waited_ns = gtimer() - t0;
        *status = ok ? 0 : (int)EBRL_ERR_TIMEOUT;
    }
}
}  // namespace

extern "C" ebrl_status_t ebrl_actgen_wait_probe(int32_t device, uint64_t limit_ns, int32_t signal_it, int32_t *out_status,
                                                uint64_t *out_waited_ns)
{
    if (!out_status || limit_ns == 0 || limit_ns > 2000000000ull) return EBRL_ERR_INVALID_ARG;
    if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return EBRL_ERR_CUDA; }
    int *st = nullptr;
    unsigned long long *w = nullptr;
    if (cudaMalloc((void **)&st, sizeof(int)) != cudaSuccess || cudaMalloc((void **)&w, sizeof(unsigned long long)) != cudaSuccess) {
        cudaGetLastError();
        if (st) cudaFree(st);
        return EBRL_ERR_NOMEM;
    }
    wait_probe_kernel<<<1, 32>>>(limit_ns, signal_it, st, w);
    int hs = -1;
    unsigned long long hw = 0;
    cudaError_t e = cudaMemcpy(&hs, st, sizeof hs, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemcpy(&hw, w, sizeof hw, cudaMemcpyDeviceToHost);
    cudaFree(st);
    cudaFree(w);
    if (e != cudaSuccess) return EBRL_ERR_CUDA;
    *out_status = hs;
    if (out_waited_ns) *out_waited_ns = hw;
    return EBRL_OK;
}
