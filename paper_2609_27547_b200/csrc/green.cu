// SM partitions ("green contexts") for the SM quota: a context that owns a subset of the SMs and
// a stream inside it.  Kernels launched on that stream can only run on the partition's SMs, so a
// quota is enforced by the driver as well as by the persistent-grid cap, and a co-running stage
// (simulation, training) keeps the rest of the chip.  The driver entry points are looked up at
// run time; if any is missing or fails, the caller falls back to the grid cap alone.
#include "actgen_internal.h"

#include <cuda.h>

namespace ebrl {

namespace {
struct Api {
    CUresult (*getDevResource)(CUdevice, CUdevResource *, CUdevResourceType) = nullptr;
    CUresult (*splitByCount)(CUdevResource *, unsigned int *, const CUdevResource *, CUdevResource *, unsigned int, unsigned int) = nullptr;
    CUresult (*generateDesc)(CUdevResourceDesc *, CUdevResource *, unsigned int) = nullptr;
    CUresult (*greenCreate)(CUgreenCtx *, CUdevResourceDesc, CUdevice, unsigned int) = nullptr;
    CUresult (*greenDestroy)(CUgreenCtx) = nullptr;
    CUresult (*streamCreate)(CUstream *, CUgreenCtx, unsigned int, int) = nullptr;
    CUresult (*deviceGet)(CUdevice *, int) = nullptr;
    bool ok = false;
};

template <typename F> bool load(const char *name, F &fn)
{
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
        cudaGetLastError();
        return false;
    }
    fn = reinterpret_cast<F>(p);
    return true;
}

const Api &api()
{
    static Api a;
    static bool tried = false;
    if (!tried) {
        tried = true;
        a.ok = load("cuDeviceGetDevResource", a.getDevResource) && load("cuDevSmResourceSplitByCount", a.splitByCount) &&
               load("cuDevResourceGenerateDesc", a.generateDesc) && load("cuGreenCtxCreate", a.greenCreate) &&
               load("cuGreenCtxDestroy", a.greenDestroy) && load("cuGreenCtxStreamCreate", a.streamCreate) &&
               load("cuDeviceGet", a.deviceGet);
    }
    return a;
}
}  // namespace

// Creates a partition of at least `sm_quota` SMs on `device` and a stream in it.  Returns 0 on
// success; sm_count is the number of SMs the driver actually put in the partition (it rounds up
// to its granularity).  The SMs left over become a second partition with a stream of its own
// (rest_*; absent when nothing is left or the driver refuses it): work launched there cannot
// reach the first partition's SMs, which is how a co-running stage is fenced OUT of the quota.
int green_partition_create(int device, int sm_quota, GreenPartition *out)
{
    const Api &a = api();
    if (!a.ok || !out || sm_quota < 1) return 1;
    CUdevice dev;
    if (a.deviceGet(&dev, device) != CUDA_SUCCESS) return 2;
    CUdevResource all, part, rest;
    if (a.getDevResource(dev, &all, CU_DEV_RESOURCE_TYPE_SM) != CUDA_SUCCESS) return 3;
    unsigned int groups = 1;
    if (a.splitByCount(&part, &groups, &all, &rest, 0, (unsigned int)sm_quota) != CUDA_SUCCESS || groups < 1) return 4;
    CUdevResourceDesc desc;
    if (a.generateDesc(&desc, &part, 1) != CUDA_SUCCESS) return 5;
    CUgreenCtx ctx;
    if (a.greenCreate(&ctx, desc, dev, CU_GREEN_CTX_DEFAULT_STREAM) != CUDA_SUCCESS) return 6;
    CUstream st;
    if (a.streamCreate(&st, ctx, CU_STREAM_NON_BLOCKING, 0) != CUDA_SUCCESS) {
        a.greenDestroy(ctx);
        return 7;
    }
    out->ctx = ctx;
    out->stream = (cudaStream_t)st;
    out->sm_count = (int)part.sm.smCount;
    out->rest_ctx = nullptr;
    out->rest_stream = nullptr;
    out->rest_sm_count = 0;
    if (rest.sm.smCount > 0) {
        CUdevResourceDesc rdesc;
        CUgreenCtx rctx;
        if (a.generateDesc(&rdesc, &rest, 1) == CUDA_SUCCESS && a.greenCreate(&rctx, rdesc, dev, CU_GREEN_CTX_DEFAULT_STREAM) == CUDA_SUCCESS) {
            CUstream rst;
            if (a.streamCreate(&rst, rctx, CU_STREAM_NON_BLOCKING, 0) == CUDA_SUCCESS) {
                out->rest_ctx = rctx;
                out->rest_stream = (cudaStream_t)rst;
                out->rest_sm_count = (int)rest.sm.smCount;
            } else {
                a.greenDestroy(rctx);
            }
        }
    }
    return 0;
}

void green_partition_destroy(GreenPartition *p)
{
    const Api &a = api();
    if (!p || !p->ctx) return;
    if (p->stream) cudaStreamDestroy(p->stream);
    if (p->rest_stream) cudaStreamDestroy(p->rest_stream);
    if (a.ok) a.greenDestroy((CUgreenCtx)p->ctx);
    if (a.ok && p->rest_ctx) a.greenDestroy((CUgreenCtx)p->rest_ctx);
    p->ctx = p->rest_ctx = nullptr;
    p->stream = p->rest_stream = nullptr;
}

}  // namespace ebrl
