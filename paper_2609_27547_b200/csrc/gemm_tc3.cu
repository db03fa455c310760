// fp32 GEMM on the tensor cores by operand splitting, for the fp32 models.  Each fp32 operand is
// written as the exact sum of three bf16 terms, a = a0 + a1 + a2 (a0 = bf16(a), a1 = bf16(a - a0),
// a2 = bf16(a - a0 - a1): 3 x 8 significand bits cover fp32's 24), and the product of two such sums
// is taken from the six partial products that are not below 2^-24 of the leading one,
//     a w  ~=  a2 w0 + a1 w1 + a0 w2 + a1 w0 + a0 w1 + a0 w0,
// each a bf16 x bf16 tcgen05.mma with fp32 accumulation in tensor memory.  The dropped products
// (a1 w2, a2 w1, a2 w2) are below 2^-24 |a w|, so a dot product carries the rounding error of an fp32
// computation: the fp32 models keep their 1e-4 bound against the fp64 oracle while the projections
// leave the FFMA pipe (2 x 128 FLOP per clock per SM) for the tensor pipe (six products still run
// several times faster).
//
// Weights are split once (split3_kernel), when they are copied into the handle; activations are
// written as their three term planes by whatever produces them (the embedding, the residual and
// GELU epilogues below, the attention kernel).  The GEMM is the single-CTA 128 x 128
// tensor-core kernel with six operand tiles per 64-wide k-block (96 KB per stage, two stages) and
// the same fused epilogues on fp32 outputs.  With K of a few hundred the epilogue of a tile takes
// longer than its mainloop, so two groups of four epilogue warps drain the two accumulators in
// turn (tile i by group i mod 2): two epilogues run while the next tile accumulates.  Every output
// element is the sum over k in order of its six products in the order above, whatever the grid
// size: results do not depend on the SM quota or on which rows share a tile.  Every wait is
// bounded (status word, as in the other kernels).
#include "actgen_internal.h"
#include "ptx_helpers.cuh"
#include "gemm_epilogue.cuh"

#include <cuda.h>

namespace ebrl {
namespace tc3 {

using namespace ptx;
using namespace tc;

constexpr int BM = 128, BN = 128, BK = 64, UMMA_K = 16, STAGES = 2, EPI_WARPS = 8;   // two groups of four
constexpr int TILE_BYTES = BM * BK * 2;                 // one bf16 operand tile
constexpr int STAGE_BYTES = 6 * TILE_BYTES;             // A0 A1 A2 W0 W1 W2
constexpr int THREADS = 64 + 32 * EPI_WARPS;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * EPI_STAGE_FLOATS * 4 + 256 + 1024;
constexpr uint32_t TMEM_COLS = 2 * BN;

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, uint32_t bar, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr)
{
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__host__ __device__ constexpr uint32_t instr_desc(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

struct Maps6 {
    CUtensorMap a[3], w[3];
};

template <int EPI>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc3_kernel(const __grid_constant__ Maps6 tm, GemmArgs g, unsigned long long limit_ns, int *status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t s0 = smem_u32(smem);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + STAGES * STAGE_BYTES + EPI_WARPS * EPI_STAGE_FLOATS * 4);
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto tfull = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
    auto tempty = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + 2 * STAGES + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * STAGES + 5);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ntm = (g.M + BM - 1) / BM, ntn = g.N / BN, ntiles = ntm * ntn, nkb = g.K / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull(b), 1); mbar_init(tempty(b), EPI_WARPS / 2); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int i = 0; i < 3; ++i) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm.a[i])) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm.w[i])) : "memory");
        }
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool ok = true;
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 0) {
        // ---- TMA producer: one thread, six tiles per k-block
        if (lane == 0 && !g.test_drop_copies) {
            int stage = 0;
            uint32_t phase = 0;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int m0 = (tile / ntn) * BM, n0 = (tile % ntn) * BN;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait_relaxed(empty(stage), phase ^ 1u, limit_ns, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(full(stage), STAGE_BYTES);
                    const uint32_t base = s0 + stage * STAGE_BYTES;
#pragma unroll
                    for (int i = 0; i < 3; ++i) {
                        tma_load_2d(base + i * TILE_BYTES, &tm.a[i], full(stage), kb * BK, m0);
                        tma_load_2d(base + (3 + i) * TILE_BYTES, &tm.w[i], full(stage), kb * BK, n0);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    } else if (warp == 1) {
        // ---- MMA issuer: one thread; per 16-wide k-slice the six products, smallest first
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(BM, BN);
            int stage = 0, it = 0;
            uint32_t phase = 0;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++it) {
                const int buf = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(tempty(buf), acc_phase ^ 1u, limit_ns, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * BN;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(full(stage), phase, limit_ns, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t base = s0 + stage * STAGE_BYTES;
                    uint64_t ad[3], wd[3];
#pragma unroll
                    for (int i = 0; i < 3; ++i) { ad[i] = smem_desc(base + i * TILE_BYTES); wd[i] = smem_desc(base + (3 + i) * TILE_BYTES); }
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t off = (uint64_t)(k * UMMA_K * 2 / 16);
                        tc_mma(d_tmem, ad[2] + off, wd[0] + off, idesc, (kb | k) != 0 ? 1u : 0u);
                        tc_mma(d_tmem, ad[1] + off, wd[1] + off, idesc, 1u);
                        tc_mma(d_tmem, ad[0] + off, wd[2] + off, idesc, 1u);
                        tc_mma(d_tmem, ad[1] + off, wd[0] + off, idesc, 1u);
                        tc_mma(d_tmem, ad[0] + off, wd[1] + off, idesc, 1u);
                        tc_mma(d_tmem, ad[0] + off, wd[0] + off, idesc, 1u);
                    }
                    tc_commit(empty(stage));
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit(tfull(buf));
            }
        }
        __syncwarp();
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    } else {
        // ---- epilogue: warp w reads TMEM lanes 32 (w % 4) .. +31; one thread per row; fp32 outputs;
        // group (w - 2) / 4 owns accumulator (w - 2) / 4, i.e. every other tile of this CTA
        const int q = warp & 3, grp = (warp - 2) >> 2;
        float *stg = reinterpret_cast<float *>(smem + STAGES * STAGE_BYTES) + (warp - 2) * EPI_STAGE_FLOATS;
        int it = 0;
        for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++it) {
            const int buf = it & 1;
            if (buf != grp) continue;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            const int m0 = (tile / ntn) * BM, n0 = (tile % ntn) * BN;
            auto acc_ready = [&] { return __all_sync(0xffffffffu, mbar_wait_relaxed(tfull(buf), acc_phase, limit_ns, abort_flag)) != 0; };
            const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN);
            if (!epilogue_rows<EPI, 128, false, float, true>(g, tacc, m0 + q * 32, n0, stg, acc_ready)) { ok = false; break; }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty(buf));
        }
    }

    // ---- teardown
    if (!ok) {
        *abort_flag = 1;
        if (lane == 0) atomicExch(status, (int)7 /* EBRL_ERR_TIMEOUT */);
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        const unsigned long long t0 = gtimer();   // give copies still in flight time to land before shared memory is released
        while (gtimer() - t0 < 200000ull) { }
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// src [n] fp32 -> three bf16 planes whose sum is src (each term the bf16 rounding of what the previous ones left).
__global__ void __launch_bounds__(512) split3_kernel(const float4 *__restrict__ src, uint2 *__restrict__ p0, uint2 *__restrict__ p1,
                                                     uint2 *__restrict__ p2, size_t n4)
{
    pdl_launch_dependents();
    pdl_wait();
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        const float4 v = src[i];
        const float a[4] = {v.x, v.y, v.z, v.w};
        __nv_bfloat16 t0[4], t1[4], t2[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) split3(a[e], t0[e], t1[e], t2[e]);
        p0[i] = *reinterpret_cast<const uint2 *>(t0);
        p1[i] = *reinterpret_cast<const uint2 *>(t1);
        p2[i] = *reinterpret_cast<const uint2 *>(t2);
    }
}

}  // namespace tc3

bool gemm_tc3_supported(int N, int K) { return N % tc3::BN == 0 && K % tc3::BK == 0; }

cudaError_t launch_split3(const float *src, void *p0, void *p1, void *p2, size_t n, int grid, cudaStream_t st)
{
    if (n == 0) return cudaSuccess;
    if (n % 4) return cudaErrorInvalidValue;
    const size_t n4 = n / 4;
    size_t need = (n4 + 511) / 512;
    const int g = (int)(need < (size_t)grid ? need : (size_t)grid);
    return launch_kernel(tc3::split3_kernel, g, 512, 0, st, 1, reinterpret_cast<const float4 *>(src), reinterpret_cast<uint2 *>(p0),
                         reinterpret_cast<uint2 *>(p1), reinterpret_cast<uint2 *>(p2), n4);
}

template <int EPI>
static cudaError_t tc3_launch(const tc3::Maps6 &m, const GemmArgs &a, int g, unsigned long long limit_ns, int *status, cudaStream_t st)
{
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tc3::gemm_tc3_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc3::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    return launch_kernel(tc3::gemm_tc3_kernel<EPI>, g, tc3::THREADS, tc3::SMEM_BYTES, st, 1, m, a, limit_ns, status);
}

// ta[i] / tw[i]: descriptors of the i-th bf16 term of the activations [M][K] and of the weights [N][K] (128-row boxes).
cudaError_t launch_gemm_tc3(const TensorMap128 *ta, const TensorMap128 *tw, const GemmArgs &a, int grid, unsigned long long limit_ns,
                            int *status, cudaStream_t st)
{
    if (a.M == 0) return cudaSuccess;
    tc3::Maps6 m;
    for (int i = 0; i < 3; ++i) {
        m.a[i] = *reinterpret_cast<const CUtensorMap *>(&ta[i]);
        m.w[i] = *reinterpret_cast<const CUtensorMap *>(&tw[i]);
    }
    const int tiles = ((a.M + tc3::BM - 1) / tc3::BM) * (a.N / tc3::BN);
    const int g = tiles < grid ? tiles : grid;
    switch (a.epi) {
    case EPI_SCALE_STORE: return tc3_launch<EPI_SCALE_STORE>(m, a, g, limit_ns, status, st);
    case EPI_SCALE_GELU: return tc3_launch<EPI_SCALE_GELU>(m, a, g, limit_ns, status, st);
    default: return tc3_launch<EPI_RESID>(m, a, g, limit_ns, status, st);
    }
}

}  // namespace ebrl
