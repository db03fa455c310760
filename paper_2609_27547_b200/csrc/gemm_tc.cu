// bf16 x bf16 -> fp32 GEMM on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// tensor memory), operands staged in shared memory by TMA, with the path's fused epilogues:
// RMSNorm row scale, GELU, residual add, gain multiply for the next norm, and the fixed-width
// sum-of-squares partials.  C[M][N] = A[M][K] W[N][K]^T, both operands K-major.
//
// One persistent CTA per SM of the quota walks a static tile list (tile = blockIdx.x + i *
// gridDim.x).  Roles: warp 0 issues TMA loads into a 4-stage ring, warp 1 issues the MMAs and
// owns tensor memory, warps 2..5 run the epilogue of tile i from one 256-column accumulator
// while tile i+1 accumulates into the other.  Every output element is the sum over k in order
// in its own accumulator, so results do not depend on the grid size, on the tile a row falls
// in, or on which rows share it.  Every wait is bounded: on a time-out the CTA records
// EBRL_ERR_TIMEOUT in the status word, lets its copies land, frees tensor memory and returns.
#include "actgen_internal.h"
#include "ptx_helpers.cuh"
#include "gemm_epilogue.cuh"

#include <cuda.h>

namespace ebrl {

namespace tc {

using namespace ptx;

constexpr int BM = 128, BK = 64, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;

// Tile shapes: 128 x 256 (4 stages of 48 KB, 8 epilogue warps: lane quarter x column half) and
// 128 x 128 (6 stages of 32 KB, 4 epilogue warps) for GEMMs with too few tiles to fill the grid.
template <int BN> struct Shape {
    static constexpr int STAGES = BN == 256 ? 4 : 6;
    static constexpr int EPI_WARPS = BN / 128 * 4;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;   // TMA warp, MMA warp, epilogue warps
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int SMEM_BYTES = STAGES * (A_BYTES + B_BYTES) + 256 + 1024 + EPI_WARPS * EPI_STAGE_FLOATS * 4;   // + barriers + alignment slack
    static constexpr uint32_t TMEM_COLS = 2 * BN;
};

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
// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) with the
// 128-byte swizzle TMA wrote: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr)
{
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;               // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;     // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;               // descriptor version of sm_100
    d |= (uint64_t)2 << 61;               // 128-byte swizzle
    return d;
}
// kind::f16 instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, M x N.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

template <int EPI, int BN>
__global__ void __launch_bounds__(Shape<BN>::THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmC, GemmArgs g,
               unsigned long long limit_ns, int *status)
{
    constexpr int STAGES = Shape<BN>::STAGES, EPI_WARPS = Shape<BN>::EPI_WARPS, B_BYTES = Shape<BN>::B_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sA = smem_u32(smem), sB = sA + STAGES * A_BYTES;
    // after the stages: the epilogue warps' staging tiles (4 KB each, 1024-byte aligned), then the barriers
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + STAGES * (A_BYTES + B_BYTES) + EPI_WARPS * EPI_STAGE_FLOATS * 4);
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
        for (int b = 0; b < 2; ++b) { mbar_init(tfull(b), 1); mbar_init(tempty(b), EPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)), "r"(Shape<BN>::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool ok = true;
    pdl_launch_dependents();
    pdl_wait();   // set-up done; from here on the previous kernel's results are needed

    if (warp == 0) {
        // ---- TMA producer: one thread (no votes, fewer instructions between a free stage and its next copies)
        if (lane == 0 && !g.test_drop_copies) {
            int stage = 0;
            uint32_t phase = 0;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int m0 = (tile / ntn) * BM, n0 = (tile % ntn) * BN;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait_relaxed(empty(stage), phase ^ 1u, limit_ns, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(full(stage), A_BYTES + B_BYTES);
                    tma_load_2d(sA + stage * A_BYTES, &tmA, full(stage), kb * BK, m0);
                    tma_load_2d(sB + stage * B_BYTES, &tmB, full(stage), kb * BK, n0);   // weight rows n0 .. n0+127 (128-row boxes)
                    if (BN == 256) tma_load_2d(sB + stage * B_BYTES + B_BYTES / 2, &tmB, full(stage), kb * BK, n0 + 128);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    } else if (warp == 1) {
        // ---- MMA issuer: one thread
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(BM, BN);
            const uint64_t ad0 = smem_desc(sA), bd0 = smem_desc(sB);
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
                    // descriptors advance by whole stages and by 32 bytes per 16-wide k-slice (address field in 16-byte units)
                    const uint64_t ad = ad0 + (uint64_t)(stage * (A_BYTES >> 4)), bd = bd0 + (uint64_t)(stage * (B_BYTES >> 4));
                    tc_mma(d_tmem, ad, bd, idesc, kb != 0 ? 1u : 0u);
#pragma unroll
                    for (int k = 1; k < BK / UMMA_K; ++k)
                        tc_mma(d_tmem, ad + (uint64_t)(k * UMMA_K * 2 / 16), bd + (uint64_t)(k * UMMA_K * 2 / 16), idesc, 1u);
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
        // ---- epilogue: warp w reads TMEM lanes 32 (w % 4) .. +31 and half of the tile's columns; one thread per row
        const int q = warp & 3, half = (warp - 2) >> 2;   // half is 0 for the 128-column shape
        float *stg = reinterpret_cast<float *>(smem + STAGES * (A_BYTES + B_BYTES)) + (warp - 2) * EPI_STAGE_FLOATS;
        int it = 0;
        for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++it) {
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            const int m0 = (tile / ntn) * BM, n0 = (tile % ntn) * BN + half * 128;
            auto acc_ready = [&] { return __all_sync(0xffffffffu, mbar_wait_relaxed(tfull(buf), acc_phase, limit_ns, abort_flag)) != 0; };
            const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + half * 128);
            bool done;
            if constexpr (EPI == EPI_RESID) done = epilogue_rows<EPI, 128>(g, tacc, m0 + q * 32, n0, stg, acc_ready);
            else done = epilogue_store_tma<EPI, 128>(g, &tmC, tacc, m0 + q * 32, n0, stg, acc_ready);
            if (!done) {
                ok = false;
                break;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty(buf));
        }
        if (EPI != EPI_RESID && lane == 0) epilogue_store_drain();
    }

    // ---- teardown
    if (!ok) {
        *abort_flag = 1;
        if (lane == 0) atomicExch(status, (int)7 /* EBRL_ERR_TIMEOUT */);
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        // give copies that were still in flight time to land before shared memory is released
        const unsigned long long t0 = gtimer();
        while (gtimer() - t0 < 200000ull) { }
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Shape<BN>::TMEM_COLS) : "memory");
    }
}

}  // namespace tc

// ---- host side -------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 tensor map of a row-major [rows][inner] matrix, box = 64 x box_rows, 128-byte swizzle.
int make_tmap_bf16(TensorMap128 *out, const void *base, uint64_t inner, uint64_t rows, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return 1;
    static_assert(sizeof(TensorMap128) == sizeof(CUtensorMap), "tensor map size");
    const cuuint64_t dims[2] = {inner, rows};
    const cuuint64_t strides[1] = {inner * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(reinterpret_cast<CUtensorMap *>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides,
                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : 2;
}

bool gemm_tc_supported(int N, int K) { return N % 256 == 0 && K % tc::BK == 0; }
int gemm_tc_box_rows_a() { return tc::BM; }
int gemm_tc_box_rows_w() { return 128; }   // weight maps serve every kernel: 128-row boxes

template <int EPI, int BN>
static cudaError_t tc_launch(const TensorMap128 &ta, const TensorMap128 &tw, const TensorMap128 &tc_, const GemmArgs &a, int g,
                             unsigned long long limit_ns, int *status, cudaStream_t st)
{
    // the attribute belongs to the function on ONE device: set it once per device
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tc::gemm_tc_kernel<EPI, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::Shape<BN>::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    return launch_kernel(tc::gemm_tc_kernel<EPI, BN>, g, tc::Shape<BN>::THREADS, tc::Shape<BN>::SMEM_BYTES, st, 1,
                         *reinterpret_cast<const CUtensorMap *>(&ta), *reinterpret_cast<const CUtensorMap *>(&tw),
                         *reinterpret_cast<const CUtensorMap *>(&tc_), a, limit_ns, status);
}

// One CTA per tile; bn = 256 or 128 columns per tile.
cudaError_t launch_gemm_tc(const TensorMap128 &ta, const TensorMap128 &tw, const GemmArgs &a, int grid, int bn, unsigned long long limit_ns,
                           int *status, cudaStream_t st)
{
    if (a.M == 0) return cudaSuccess;
    // the store epilogues write C through the copy engine: a descriptor of C as [M][N], boxes of 32 rows x 64 columns
    TensorMap128 tcm = ta;
    if (a.epi != EPI_RESID && make_tmap_bf16(&tcm, a.C, (uint64_t)a.N, (uint64_t)a.M, 32)) return cudaErrorInvalidValue;
    const int tiles = ((a.M + tc::BM - 1) / tc::BM) * (a.N / bn);
    const int g = tiles < grid ? tiles : grid;
    if (bn == 256) {
        switch (a.epi) {
        case EPI_SCALE_STORE: return tc_launch<EPI_SCALE_STORE, 256>(ta, tw, tcm, a, g, limit_ns, status, st);
        case EPI_SCALE_GELU: return tc_launch<EPI_SCALE_GELU, 256>(ta, tw, tcm, a, g, limit_ns, status, st);
        default: return tc_launch<EPI_RESID, 256>(ta, tw, tcm, a, g, limit_ns, status, st);
        }
    }
    switch (a.epi) {
    case EPI_SCALE_STORE: return tc_launch<EPI_SCALE_STORE, 128>(ta, tw, tcm, a, g, limit_ns, status, st);
    case EPI_SCALE_GELU: return tc_launch<EPI_SCALE_GELU, 128>(ta, tw, tcm, a, g, limit_ns, status, st);
    default: return tc_launch<EPI_RESID, 128>(ta, tw, tcm, a, g, limit_ns, status, st);
    }
}

}  // namespace ebrl
