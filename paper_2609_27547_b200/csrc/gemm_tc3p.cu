// The fp32 models' tensor-core GEMM (three-term bf16 operand splitting, six products per k-slice:
// see gemm_tc3.cu) on CTA pairs: two CTAs of a cluster compute one 256 x 256 tile with
// tcgen05.mma.cta_group::2.  Each CTA stages the three term planes of its own 128 rows of A and of
// HALF of the weight tile (128 of its 256 rows) per 64-wide k-block -- 96 KB per stage, two stages --
// so an SM takes in half the operand bytes per FLOP of the single-CTA 128 x 128 kernel, which is
// bound by operand delivery.  The leader CTA issues the MMAs for both; each CTA drains its own 128
// accumulator rows with the same fused epilogues (fp32 outputs, term planes for the next projection).
// Every output element is the sum over k in order of its six products in the same order as in the
// single-CTA kernel: results are bit-identical between the two, whatever the grid.
//
// Barriers as in the bf16 pair kernel: full[s] of the LEADER collects the copy bytes of both CTAs;
// empty[s] and tfull[b] live in each CTA and are signalled by the leader's tcgen05.commit multicast;
// tempty[b] of the leader counts the epilogue warps of both CTAs.  Every wait is bounded.
#include "actgen_internal.h"
#include "ptx_helpers.cuh"
#include "gemm_epilogue.cuh"
#include "pair_helpers.cuh"

#include <cuda.h>

namespace ebrl {
namespace tc3p {

using namespace ptx;
using namespace tc;
using namespace pairx;

constexpr int BM = 128;          // rows per CTA (256 per pair)
constexpr int BN = 256;          // columns per pair tile
constexpr int BNH = 128;         // weight rows staged per CTA
constexpr int BK = 64, UMMA_K = 16, STAGES = 2;
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 64 + 32 * EPI_WARPS;          // TMA warp, MMA warp, 8 epilogue warps
constexpr int TILE_BYTES = BM * BK * 2;                // one bf16 operand tile of 128 rows
constexpr int STAGE_BYTES = 6 * TILE_BYTES;            // A0 A1 A2 W0 W1 W2 (this CTA's rows of each)
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * EPI_STAGE_FLOATS * 4 + 256 + 1024;

struct Maps6 {
    CUtensorMap a[3], w[3];
};

template <int EPI>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc3p_kernel(const __grid_constant__ Maps6 tm, GemmArgs g, unsigned long long limit_ns, int *status)
{
    extern __shared__ uint8_t smem_raw[];
    // the same offset in both CTAs of the pair (the dynamic shared window starts at the same address in every CTA)
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
    const uint32_t rank = cluster_rank();          // 0 = leader
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int ntm = (g.M + 2 * BM - 1) / (2 * BM), ntn = g.N / BN, ntiles = ntm * ntn, nkb = g.K / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull(b), 1); mbar_init(tempty(b), 2 * EPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int i = 0; i < 3; ++i) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm.a[i])) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm.w[i])) : "memory");
        }
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void *)tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();      // barriers of both CTAs initialised, tensor memory of both allocated
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool ok = true;
    pdl_launch_dependents();
    pdl_wait();   // set-up done; from here on the previous kernel's results are needed

    if (warp == 0) {
        // ---- TMA producer (both CTAs), one thread: the term planes of its own A rows and of its half of the weight
        // tile; the bytes land on the leader's barrier
        if (lane == 0 && !g.test_drop_copies) {
            int stage = 0;
            uint32_t phase = 0;
            for (int tile = pair; tile < ntiles && ok; tile += npairs) {
                const int m0 = (tile / ntn) * (2 * BM) + (int)rank * BM, n0 = (tile % ntn) * BN + (int)rank * BNH;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait_relaxed(empty(stage), phase ^ 1u, limit_ns, abort_flag)) { ok = false; break; }
                    if (rank == 0) mbar_expect_tx(full(stage), 2 * STAGE_BYTES);
                    const uint32_t lead_full = mapa(full(stage), 0);
                    const uint32_t base = s0 + stage * STAGE_BYTES;
#pragma unroll
                    for (int i = 0; i < 3; ++i) {
                        tma_load_2d_pair(base + i * TILE_BYTES, &tm.a[i], lead_full, kb * BK, m0);
                        tma_load_2d_pair(base + (3 + i) * TILE_BYTES, &tm.w[i], lead_full, kb * BK, n0);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    } else if (warp == 1) {
        // ---- MMA issuer: one thread of the leader, for both CTAs; per 16-wide k-slice the six products, smallest first
        if (rank == 0 && lane == 0) {
            constexpr uint32_t idesc = instr_desc_bf16(2 * BM, BN);
            int stage = 0, it = 0;
            uint32_t phase = 0;
            for (int tile = pair; tile < ntiles && ok; tile += npairs, ++it) {
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
                    for (int i = 0; i < 3; ++i) { ad[i] = smem_desc_sw128(base + i * TILE_BYTES); wd[i] = smem_desc_sw128(base + (3 + i) * TILE_BYTES); }
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t off = (uint64_t)(k * UMMA_K * 2 / 16);
                        tc_mma_pair(d_tmem, ad[2] + off, wd[0] + off, idesc, (kb | k) != 0 ? 1u : 0u);
                        tc_mma_pair(d_tmem, ad[1] + off, wd[1] + off, idesc, 1u);
                        tc_mma_pair(d_tmem, ad[0] + off, wd[2] + off, idesc, 1u);
                        tc_mma_pair(d_tmem, ad[1] + off, wd[0] + off, idesc, 1u);
                        tc_mma_pair(d_tmem, ad[0] + off, wd[1] + off, idesc, 1u);
                        tc_mma_pair(d_tmem, ad[0] + off, wd[0] + off, idesc, 1u);
                    }
                    tc_commit_pair(empty(stage));     // frees the stage in both CTAs
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit_pair(tfull(buf));  // accumulators of both CTAs are complete
            }
        }
        __syncwarp();
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    } else {
        // ---- epilogue (both CTAs): own 128 rows of the pair tile; each warp a lane quarter and half of the columns
        const int q = warp & 3, half = (warp - 2) >> 2;
        float *stg = reinterpret_cast<float *>(smem + STAGES * STAGE_BYTES) + (warp - 2) * EPI_STAGE_FLOATS;
        int it = 0;
        for (int tile = pair; tile < ntiles && ok; tile += npairs, ++it) {
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            const int m0 = (tile / ntn) * (2 * BM) + (int)rank * BM, n0 = (tile % ntn) * BN + half * (BN / 2);
            auto acc_ready = [&] { return __all_sync(0xffffffffu, mbar_wait_relaxed(tfull(buf), acc_phase, limit_ns, abort_flag)) != 0; };
            const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + half * (BN / 2));
            if (!epilogue_rows<EPI, BN / 2, false, float, true>(g, tacc, m0 + q * 32, n0, stg, acc_ready)) { ok = false; break; }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa(tempty(buf), 0));
        }
    }

    // ---- teardown: nobody leaves while its partner may still touch its memory
    if (!ok) {
        *abort_flag = 1;
        if (lane == 0) atomicExch(status, 7 /* EBRL_ERR_TIMEOUT */);
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        const unsigned long long t0 = gtimer();   // give copies still in flight time to land
        while (gtimer() - t0 < 200000ull) { }
    }
    __syncthreads();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

}  // namespace tc3p

bool gemm_tc3p_supported(int N, int K) { return N % tc3p::BN == 0 && K % tc3p::BK == 0; }

template <int EPI>
static cudaError_t tc3p_launch(const tc3p::Maps6 &m, const GemmArgs &a, int g, unsigned long long limit_ns, int *status, cudaStream_t st)
{
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tc3p::gemm_tc3p_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc3p::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    return launch_kernel(tc3p::gemm_tc3p_kernel<EPI>, g, tc3p::THREADS, tc3p::SMEM_BYTES, st, 2, m, a, limit_ns, status);
}

// grid = SM quota; the kernel uses floor(grid / 2) CTA pairs.  Needs grid >= 2 and N a multiple of 256.
// ta[i] / tw[i]: descriptors of the i-th bf16 term of the activations [M][K] and of the weights [N][K] (128-row boxes).
cudaError_t launch_gemm_tc3p(const TensorMap128 *ta, const TensorMap128 *tw, const GemmArgs &a, int grid, unsigned long long limit_ns,
                             int *status, cudaStream_t st)
{
    if (a.M == 0) return cudaSuccess;
    tc3p::Maps6 m;
    for (int i = 0; i < 3; ++i) {
        m.a[i] = *reinterpret_cast<const CUtensorMap *>(&ta[i]);
        m.w[i] = *reinterpret_cast<const CUtensorMap *>(&tw[i]);
    }
    const int tiles = ((a.M + 2 * tc3p::BM - 1) / (2 * tc3p::BM)) * (a.N / tc3p::BN);
    int pairs = grid / 2;
    if (pairs > tiles) pairs = tiles;
    const int g = 2 * pairs;
    switch (a.epi) {
    case EPI_SCALE_STORE: return tc3p_launch<EPI_SCALE_STORE>(m, a, g, limit_ns, status, st);
    case EPI_SCALE_GELU: return tc3p_launch<EPI_SCALE_GELU>(m, a, g, limit_ns, status, st);
    default: return tc3p_launch<EPI_RESID>(m, a, g, limit_ns, status, st);
    }
}

}  // namespace ebrl
