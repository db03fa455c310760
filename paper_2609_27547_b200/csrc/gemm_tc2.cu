// The tensor-core GEMM on CTA pairs: two CTAs of a cluster (two SMs) compute one 256 x 256 tile
// with tcgen05.mma.cta_group::2.  Each CTA stages its own 128 rows of A and only HALF of the
// weight tile (128 of its 256 rows) per k-block, so the bytes an SM pulls from L2 per FLOP drop
// by a third compared with one CTA per 128 x 256 tile -- the single-CTA kernel is bound by that
// L2 -> SM traffic.  The leader CTA (rank 0 of the pair) issues the MMAs for both; each CTA
// reads its own 128 accumulator rows from its own tensor memory and runs the same epilogue as
// the single-CTA kernel.  Same arithmetic per output element, same bounded waits.
//
// Barriers: full[s] of the LEADER collects the copy bytes of both CTAs; empty[s] and tfull[b]
// live in each CTA and are signalled by the leader's tcgen05.commit multicast; tempty[b] of the
// leader counts the epilogue warps of both CTAs (the peer arrives remotely).
#include "actgen_internal.h"
#include "ptx_helpers.cuh"
#include "gemm_epilogue.cuh"
#include "pair_helpers.cuh"

#include <cuda.h>

namespace ebrl {
namespace tc2 {

using namespace ptx;
using namespace tc;
using namespace pairx;

constexpr int BM = 128;          // rows per CTA (256 per pair)
constexpr int BN = 256;          // columns per pair tile
constexpr int BNH = 128;         // weight rows staged per CTA
constexpr int BK = 64, UMMA_K = 16, STAGES = 6;
constexpr int THREADS = 320;          // TMA warp, MMA warp, 8 epilogue warps
constexpr int EPI_WARPS = 8;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BNH * BK * 2;
constexpr int SMEM_BYTES = STAGES * (A_BYTES + B_BYTES) + 256 + 1024 + EPI_WARPS * EPI_STAGE_FLOATS * 4;

template <int EPI>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmC, GemmArgs g,
                unsigned long long limit_ns, int *status)
{
    extern __shared__ uint8_t smem_raw[];
    // the same offset in both CTAs of the pair: the dynamic shared window starts at the same
    // address in every CTA of a kernel, so rounding up gives matching layouts
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
    const uint32_t rank = cluster_rank();          // 0 = leader
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int ntm = (g.M + 2 * BM - 1) / (2 * BM), ntn = g.N / BN, ntiles = ntm * ntn, nkb = g.K / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull(b), 1); mbar_init(tempty(b), 2 * EPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
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
        // ---- TMA producer (both CTAs), one thread: own A rows, own half of the weight tile; bytes land on the
        // leader's barrier.  (One thread instead of a converged warp: fewer instructions between a stage
        // falling free and its next copies, and no issue slots spent on votes.)
        if (lane == 0 && !g.test_drop_copies) {
            int stage = 0;
            uint32_t phase = 0;
            for (int tile = pair; tile < ntiles && ok; tile += npairs) {
                const int m0 = (tile / ntn) * (2 * BM) + (int)rank * BM, n0 = (tile % ntn) * BN + (int)rank * BNH;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait_relaxed(empty(stage), phase ^ 1u, limit_ns, abort_flag)) { ok = false; break; }
                    if (rank == 0) mbar_expect_tx(full(stage), 2 * (A_BYTES + B_BYTES));
                    const uint32_t lead_full = mapa(full(stage), 0);
                    tma_load_2d_pair(sA + stage * A_BYTES, &tmA, lead_full, kb * BK, m0);
                    tma_load_2d_pair(sB + stage * B_BYTES, &tmB, lead_full, kb * BK, n0);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    } else if (warp == 1) {
        // ---- MMA issuer: one thread of the leader, for both CTAs
        if (rank == 0 && lane == 0) {
            constexpr uint32_t idesc = instr_desc_bf16(2 * BM, BN);
            const uint64_t ad0 = smem_desc_sw128(sA), bd0 = smem_desc_sw128(sB);
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
                    // descriptors advance by whole stages and by 32 bytes per 16-wide k-slice (address field in 16-byte units)
                    const uint64_t ad = ad0 + (uint64_t)(stage * (A_BYTES >> 4)), bd = bd0 + (uint64_t)(stage * (B_BYTES >> 4));
                    tc_mma_pair(d_tmem, ad, bd, idesc, kb != 0 ? 1u : 0u);
#pragma unroll
                    for (int k = 1; k < BK / UMMA_K; ++k)
                        tc_mma_pair(d_tmem, ad + (uint64_t)(k * UMMA_K * 2 / 16), bd + (uint64_t)(k * UMMA_K * 2 / 16), idesc, 1u);
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
        float *stg = reinterpret_cast<float *>(smem + STAGES * (A_BYTES + B_BYTES)) + (warp - 2) * EPI_STAGE_FLOATS;
        int it = 0;
        for (int tile = pair; tile < ntiles && ok; tile += npairs, ++it) {
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            const int m0 = (tile / ntn) * (2 * BM) + (int)rank * BM, n0 = (tile % ntn) * BN + half * (BN / 2);
            auto acc_ready = [&] { return __all_sync(0xffffffffu, mbar_wait_relaxed(tfull(buf), acc_phase, limit_ns, abort_flag)) != 0; };
            const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + half * (BN / 2));
            bool done;
            if constexpr (EPI == EPI_RESID) done = epilogue_rows<EPI, BN / 2>(g, tacc, m0 + q * 32, n0, stg, acc_ready);
            else done = epilogue_store_tma<EPI, BN / 2>(g, &tmC, tacc, m0 + q * 32, n0, stg, acc_ready);
            if (!done) {
                ok = false;
                break;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa(tempty(buf), 0));
        }
        if (EPI != EPI_RESID && lane == 0) epilogue_store_drain();
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

}  // namespace tc2

template <int EPI>
static cudaError_t tc2_launch(const TensorMap128 &ta, const TensorMap128 &tw, const TensorMap128 &tc_, const GemmArgs &a, int g,
                              unsigned long long limit_ns, int *status, cudaStream_t st)
{
    // the attribute belongs to the function on ONE device: set it once per device
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tc2::gemm_tc2_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc2::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    return launch_kernel(tc2::gemm_tc2_kernel<EPI>, g, tc2::THREADS, tc2::SMEM_BYTES, st, 2, *reinterpret_cast<const CUtensorMap *>(&ta),
                         *reinterpret_cast<const CUtensorMap *>(&tw), *reinterpret_cast<const CUtensorMap *>(&tc_), a, limit_ns, status);
}

// grid = SM quota; the kernel uses floor(grid / 2) CTA pairs.  Needs grid >= 2.
cudaError_t launch_gemm_tc2(const TensorMap128 &ta, const TensorMap128 &tw, const GemmArgs &a, int grid, unsigned long long limit_ns,
                            int *status, cudaStream_t st)
{
    if (a.M == 0) return cudaSuccess;
    // the store epilogues write C through the copy engine: a descriptor of C as [M][N], boxes of 32 rows x 64 columns
    TensorMap128 tcm = ta;
    if (a.epi != EPI_RESID && make_tmap_bf16(&tcm, a.C, (uint64_t)a.N, (uint64_t)a.M, 32)) return cudaErrorInvalidValue;
    const int tiles = ((a.M + 2 * tc2::BM - 1) / (2 * tc2::BM)) * (a.N / tc2::BN);
    int pairs = grid / 2;
    if (pairs > tiles) pairs = tiles;
    const int g = 2 * pairs;
    switch (a.epi) {
    case EPI_SCALE_STORE: return tc2_launch<EPI_SCALE_STORE>(ta, tw, tcm, a, g, limit_ns, status, st);
    case EPI_SCALE_GELU: return tc2_launch<EPI_SCALE_GELU>(ta, tw, tcm, a, g, limit_ns, status, st);
    default: return tc2_launch<EPI_RESID>(ta, tw, tcm, a, g, limit_ns, status, st);
    }
}

}  // namespace ebrl
