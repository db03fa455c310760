// Softmax attention for the bf16 models: the H (<= 16) query tokens of one environment against
// its keys/values -- the cached prefix planes (cross-attention) or its own H rows of the QKV
// buffer (self-attention).  The kernel is bandwidth-shaped: every K/V element is used by only H
// queries, so the planes are streamed once through shared memory.  Each environment's planes
// are described by a 3-D TMA descriptor (64-column group, row, group index) whose box covers a
// whole slab of heads for a block of keys, so one copy instruction moves 32 KB and lands it as
// [group][key][128 B] tiles with the 128-byte swizzle: ldmatrix reads them conflict-free.  The
// small contractions run on mma.sync (m16n8k16, bf16 in, fp32 accumulate) with the softmax
// statistics kept per row by quad shuffles.
//
// Work item = (environment, slab of up to 8 heads); one warp per head; a ninth warp issues the
// copies into a 3-stage ring.  Keys are visited in blocks of 16 in index order with a running
// maximum and sum, so an environment's result does not depend on the grid size or on what else
// is in the batch.  Every wait is bounded (status word, as in the GEMM).
#include "actgen_internal.h"
#include "ptx_helpers.cuh"

#include <cuda.h>
#include <cstdlib>

namespace ebrl {
namespace am {

using namespace ptx;

constexpr int NSTAGE = 3;
// consumer warps = heads per slab: 8 heads of 128 columns or 16 heads of 64 -- a slab is 1024 columns (16 keys per
// stage) either way, and the narrower heads, whose softmax costs twice as much per byte, get twice the warps to hide it
__host__ __device__ constexpr int maxw(int hd) { return hd == 64 ? 16 : 8; }
constexpr int STAGE_ROWS_BYTES = 32768; // payload bytes of K (and of V) per stage

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Keys per stage for a slab of W columns: a whole number of 16-key blocks within the stage budget.
__host__ __device__ inline int stage_keys(int W) { int k = STAGE_ROWS_BYTES / (W * 2); k &= ~15; return k < 16 ? 16 : (k > 64 ? 64 : k); }

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void *tmap, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// 4 x 4 transpose of 32-bit words across the four lanes of a quad: on return r[c] of lane t holds what
// lane c had in r[t].
__device__ __forceinline__ void quad_transpose(uint32_t (&r)[4], int t)
{
    const bool odd = t & 1, hi = t & 2;
    uint32_t x = __shfl_xor_sync(0xffffffffu, odd ? r[0] : r[1], 1);
    uint32_t y = __shfl_xor_sync(0xffffffffu, odd ? r[2] : r[3], 1);
    if (odd) { r[0] = x; r[2] = y; } else { r[1] = x; r[3] = y; }
    x = __shfl_xor_sync(0xffffffffu, hi ? r[0] : r[2], 2);
    y = __shfl_xor_sync(0xffffffffu, hi ? r[1] : r[3], 2);
    if (hi) { r[0] = x; r[1] = y; } else { r[2] = x; r[3] = y; }
}

template <int HD>
__global__ void __launch_bounds__((maxw(HD) + 1) * 32, 1) attn_mma_kernel(AttnArgs a, int hpc, int la_blocks, unsigned long long limit_ns, int *status)
{
    constexpr int MAXW = maxw(HD);
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int W = hpc * HD;                       // slab width in columns
    const int G = W / 64;                         // 64-column groups per slab
    const int KB = stage_keys(W);                 // keys per stage (a multiple of 16)
    const int stage_bytes = G * KB * 128;         // one box: [G][KB][128 B]
    const uint32_t sK = smem_u32(smem), sV = sK + NSTAGE * stage_bytes;
    const uint32_t sQ = sV + NSTAGE * stage_bytes;   // per consumer warp: its head's queries, [16 rows][HD] bf16, 16-byte chunks swizzled
    constexpr int Q_BYTES = 16 * HD * 2;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + 2 * NSTAGE * stage_bytes + MAXW * Q_BYTES);
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (NSTAGE + s); };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * NSTAGE);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int H = a.H, nslab = a.n_heads / hpc, items = a.n_envs * nslab;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), hpc); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_launch_dependents();
    pdl_wait();

    bool ok = true;

    if (warp == MAXW) {
        // ---- producer: per key block one box of K and one of V (rows past the planes' end are
        // zero-filled by the copy; rows of the V plane read through the K box are masked later).
        // A second cursor runs `la_blocks` key blocks ahead and asks L2 to fetch those boxes, so
        // that the bytes in flight from HBM are not bounded by the three stages of the ring.
        int stage = 0;
        uint32_t phase = 0;
        auto locate = [&](int item, const void *&tm, int &P, int &krow, int &vrow, int &kgrp, int &vgrp) {
            const int env = item / nslab, slab = item - env * nslab;
            if (a.self) {
                tm = a.self_map; P = H;
                krow = vrow = env * H;
                kgrp = (a.d + slab * W) / 64; vgrp = (2 * a.d + slab * W) / 64;
            } else {
                tm = a.kv_maps + env; P = a.meta[env].P;
                const int pr = a.plane_rows ? a.plane_rows : P;
                krow = a.kv_plane * 2 * pr; vrow = krow + pr;
                kgrp = vgrp = slab * G;
            }
        };
        // look-ahead cursor
        int la_item = blockIdx.x, la_j0 = 0, la_P = 0, la_krow = 0, la_vrow = 0, la_kgrp = 0, la_vgrp = 0;
        const void *la_tm = nullptr;
        const bool use_la = la_blocks > 0 && !a.self;
        auto la_step = [&]() {
            if (la_item >= items) return;
            if (lane == 0) {
                asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global [%0, {%1, %2, %3}];"
                             ::"l"(reinterpret_cast<uint64_t>(la_tm)), "r"(0), "r"(la_krow + la_j0), "r"(la_kgrp) : "memory");
                asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global [%0, {%1, %2, %3}];"
                             ::"l"(reinterpret_cast<uint64_t>(la_tm)), "r"(0), "r"(la_vrow + la_j0), "r"(la_vgrp) : "memory");
            }
            la_j0 += KB;
            if (la_j0 >= la_P) {
                la_item += gridDim.x; la_j0 = 0;
                if (la_item < items) locate(la_item, la_tm, la_P, la_krow, la_vrow, la_kgrp, la_vgrp);
            }
        };
        if (use_la && la_item < items) {
            locate(la_item, la_tm, la_P, la_krow, la_vrow, la_kgrp, la_vgrp);
            for (int i = 0; i < la_blocks; ++i) la_step();
        }
        for (int item = blockIdx.x; item < items && ok && !a.test_drop_copies; item += gridDim.x) {
            const void *tm;
            int P, krow, vrow, kgrp, vgrp;
            locate(item, tm, P, krow, vrow, kgrp, vgrp);
            if (!a.self) {
                // descriptors are rewritten by the host between batches: drop any stale cached copy
                if (lane == 0) asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(reinterpret_cast<uint64_t>(tm)) : "memory");
                __syncwarp();
            }
            for (int j0 = 0; j0 < P; j0 += KB) {
                if (use_la) la_step();
                if (!__all_sync(0xffffffffu, mbar_wait_relaxed(empty(stage), phase ^ 1u, limit_ns, abort_flag))) { ok = false; break; }
                if (lane == 0) {
                    mbar_expect_tx(full(stage), (uint32_t)(2 * stage_bytes));
                    tma_load_3d(sK + stage * stage_bytes, tm, full(stage), 0, krow + j0, kgrp);
                    tma_load_3d(sV + stage * stage_bytes, tm, full(stage), 0, vrow + j0, vgrp);
                }
                __syncwarp();
                if (++stage == NSTAGE) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp < hpc) {
        // ---- consumers: warp = head within the slab
        const int g = lane >> 2, t = lane & 3;
        const float sc = 1.4426950408889634f / sqrtf((float)HD);   // log2(e) / sqrt(hd): scores in base-2 units
        int qbase = 0;                                              // stages consumed by earlier items
        const uint32_t myq = sQ + (uint32_t)warp * Q_BYTES;
        for (int i = lane; i < Q_BYTES / 16; i += 32)               // rows >= H are never copied: keep them zero
            asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(myq + (uint32_t)i * 16), "r"(0u) : "memory");
        __syncwarp();
        // asynchronous copy of one item's queries of this warp's head: chunk c of row r goes to c ^ (r & 7)
        auto fetch_q = [&](int it) {
            const int e2 = it / nslab, hd2 = (it - e2 * nslab) * hpc + warp;
            const __nv_bfloat16 *qb = (const __nv_bfloat16 *)a.q + (size_t)e2 * H * a.q_stride + hd2 * HD;
            constexpr int CPR = HD / 8;   // 16-byte chunks per row
            for (int idx = lane; idx < H * CPR; idx += 32) {
                const int r = idx / CPR, cch = idx % CPR;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(myq + (uint32_t)(r * (HD * 2) + ((cch ^ (r & 7)) << 4))),
                             "l"(qb + (size_t)r * a.q_stride + cch * 8) : "memory");
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        if ((int)blockIdx.x < items) fetch_q(blockIdx.x);
        const int bps_sh = KB == 16 ? 0 : (KB == 32 ? 1 : 2), bps_mask = (1 << bps_sh) - 1;   // 16-key blocks per stage: 1, 2 or 4
        for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
            const int env = item / nslab, slab = item - env * nslab;
            const int P = a.self ? H : a.meta[env].P;
            const int head = slab * hpc + warp;
            // Q fragments (A operand, 16 x HD; rows >= H stay zero): this item's queries were copied
            // into the warp's buffer asynchronously while the previous item was processed
            uint32_t qf[HD / 16][4];
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncwarp();
#pragma unroll
            for (int ks = 0; ks < HD / 16; ++ks) {
                const int qr = (lane & 7) + ((lane >> 3) & 1) * 8, qc = 2 * ks + (lane >> 4);
                ldsm_x4(myq + (uint32_t)(qr * (HD * 2) + ((qc ^ (qr & 7)) << 4)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
            }
            __syncwarp();
            if (item + (int)gridDim.x < items) fetch_q(item + gridDim.x);   // lands during this item
            float o[HD / 8][4];
#pragma unroll
            for (int n = 0; n < HD / 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
            float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // rows g and g + 8
            const int g0 = warp * (HD / 64);   // first 64-column group of this warp's head
            const int nblk = (P + 15) >> 4;                // 16-key blocks in this item; BPS = 1 << bps_sh of them per stage
            // stage of block b: ring slot (qbase + (b >> bps_sh)) % NSTAGE, parity ((qbase + (b >> bps_sh)) / NSTAGE) & 1
            auto qk = [&](int b, float (&s0)[4], float (&s1)[4]) {
                const int qs = qbase + (b >> bps_sh);
                const uint32_t kst = sK + (uint32_t)(qs % NSTAGE) * stage_bytes;
                const int r = (b & bps_mask) * 16 + (lane >> 4) * 8 + (lane & 7);   // key row within the stage; r & 7 == lane & 7
                const int ch = (lane >> 3) & 1;                                  // 16-byte chunk within the k-step
                auto kaddr = [&](int ks) {   // tile [group][KB rows][128 B], chunk index XOR (row & 7)
                    return kst + (uint32_t)(((g0 + (ks >> 2)) * KB + r) * 128 + (((((ks & 3) << 1) | ch) ^ (lane & 7)) << 4));
                };
                // four accumulation chains per n-tile (k-steps modulo 4), added pairwise at the end: the block's
                // score latency is two dependent MMAs instead of four (the ring holds a stage for about two
                // block times, so latency on the consumers' chain costs bandwidth: 193.5 -> 190.2 ms)
                float acc[4][2][4];
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[c][0][i] = acc[c][1][i] = 0.f;
#pragma unroll
                for (int ks = 0; ks < HD / 16; ks += 2) {
                    uint32_t b0, b1, b2, b3, c0, c1, c2, c3;
                    ldsm_x4(kaddr(ks), b0, b1, b2, b3);
                    ldsm_x4(kaddr(ks + 1), c0, c1, c2, c3);
                    mma_bf16(acc[ks & 3][0], qf[ks], b0, b1);
                    mma_bf16(acc[ks & 3][1], qf[ks], b2, b3);
                    mma_bf16(acc[(ks + 1) & 3][0], qf[ks + 1], c0, c1);
                    mma_bf16(acc[(ks + 1) & 3][1], qf[ks + 1], c2, c3);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    s0[i] = (acc[0][0][i] + acc[1][0][i]) + (acc[2][0][i] + acc[3][0][i]);
                    s1[i] = (acc[0][1][i] + acc[1][1][i]) + (acc[2][1][i] + acc[3][1][i]);
                }
            };
            auto wait_block = [&](int b) -> bool {   // first block of a stage: wait until the copies have landed
                if (b & bps_mask) return true;
                const int qs = qbase + (b >> bps_sh);
                // one lane polls the barrier (32 lanes polling the same word are 32 shared-memory operations per
                // round, beside the copies and the ldmatrix traffic); the warp-level exchange orders the others
                // behind it.  (The same change in the producer's sleeping wait measured 10 % slower.)
                int landed = 1;
                if (lane == 0) landed = mbar_wait(full(qs % NSTAGE), (uint32_t)(qs / NSTAGE) & 1u, limit_ns, abort_flag) ? 1 : 0;
                return __shfl_sync(0xffffffffu, landed, 0) != 0;
            };
            for (int b = 0; b < nblk; ++b) {
                // A block's Q K^T is issued when its stage is needed, not a block early: touching the next
                // stage early keeps two of the three stages occupied and only one in flight, and the ring --
                // not the arithmetic -- sets the kernel's speed (190 -> 173 ms on the large configuration).
                float s0[4], s1[4];
                if (!wait_block(b)) { ok = false; break; }
                qk(b, s0, s1);
                // running max / sum per row on the raw scores (the scale log2(e)/sqrt(hd) is positive and is
                // folded into the exponent); keys past the prefix are masked, which only the last block needs
                // the first V fragments are requested before the softmax so that P V can start the moment P exists
                const int qs = qbase + (b >> bps_sh);
                const uint32_t vst = sV + (uint32_t)(qs % NSTAGE) * stage_bytes;
                const int vr = (b & bps_mask) * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
                auto vaddr = [&](int n) {
                    const int col0 = n * 8 + (lane >> 4) * 8;   // first column of this lane's 8x8 matrix within the head
                    return vst + (uint32_t)(((g0 + (col0 >> 6)) * KB + vr) * 128 + ((((col0 & 63) >> 3) ^ (lane & 7)) << 4));
                };
                constexpr int NPRE = 2;   // measured: two loads ahead 169 -> 165 ms, four no better
                uint32_t vf[NPRE][4];
#pragma unroll
                for (int i = 0; i < NPRE; ++i) ldsm_x4_t(vaddr(2 * i), vf[i][0], vf[i][1], vf[i][2], vf[i][3]);
                float v[8] = {s0[0], s0[1], s0[2], s0[3], s1[0], s1[1], s1[2], s1[3]};
                if (b == nblk - 1) {
                    const int kleft = P - b * 16;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int key = (e >> 2) * 8 + 2 * t + (e & 1);
                        if (key >= kleft) v[e] = -INFINITY;
                    }
                }
                float mx0 = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[4], v[5]));
                float mx1 = fmaxf(fmaxf(v[2], v[3]), fmaxf(v[6], v[7]));
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
                const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
                const bool rescale = __any_sync(0xffffffffu, (mn0 != m0) || (mn1 != m1));   // warp-uniform
                float al0 = 1.f, al1 = 1.f;
                if (rescale) { al0 = ex2((m0 - mn0) * sc); al1 = ex2((m1 - mn1) * sc); }
                m0 = mn0; m1 = mn1;
                const float ms0 = -mn0 * sc, ms1 = -mn1 * sc;
                float p[8];
                p[0] = ex2(fmaf(v[0], sc, ms0)); p[1] = ex2(fmaf(v[1], sc, ms0)); p[4] = ex2(fmaf(v[4], sc, ms0)); p[5] = ex2(fmaf(v[5], sc, ms0));
                p[2] = ex2(fmaf(v[2], sc, ms1)); p[3] = ex2(fmaf(v[3], sc, ms1)); p[6] = ex2(fmaf(v[6], sc, ms1)); p[7] = ex2(fmaf(v[7], sc, ms1));
                l0 = l0 * al0 + ((p[0] + p[1]) + (p[4] + p[5]));
                l1 = l1 * al1 + ((p[2] + p[3]) + (p[6] + p[7]));
                uint32_t pf[4];
                pf[0] = pack2(p[0], p[1]); pf[1] = pack2(p[2], p[3]); pf[2] = pack2(p[4], p[5]); pf[3] = pack2(p[6], p[7]);
                // O = O * alpha + P V   (alpha is exactly 1 in every lane when no row maximum moved)
                if (rescale) {
#pragma unroll
                    for (int n = 0; n < HD / 8; ++n) { o[n][0] *= al0; o[n][1] *= al0; o[n][2] *= al1; o[n][3] *= al1; }
                }
#pragma unroll
                for (int i = 0; i < NPRE; ++i) {
                    mma_bf16(o[2 * i], pf, vf[i][0], vf[i][1]);
                    mma_bf16(o[2 * i + 1], pf, vf[i][2], vf[i][3]);
                }
#pragma unroll
                for (int n = 2 * NPRE; n < HD / 8; n += 2) {
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4_t(vaddr(n), b0, b1, b2, b3);
                    mma_bf16(o[n], pf, b0, b1);
                    mma_bf16(o[n + 1], pf, b2, b3);
                }
                if ((b & bps_mask) == bps_mask || b == nblk - 1) {   // last block of its stage: hand the stage back
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty(qs % NSTAGE));
                }
            }
            qbase += (nblk + bps_mask) >> bps_sh;
            if (!ok) break;
            // row sums across the quad, normalise, store
            l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
            const float i0 = 1.0f / l0, i1 = 1.0f / l1;
            // The accumulator fragment gives a lane two adjacent columns of each 8-column tile.  Four tiles
            // at a time are transposed across the quad (lane t ends up with all 8 columns of tile 4 j + t),
            // so that a lane stores 16 contiguous bytes and a warp instruction fills whole 32-byte sectors.
            __nv_bfloat16 *ob = (__nv_bfloat16 *)a.out + (size_t)env * H * a.o_stride + head * HD + 8 * t;
#pragma unroll
            for (int j = 0; j < HD / 32; ++j) {
                uint32_t r0[4], r1[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    r0[k] = pack2(o[4 * j + k][0] * i0, o[4 * j + k][1] * i0);
                    r1[k] = pack2(o[4 * j + k][2] * i1, o[4 * j + k][3] * i1);
                }
                quad_transpose(r0, t);
                quad_transpose(r1, t);
                if (g < H) *reinterpret_cast<uint4 *>(ob + (size_t)g * a.o_stride + j * 32) = make_uint4(r0[0], r0[1], r0[2], r0[3]);
                if (g + 8 < H) *reinterpret_cast<uint4 *>(ob + (size_t)(g + 8) * a.o_stride + j * 32) = make_uint4(r1[0], r1[1], r1[2], r1[3]);
            }
        }
    }

    if (!ok) {
        *abort_flag = 1;
        if (lane == 0) atomicExch(status, 7 /* EBRL_ERR_TIMEOUT */);
    }
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        const unsigned long long t0 = gtimer();   // let copies still in flight land
        while (gtimer() - t0 < 200000ull) { }
    }
    __syncthreads();
}

}  // namespace am

// Heads per slab (= consumer warps that work): as many as the kernel has warps for -- 16 heads of 64 columns or 8 of
// 128 -- when `wide`; 8 otherwise (the persistent step kernel reads the same descriptors and has 8 attention warps).
int attn_mma_slab_heads(int n_heads, int hd, bool wide)
{
    const int top = wide ? am::maxw(hd) : 8;
    if (n_heads <= top) return n_heads;
    if (n_heads % top == 0) return top;
    return 8;
}
// Shapes the kernel covers: bf16, H <= 16, head_dim 64 or 128, heads a multiple of the slab.
bool attn_mma_supported(int H, int n_heads, int hd)
{
    if (H > 16 || (hd != 64 && hd != 128)) return false;
    return n_heads % attn_mma_slab_heads(n_heads, hd, false) == 0;
}

typedef CUresult (*EncodeTiledFn3)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                   const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 3-D descriptor of a row-major bf16 matrix [rows][width] seen as (64-column group, row, group
// index): box = one slab of heads x one stage of keys, 128-byte swizzle, zero fill out of range.
int attn_mma_make_map(TensorMap128 *out, const void *base, uint64_t rows, uint64_t width, int hpc, int hd)
{
    static EncodeTiledFn3 fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) return 1;
        fn = reinterpret_cast<EncodeTiledFn3>(p);
    }
    const int W = hpc * hd;
    const cuuint64_t dims[3] = {64, rows, width / 64};
    const cuuint64_t strides[2] = {width * 2, 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)am::stage_keys(W), (cuuint32_t)(W / 64)};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(reinterpret_cast<CUtensorMap *>(out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box,
                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : 2;
}

// hpc = heads per slab, as in the descriptors; la = L2 look-ahead of the producer in key blocks (0 disables).
cudaError_t launch_attn_mma(const AttnArgs &a, int grid, int hpc, int la, unsigned long long limit_ns, int *status, cudaStream_t st)
{
    const int items = a.n_envs * (a.n_heads / hpc);
    if (items == 0) return cudaSuccess;
    const int g = items < grid ? items : grid;
    const int W = hpc * a.hd;
    const size_t smem = (size_t)2 * am::NSTAGE * am::stage_keys(W) * (W / 64) * 128 + (size_t)am::maxw(a.hd) * 16 * a.hd * 2 + 64 + 1024;
    cudaError_t e;
    if (a.hd == 128) {
        e = cudaFuncSetAttribute(am::attn_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        return launch_kernel(am::attn_mma_kernel<128>, g, (am::maxw(128) + 1) * 32, smem, st, 1, a, hpc, la, limit_ns, status);
    } else {
        e = cudaFuncSetAttribute(am::attn_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        return launch_kernel(am::attn_mma_kernel<64>, g, (am::maxw(64) + 1) * 32, smem, st, 1, a, hpc, la, limit_ns, status);
    }
    return cudaGetLastError();
}

}  // namespace ebrl
