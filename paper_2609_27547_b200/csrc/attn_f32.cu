// Softmax attention for the fp32 models (head_dim 64, up to 8 query tokens): one WARP per
// (environment, head) item, no shared state between warps and no block-wide barrier.
//
// The contraction is tiny -- 8 query rows against P keys of 64 columns -- so what decides the
// speed is how many operand fetches an FMA costs.  Here the query block lives in registers for
// the whole item and every key / value element fetched from shared memory feeds 8 FMAs:
//
//   lane = (key slot k4 = lane / 8, column group cq = lane % 8); a lane owns the 8 columns
//   4 cq .. 4 cq + 3 and 32 + 4 cq .. 32 + 4 cq + 3 of every row it touches;
//   q[8 rows][8 columns]   registers, scaled by 1 / sqrt(head_dim), loaded once per item
//   o[8 rows][8 columns]   registers, this lane's share of the output over ITS keys
//   scores: 8 partial dot products per lane and key (64 FMAs on two 16-byte reads of the key),
//   folded across the 8 column groups by a halving exchange (7 shuffles) that leaves the score
//   of row rho(cq) with lane cq; values: the 8 weights of the key are gathered back (8
//   shuffles) for 64 FMAs on two 16-byte reads.  The FMAs are issued two per instruction
//   (f32x2 on column pairs): the kernel is bound by issue slots, not by the FMA pipe.
//
// Keys and values stream through a per-warp ring of 16-key stages filled by cp.async (zero fill
// past the prefix), so a warp's global-memory latency hides behind its own arithmetic and the
// eight warps of a CTA never wait on one another.  The copies run two stages ahead across item
// boundaries (an item's first stage carries its query block), so short prefixes and the 8-key
// self-attention do not pay a round trip to memory per item.  Keys are visited in blocks of 16 in index
// order with a running maximum and sum; an item's arithmetic involves nothing but the item, so
// the result does not depend on the grid size or on what else is in the batch.
#include "actgen_internal.h"
#include "split3.cuh"
#include "f32x2.cuh"

#include <cuda_runtime.h>
#include <math.h>

namespace ebrl {
namespace af {

constexpr int HD = 64;            // head_dim
constexpr int ROWS = 8;           // query rows held per item
constexpr int WARPS = 8;          // items in flight per CTA
constexpr int SK = 16;            // keys per stage
constexpr int NST = 3;            // stages per warp
constexpr int PLANE_FLOATS = SK * HD;
constexpr int STAGE_FLOATS = 2 * PLANE_FLOATS;                 // keys, then values
constexpr int WARP_FLOATS = NST * STAGE_FLOATS + 2 * ROWS * HD;   // a warp's ring and its two query blocks: 28 KB
constexpr int SMEM_BYTES = WARPS * (WARP_FLOATS * 4 + 16);         // plus the prefix lengths of those two items
constexpr unsigned FULL = 0xffffffffu;

__device__ __forceinline__ void cp16(uint32_t dst, const void *src, uint32_t nbytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(nbytes) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// The score fold: 8 partial sums per lane (one per query row) are added over the 8 lanes that differ in lane
// bits 0..2 by three halving exchanges (4 + 2 + 1 shuffles): with lane ^ 1 a lane hands over four rows and keeps
// four, with lane ^ 2 two and two, with lane ^ 4 one and one.  Which rows a lane keeps follows its bits: it ends
// with the total of row rho(lane % 8) = 4 bit0 + 2 bit1 + bit2 (the bit reversal of its column group).
// rho is its own inverse (the column group whose lane holds row r) and distributes over xor
__device__ __forceinline__ int rho(int r) { return ((r >> 2) & 1) | (r & 2) | ((r & 1) << 2); }

// Where the copies of a warp stand: the next stage to request belongs to block b of `item`.
struct Cursor {
    int item, seq, b, nblk, P, kvs;     // seq = how many items this warp has started before this one
    const float *kbase, *vbase, *qg;
};

__global__ void __launch_bounds__(WARPS * 32, 1) attn_f32_kernel(AttnArgs a)
{
    extern __shared__ __align__(16) float smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k4 = lane >> 3, cq = lane & 7;
    float *ring = smem + (size_t)warp * WARP_FLOATS;
    float *qring = ring + NST * STAGE_FLOATS;                  // two query blocks: items alternate
    int *pmeta = reinterpret_cast<int *>(smem + (size_t)WARPS * WARP_FLOATS) + warp * 4;   // their prefix lengths
    const uint32_t ring_u = (uint32_t)__cvta_generic_to_shared(ring), qring_u = (uint32_t)__cvta_generic_to_shared(qring);
    const int H = a.H;
    const float qs = 1.4426950408889634f / sqrtf((float)HD);   // scores in units of log 2: the weights are exp2
    const int items = a.n_envs * a.n_heads, stride = gridDim.x * WARPS;
    const int perm = rho(cq);
    pdl_launch_dependents();
    pdl_wait();

    auto seek = [&](Cursor &c, int item) {
        c.item = item; c.b = 0;
        if (item >= items) return;
        const int env = item / a.n_heads, h = item - env * a.n_heads;
        if (a.self) {
            c.kbase = (const float *)a.k_self + (size_t)env * H * a.kv_stride + h * HD;
            c.vbase = (const float *)a.v_self + (size_t)env * H * a.kv_stride + h * HD;
            c.P = H; c.kvs = a.kv_stride;
        } else {
            const EnvMeta m = a.meta[env];
            c.P = m.P; c.kvs = a.d;
            const int pr = a.plane_rows ? a.plane_rows : m.P;
            c.kbase = (const float *)m.kv + (size_t)a.kv_plane * 2 * pr * a.d + h * HD;
            c.vbase = c.kbase + (size_t)pr * a.d;
        }
        c.nblk = c.P > SK ? (c.P + SK - 1) / SK : 1;
        c.qg = (const float *)a.q + (size_t)env * H * a.q_stride + h * HD;
    };
    // Requests the cursor's stage into ring slot `slot` (16 keys x 256 bytes of each plane, 16 bytes per copy, two
    // keys per warp instruction; an item's first stage brings its query block and prefix length along) and moves
    // the cursor on, into the next item when this one is exhausted.  One commit group per call, empty at the end.
    auto issue_next = [&](Cursor &c, int slot) {
        if (c.item < items) {
            const uint32_t dst = ring_u + (uint32_t)(slot * STAGE_FLOATS * 4);
            if (c.b == 0) {
                const uint32_t qdst = qring_u + (uint32_t)((c.seq & 1) * ROWS * HD * 4);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int ch = lane + 32 * u, r = ch >> 4, col = (ch & 15) << 2;
                    cp16(qdst + (uint32_t)((r * HD + col) * 4), c.qg + (size_t)(r < H ? r : 0) * a.q_stride + col, r < H ? 16u : 0u);
                }
                if (lane == 0) pmeta[c.seq & 1] = c.P;
            }
            if (c.b * SK + SK <= c.P) {   // a whole stage: no predicates
                const size_t row0 = (size_t)c.b * SK * c.kvs;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int ch = lane + 32 * u, key = ch >> 4, col = (ch & 15) << 2;
                    cp16(dst + (uint32_t)((key * HD + col) * 4), c.kbase + row0 + (size_t)key * c.kvs + col, 16u);
                    cp16(dst + (uint32_t)((PLANE_FLOATS + key * HD + col) * 4), c.vbase + row0 + (size_t)key * c.kvs + col, 16u);
                }
            } else {                      // the last, partial stage: keys past the prefix are filled with zeros
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int ch = lane + 32 * u, key = ch >> 4, col = (ch & 15) << 2;
                    const bool in = c.b * SK + key < c.P;
                    const size_t src = (size_t)(in ? c.b * SK + key : 0) * c.kvs + col;
                    cp16(dst + (uint32_t)((key * HD + col) * 4), c.kbase + src, in ? 16u : 0u);
                    cp16(dst + (uint32_t)((PLANE_FLOATS + key * HD + col) * 4), c.vbase + src, in ? 16u : 0u);
                }
            }
            if (++c.b == c.nblk) {
                const int seq = c.seq + 1;
                seek(c, c.item + stride);
                c.seq = seq;
            }
        }
        cp_commit();
    };

    // The copies run NST - 1 stages ahead of the arithmetic, across item boundaries: while an item's last blocks
    // are computed the next item's first blocks (and queries) are already on their way.
    Cursor ic;
    ic.seq = 0;
    seek(ic, blockIdx.x * WARPS + warp);
    int g = 0;   // stages computed so far by this warp; stage g lives in ring slot g % NST
#pragma unroll
    for (int t = 0; t < NST - 1; ++t) issue_next(ic, t);

    int seq = 0;
    for (int item = blockIdx.x * WARPS + warp; item < items; item += stride, ++seq) {
        const int env = item / a.n_heads, h = item - env * a.n_heads;
        // rows in a lane-dependent order: register i holds row i ^ perm.  The halving exchanges of the score fold then
        // keep the low registers and send the high ones in EVERY lane (no selects), and the lane that owns the
        // weight of register i's row is simply lane ^ rho(i).
        uint64_t q2[ROWS][4], o2[ROWS][4];
#pragma unroll
        for (int i = 0; i < ROWS; ++i)
#pragma unroll
            for (int c = 0; c < 4; ++c) o2[i][c] = 0ull;
        float mrun = -INFINITY, lrun = 0.f;   // running maximum and (this lane's keys') sum of row rho(cq)
        int P = 0, nblk = 1;

        for (int b = 0; b < nblk; ++b, ++g) {
            cp_wait<NST - 2>();      // this lane's copies of stage g have landed ...
            __syncwarp();            // ... and so have the other lanes'; everyone is done with stage g - 1
            if (b == 0) {
                P = pmeta[seq & 1];
                nblk = P > SK ? (P + SK - 1) / SK : 1;
                const float *qsm = qring + (seq & 1) * ROWS * HD;
#pragma unroll
                for (int i = 0; i < ROWS; ++i) {
                    const float4 lo = *reinterpret_cast<const float4 *>(qsm + (i ^ perm) * HD + 4 * cq);
                    const float4 hi = *reinterpret_cast<const float4 *>(qsm + (i ^ perm) * HD + 32 + 4 * cq);
                    q2[i][0] = pk2(lo.x * qs, lo.y * qs); q2[i][1] = pk2(lo.z * qs, lo.w * qs);
                    q2[i][2] = pk2(hi.x * qs, hi.y * qs); q2[i][3] = pk2(hi.z * qs, hi.w * qs);
                }
                __syncwarp();        // every lane has read the queries and the prefix length before anyone's copies replace them
            }
            issue_next(ic, (g + NST - 1) % NST);   // into the slot of stage g - 1 (and, for a new item, over the queries
                                                   // and prefix length of the item before this one: read above)
            const float *ks = ring + (g % NST) * STAGE_FLOATS, *vs = ks + PLANE_FLOATS;
            float s[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int key = 4 * j + k4;
                const ulonglong2 klo = *reinterpret_cast<const ulonglong2 *>(ks + key * HD + 4 * cq);
                const ulonglong2 khi = *reinterpret_cast<const ulonglong2 *>(ks + key * HD + 32 + 4 * cq);
                float part[ROWS];
#pragma unroll
                for (int i = 0; i < ROWS; ++i) {
                    uint64_t t = mul2(q2[i][0], klo.x);
                    t = fma2(q2[i][1], klo.y, t); t = fma2(q2[i][2], khi.x, t); t = fma2(q2[i][3], khi.y, t);
                    float te, to;
                    upk2(t, te, to);
                    part[i] = te + to;
                }
                // fold across the eight column groups: 4 + 2 + 1 exchanges, register 0 ends as the score of row rho(cq)
#pragma unroll
                for (int i = 0; i < 4; ++i) part[i] += __shfl_xor_sync(FULL, part[i + 4], 1);
#pragma unroll
                for (int i = 0; i < 2; ++i) part[i] += __shfl_xor_sync(FULL, part[i + 2], 2);
                const float sc = part[0] + __shfl_xor_sync(FULL, part[1], 4);
                s[j] = (b * SK + key < P) ? sc : -INFINITY;
            }
            // running softmax statistics of row rho(cq): the block's maximum over this lane's four keys and the
            // four key slots (the block's first key always exists, so the maximum is finite)
            float bm = fmaxf(fmaxf(s[0], s[1]), fmaxf(s[2], s[3]));
            bm = fmaxf(bm, __shfl_xor_sync(FULL, bm, 8));
            bm = fmaxf(bm, __shfl_xor_sync(FULL, bm, 16));
            const float mnew = fmaxf(mrun, bm);
            const float al = exp2f(mrun - mnew);
            float p[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) p[j] = exp2f(s[j] - mnew);
            lrun = lrun * al + ((p[0] + p[1]) + (p[2] + p[3]));
            mrun = mnew;
            if (__any_sync(FULL, al != 1.0f)) {   // once the maxima have settled every factor is exactly 1
#pragma unroll
                for (int i = 0; i < ROWS; ++i) {
                    const float ar = __shfl_xor_sync(FULL, al, rho(i));
                    const uint64_t aa = pk2(ar, ar);
#pragma unroll
                    for (int c = 0; c < 4; ++c) o2[i][c] = mul2(o2[i][c], aa);
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int key = 4 * j + k4;
                const ulonglong2 vlo = *reinterpret_cast<const ulonglong2 *>(vs + key * HD + 4 * cq);
                const ulonglong2 vhi = *reinterpret_cast<const ulonglong2 *>(vs + key * HD + 32 + 4 * cq);
#pragma unroll
                for (int i = 0; i < ROWS; ++i) {
                    const float pr = __shfl_xor_sync(FULL, p[j], rho(i));   // weight of (register i's row, this lane's key)
                    const uint64_t pp = pk2(pr, pr);
                    o2[i][0] = fma2(pp, vlo.x, o2[i][0]); o2[i][1] = fma2(pp, vlo.y, o2[i][1]);
                    o2[i][2] = fma2(pp, vhi.x, o2[i][2]); o2[i][3] = fma2(pp, vhi.y, o2[i][3]);
                }
            }
        }
        float o[ROWS][8];
#pragma unroll
        for (int i = 0; i < ROWS; ++i)
#pragma unroll
            for (int c = 0; c < 4; ++c) upk2(o2[i][c], o[i][2 * c], o[i][2 * c + 1]);
        // totals over the four key slots (lane bits 3 and 4): the row sums everywhere, the outputs by two
        // halving exchanges that leave registers 4 bit3 + 2 bit4 + {0, 1} (rows: those ^ perm) with the lane
        lrun += __shfl_xor_sync(FULL, lrun, 8);
        lrun += __shfl_xor_sync(FULL, lrun, 16);
        const bool b3 = lane & 8, b4 = lane & 16;
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float send = b3 ? o[i][c] : o[i + 4][c], keep = b3 ? o[i + 4][c] : o[i][c];
                o[i][c] = keep + __shfl_xor_sync(FULL, send, 8);
            }
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float send = b4 ? o[i][c] : o[i + 2][c], keep = b4 ? o[i + 2][c] : o[i][c];
                o[i][c] = keep + __shfl_xor_sync(FULL, send, 16);
            }
        const int rbase = (b3 ? 4 : 0) + (b4 ? 2 : 0);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int r = (rbase + i) ^ perm;
            const float lr = __shfl_sync(FULL, lrun, rho(r));
            if (r < H) {
                const size_t off = (size_t)(env * H + r) * a.o_stride + h * HD + 4 * cq;
                float v[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) v[c] = o[i][c] / lr;
                if (a.split_out) {   // the three bf16 terms of the result, for the tensor-core projection that follows
                    store_split4(a.out, a.out_t1, a.out_t2, off, v[0], v[1], v[2], v[3]);
                    store_split4(a.out, a.out_t1, a.out_t2, off + 32, v[4], v[5], v[6], v[7]);
                } else {
                    *reinterpret_cast<float4 *>((float *)a.out + off) = make_float4(v[0], v[1], v[2], v[3]);
                    *reinterpret_cast<float4 *>((float *)a.out + off + 32) = make_float4(v[4], v[5], v[6], v[7]);
                }
            }
        }
    }
    cp_wait<0>();   // only empty groups are left
}

}  // namespace af

// Shapes the warp-per-item kernel covers (fp32 planes and activations).
bool attn_f32_supported(int H, int hd) { return hd == af::HD && H >= 1 && H <= af::ROWS; }

// grid = SM quota; each CTA keeps eight items in flight.
cudaError_t launch_attn_f32(const AttnArgs &a, int grid, cudaStream_t st)
{
    const int items = a.n_envs * a.n_heads;
    if (items == 0) return cudaSuccess;
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(af::attn_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, af::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const int need = (items + af::WARPS - 1) / af::WARPS;
    const int g = need < grid ? need : grid;
    return launch_kernel(af::attn_f32_kernel, g, af::WARPS * 32, af::SMEM_BYTES, st, 1, a);
}

}  // namespace ebrl
