// The persistent action-head kernel: ONE resident grid of at most `sm_quota` CTAs runs every
// Euler step of a batch -- embedding, the layers' six projections, self- and cross-attention, the
// velocity head and the Euler update -- by walking a static task list.  It serves the small-group
// regime, where the per-operation kernels are bound by launches and by the fill and drain of each
// grid rather than by arithmetic (the paper's "each denoising step launches small kernels").
//
// Tasks.  Every operation of a step is cut into tasks: a 128 x 128 output tile of a projection,
// one (environment, slab of 8 heads) item of an attention, one 128-row block of the embedding or
// of the head.  Tasks are numbered in path order (operation-major, row-block-major inside an
// operation) and task t belongs to CTA t mod gridDim.x; each CTA takes its tasks in order.
//
// Dependencies.  A task needs the previous operation's results for its 128-row block only, so a
// row block can run ahead of the others: there is one completion counter per (Euler step, row
// block), raised by every warp that finishes its part of a task on that block, and a task waits
// until the counter has reached what all earlier operations of the step contribute to the block
// (a closed formula).  Because every task waits only for tasks with smaller numbers and all CTAs
// are resident (cooperative launch), the walk cannot deadlock.  Every wait is bounded: on a
// time-out the CTA records EBRL_ERR_TIMEOUT in the status word, which the other CTAs poll, lets
// its copies land, frees tensor memory and returns.
//
// Roles per CTA (320 threads): warp 0 = one thread issuing TMA copies into a ring of six 32 KB
// slots (a projection k-block = 16 KB of A + 16 KB of W; an attention key block = one slot of K and
// one of V), running ahead of the other roles across task boundaries -- weight tiles are requested
// before the task's dependency is even satisfied; warp 1 = one thread issuing tcgen05.mma into
// two 128-column accumulators in tensor memory; warps 2..9 = two groups of four epilogue warps
// (tile i is drained by group i mod 2 while tile i+1 accumulates), which are also the eight
// attention consumers (one head each, mma.sync + online softmax) and the row workers of the
// embedding and the head.
//
// Arithmetic.  Every output element is computed by the same instruction sequence as in the
// per-operation kernels (same accumulation order over k, same epilogue functions, same key-block
// order, same row routines), so the two paths deliver identical bits and the result does not
// depend on the grid size.  Data another CTA produced during the kernel is read through L2
// (TMA, cp.async.cg, ld.global.cg), never through this SM's L1.
#include "actgen_internal.h"
#include "ptx_helpers.cuh"
#include "gemm_epilogue.cuh"
#include "rowops.cuh"

#include <cuda.h>
#include <algorithm>

namespace ebrl {
namespace fs {

using namespace ptx;
using namespace tc;

constexpr int BM = 128, BN = 128, BK = 64, UMMA_K = 16;
constexpr int NST = 6, SLOT_BYTES = 32768;
constexpr int A_BYTES = BM * BK * 2;
constexpr int WORKERS = 8, THREADS = (2 + WORKERS) * 32;
constexpr int STG_BYTES = 4096;                      // per worker warp: epilogue staging tile / attention queries
constexpr int SMEM_BYTES = NST * SLOT_BYTES + WORKERS * STG_BYTES + 512 + 1024;
constexpr uint32_t TMEM_COLS = 2 * BN;

enum { OP_EMBED = 0, OP_GEMM = 1, OP_ATTN = 2, OP_HEAD = 3 };

// Event log, compiled in only for tuning builds (-DEBRL_FUSED_PROF): {type, global task number, cta, globaltimer} for the
// tasks of row block 0 in the first step, behind the progress notes.
#ifdef EBRL_FUSED_PROF
#define PROF_EVT(type, o, t, m) if (f.trace && (o).s == 0 && (m) == 0) { \
        int *lg_ = f.trace + 4 * 256 + 2 * 12 * 4 * 256; const int i_ = atomicAdd(lg_, 1); \
        if (i_ < 4000) { long long *e_ = reinterpret_cast<long long *>(lg_ + 4) + 2 * i_; \
            e_[0] = ((long long)(type) << 48) | ((long long)cta << 32) | (unsigned)((o).base + (t)); e_[1] = (long long)gtimer(); } }
#else
#define PROF_EVT(type, o, t, m)
#endif

struct OpDesc {
    int kind, s, ne, M, MT;
    int ntasks, base;                      // tasks of this operation, global number of its first task
    int dep_step, dep_fixed, dep_attn, dep_ne;   // wait: done[dep_step][m] >= dep_fixed + dep_attn * n_heads * envs_in_block(dep_ne, m)
    const CUtensorMap *tmA, *tmW, *tmC;    // projections
    int N, K, epi;
    const float *gain;
    void *C;
    int self, layer;                       // attention
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, uint32_t bar, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void *tmap, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
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
// K-major tile with 128-byte rows in the 128-byte swizzle TMA wrote: 8-row groups 1024 bytes apart.
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
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ int ld_acquire(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_relaxed(const int *p)
{
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Bounded wait for a completion counter.  false: the limit ran out, or this or another CTA gave up.
__device__ __forceinline__ bool wait_counter(const int *ctr, int target, unsigned long long limit_ns, volatile int *abort_flag,
                                             const int *status)
{
    if (ld_acquire(ctr) >= target) return true;
    const unsigned long long t0 = gtimer();
    for (;;) {
        // plain polls (one load in flight per poller), then one acquiring load to order what follows
        for (int i = 0; i < 64; ++i) {
            if (ld_relaxed(ctr) >= target) return ld_acquire(ctr) >= target;
            __nanosleep(100);
        }
        if (*abort_flag || ld_relaxed(status) != 0) return false;
        if (gtimer() - t0 > limit_ns) return false;
    }
}
// Where a bounded wait gave up (first failure of the launch only): words 1..3 of the status block get the site,
// the task and a detail, which ebrl_actgen_sync puts into the error text.
__device__ __forceinline__ void note_failure(int *status, int site, int kind, int s, int task, int detail)
{
    if (atomicCAS(status + 1, 0, (int)(0x40000000u | (unsigned)site | ((unsigned)kind << 8) | ((unsigned)s << 12))) == 0) {
        status[2] = task;
        status[3] = detail;
    }
}
// A warp has finished its part of a task on a row block: its writes (by any lane, through the generic
// proxy) become visible device-wide, to plain loads and to TMA, before the counter moves.
__device__ __forceinline__ void signal_block(int *ctr, int lane)
{
    fence_proxy_async_global();     // each lane's generic-proxy writes before any later TMA read of them
    __syncwarp();                   // orders the other lanes' writes before lane 0's release (which is cumulative)
    if (lane == 0) asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(ctr) : "memory");
}

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
// Keys per slot for a slab of W columns (the same rule as the per-operation attention kernel's ring stage).
__host__ __device__ inline int slot_keys(int W) { int k = SLOT_BYTES / (W * 2); k &= ~15; return k < 16 ? 16 : (k > 64 ? 64 : k); }

__device__ __forceinline__ int envs_in_block(int ne, int m, int epb)
{
    const int left = ne - m * epb;
    return left < epb ? (left < 0 ? 0 : left) : epb;
}

// Calls fn(op) for every operation of the batch in path order; every role of every CTA walks the same list.
template <typename F>
__device__ __forceinline__ bool walk_ops(const FusedArgs &f, F &&fn)
{
    const int nt_d = f.d / BN, nt_qkv = 3 * f.d / BN, nt_md = f.md / BN;
    const int nslab = f.n_heads / f.hpc;
    const int layer_fixed = 4 * (nt_qkv + 4 * nt_d + nt_md);
    const int step_fixed = WORKERS + f.n_layers * layer_fixed + WORKERS, step_attn = 2 * f.n_layers;
    const CUtensorMap *a_xg = reinterpret_cast<const CUtensorMap *>(&f.maps->a_xg);
    const CUtensorMap *a_att = reinterpret_cast<const CUtensorMap *>(&f.maps->a_att);
    const CUtensorMap *a_u = reinterpret_cast<const CUtensorMap *>(&f.maps->a_u);
    int base = 0;
    for (int s = 0; s < f.S; ++s) {
        const int ne = f.n_active[s];
        if (ne == 0) break;
        OpDesc o{};
        o.s = s; o.ne = ne; o.M = ne * f.H; o.MT = (o.M + BM - 1) / BM;
        int cum_fixed = 0, cum_attn = 0;
        auto emit = [&](int ntasks) {
            o.ntasks = ntasks; o.base = base;
            const bool go = fn(o);
            base += ntasks;
            return go;
        };
        auto dep_here = [&]() { o.dep_step = s; o.dep_fixed = cum_fixed; o.dep_attn = cum_attn; o.dep_ne = ne; };
        // embedding: needs the previous step's head on the same rows
        o.kind = OP_EMBED;
        if (s > 0) { o.dep_step = s - 1; o.dep_fixed = step_fixed; o.dep_attn = step_attn; o.dep_ne = f.n_active[s - 1]; }
        else { o.dep_step = -1; o.dep_fixed = o.dep_attn = 0; o.dep_ne = ne; }
        if (!emit(o.MT)) return false;
        cum_fixed += WORKERS;
        for (int l = 0; l < f.n_layers; ++l) {
            const FusedLayerTab *L = f.layers + l;
            auto gemm = [&](const CUtensorMap *tmA, const TensorMap128 *tmW, const TensorMap128 *tmC, int N, int K, int epi, void *C,
                            const float *gain) {
                o.kind = OP_GEMM; o.tmA = tmA; o.tmW = reinterpret_cast<const CUtensorMap *>(tmW);
                o.tmC = reinterpret_cast<const CUtensorMap *>(tmC); o.N = N; o.K = K; o.epi = epi; o.C = C; o.gain = gain;
                dep_here();
                const bool go = emit(o.MT * (N / BN));
                cum_fixed += 4 * (N / BN);
                return go;
            };
            auto attn = [&](int self) {
                o.kind = OP_ATTN; o.self = self; o.layer = l;
                dep_here();
                const bool go = emit(ne * nslab);
                cum_attn += 1;
                return go;
            };
            if (!gemm(a_xg, &L->t_qkv, &f.maps->c_qkv, 3 * f.d, f.d, EPI_SCALE_STORE, f.qkv, nullptr)) return false;
            if (!attn(1)) return false;
            if (!gemm(a_att, &L->t_o, nullptr, f.d, f.d, EPI_RESID, nullptr, L->g2)) return false;
            if (!gemm(a_xg, &L->t_qc, &f.maps->c_qc, f.d, f.d, EPI_SCALE_STORE, f.qc, nullptr)) return false;
            if (!attn(0)) return false;
            if (!gemm(a_att, &L->t_oc, nullptr, f.d, f.d, EPI_RESID, nullptr, L->g3)) return false;
            if (!gemm(a_xg, &L->t_1, &f.maps->c_u, f.md, f.d, EPI_SCALE_GELU, f.u, nullptr)) return false;
            if (!gemm(a_u, &L->t_2, nullptr, f.d, f.md, EPI_RESID, nullptr, (l + 1 < f.n_layers) ? f.layers[l + 1].g1 : f.g_final))
                return false;
        }
        o.kind = OP_HEAD;
        dep_here();
        if (!emit(o.MT)) return false;
    }
    return true;
}

// One attention item for one head: the consumer of the per-operation attention kernel, reading its key and value
// blocks from ring slots sc0, sc0 + 1, ... (K and V of a block of KBk keys in consecutive slots).  Kept out of line so
// that the compiler gives its inner loop the whole register budget instead of sharing it with the task walker's state.
struct AttnItem {
    const __nv_bfloat16 *qb;   // this head's queries [H][q_stride]
    __nv_bfloat16 *ob;         // this head's outputs [H][o_stride]
    int q_stride, o_stride, H, P, KBk, g0, sc0;
    uint32_t slots, full_a0, empty_a0, myq, pa;
    unsigned long long limit_ns;
    volatile int *abort_flag;
};
// returns 0, or 1 + the slot number whose copy never landed
template <int HD>
__device__ __noinline__ int attn_item(AttnItem &ai, int lane)
{
    const int H = ai.H, P = ai.P, KBk = ai.KBk, g0 = ai.g0, sc0 = ai.sc0;
    const uint32_t slots = ai.slots, myq = ai.myq;
    uint32_t pa = ai.pa;
    const unsigned long long limit_ns = ai.limit_ns;
    volatile int *abort_flag = ai.abort_flag;
    const float sc2 = 1.4426950408889634f / sqrtf((float)HD);   // log2(e) / sqrt(hd): scores in base-2 units
    const int bps_sh = KBk == 16 ? 0 : (KBk == 32 ? 1 : 2), bps_mask = (1 << bps_sh) - 1;   // 16-key blocks per slot
    const int nblk = (P + 15) >> 4;
    const int g8 = lane >> 2, tq = lane & 3;
    constexpr int Q_BYTES = 16 * HD * 2, CPR = HD / 8;
    // rows >= H of the query tile are never copied: zero them (the tile doubles as epilogue staging)
    for (int i = H * CPR + lane; i < Q_BYTES / 16; i += 32)
        asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(myq + (uint32_t)i * 16), "r"(0u) : "memory");
    __syncwarp();
    for (int idx = lane; idx < H * CPR; idx += 32) {
        const int r = idx / CPR, cch = idx % CPR;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(myq + (uint32_t)(r * (HD * 2) + ((cch ^ (r & 7)) << 4))),
                     "l"(ai.qb + (size_t)r * ai.q_stride + cch * 8) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    uint32_t qf[HD / 16][4];
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncwarp();
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks) {
        const int qr = (lane & 7) + ((lane >> 3) & 1) * 8, qc = 2 * ks + (lane >> 4);
        ldsm_x4(myq + (uint32_t)(qr * (HD * 2) + ((qc ^ (qr & 7)) << 4)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
    }
    __syncwarp();
    float oacc[HD / 8][4];
#pragma unroll
    for (int n = 0; n < HD / 8; ++n) { oacc[n][0] = oacc[n][1] = oacc[n][2] = oacc[n][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // rows g8 and g8 + 8
    int failed = 0;
    auto slot_wait = [&](int n) -> bool {   // one lane polls, the warp follows
        const int sl = n % NST;
        int landed = 1;
        if (lane == 0) landed = mbar_wait(ai.full_a0 + 8u * sl, (pa >> sl) & 1u, limit_ns, abort_flag) ? 1 : 0;
        pa ^= 1u << sl;
        landed = __shfl_sync(0xffffffffu, landed, 0);
        if (!landed) failed = 1 + n;
        return landed != 0;
    };
    for (int b = 0; b < nblk; ++b) {
        const int ks_n = sc0 + 2 * (b >> bps_sh), vs_n = ks_n + 1;
        if ((b & bps_mask) == 0 && !slot_wait(ks_n)) break;
        float s0[4], s1[4];
        {
            const uint32_t kst = slots + (uint32_t)(ks_n % NST) * SLOT_BYTES;
            const int r = (b & bps_mask) * 16 + (lane >> 4) * 8 + (lane & 7);   // key row within the slot; r & 7 == lane & 7
            const int ch = (lane >> 3) & 1;
            auto kaddr = [&](int ks) {   // tile [group][KBk rows][128 B], chunk index XOR (row & 7)
                return kst + (uint32_t)(((g0 + (ks >> 2)) * KBk + r) * 128 + (((((ks & 3) << 1) | ch) ^ (lane & 7)) << 4));
            };
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
        }
        if ((b & bps_mask) == 0 && !slot_wait(vs_n)) break;
        const uint32_t vst = slots + (uint32_t)(vs_n % NST) * SLOT_BYTES;
        const int vr = (b & bps_mask) * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
        auto vaddr = [&](int n) {
            const int col0 = n * 8 + (lane >> 4) * 8;   // first column of this lane's 8x8 matrix within the head
            return vst + (uint32_t)(((g0 + (col0 >> 6)) * KBk + vr) * 128 + ((((col0 & 63) >> 3) ^ (lane & 7)) << 4));
        };
        constexpr int NPRE = 2;
        uint32_t vf[NPRE][4];
#pragma unroll
        for (int i = 0; i < NPRE; ++i) ldsm_x4_t(vaddr(2 * i), vf[i][0], vf[i][1], vf[i][2], vf[i][3]);
        float v[8] = {s0[0], s0[1], s0[2], s0[3], s1[0], s1[1], s1[2], s1[3]};
        if (b == nblk - 1) {
            const int kleft = P - b * 16;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int key = (e >> 2) * 8 + 2 * tq + (e & 1);
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
        if (rescale) { al0 = ex2((m0 - mn0) * sc2); al1 = ex2((m1 - mn1) * sc2); }
        m0 = mn0; m1 = mn1;
        const float ms0 = -mn0 * sc2, ms1 = -mn1 * sc2;
        float p[8];
        p[0] = ex2(fmaf(v[0], sc2, ms0)); p[1] = ex2(fmaf(v[1], sc2, ms0)); p[4] = ex2(fmaf(v[4], sc2, ms0)); p[5] = ex2(fmaf(v[5], sc2, ms0));
        p[2] = ex2(fmaf(v[2], sc2, ms1)); p[3] = ex2(fmaf(v[3], sc2, ms1)); p[6] = ex2(fmaf(v[6], sc2, ms1)); p[7] = ex2(fmaf(v[7], sc2, ms1));
        l0 = l0 * al0 + ((p[0] + p[1]) + (p[4] + p[5]));
        l1 = l1 * al1 + ((p[2] + p[3]) + (p[6] + p[7]));
        uint32_t pf[4];
        pf[0] = pack2(p[0], p[1]); pf[1] = pack2(p[2], p[3]); pf[2] = pack2(p[4], p[5]); pf[3] = pack2(p[6], p[7]);
        if (rescale) {
#pragma unroll
            for (int n = 0; n < HD / 8; ++n) { oacc[n][0] *= al0; oacc[n][1] *= al0; oacc[n][2] *= al1; oacc[n][3] *= al1; }
        }
#pragma unroll
        for (int i = 0; i < NPRE; ++i) {
            mma_bf16(oacc[2 * i], pf, vf[i][0], vf[i][1]);
            mma_bf16(oacc[2 * i + 1], pf, vf[i][2], vf[i][3]);
        }
#pragma unroll
        for (int n = 2 * NPRE; n < HD / 8; n += 2) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4_t(vaddr(n), b0, b1, b2, b3);
            mma_bf16(oacc[n], pf, b0, b1);
            mma_bf16(oacc[n + 1], pf, b2, b3);
        }
        if ((b & bps_mask) == bps_mask || b == nblk - 1) {   // last block of its slots: hand both back
            __syncwarp();
            if (lane == 0) { mbar_arrive(ai.empty_a0 + 8u * (ks_n % NST)); mbar_arrive(ai.empty_a0 + 8u * (vs_n % NST)); }
        }
    }
    ai.pa = pa;
    if (failed) return failed;
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float i0 = 1.0f / l0, i1 = 1.0f / l1;
    __nv_bfloat16 *ob = ai.ob + 8 * tq;
#pragma unroll
    for (int j = 0; j < HD / 32; ++j) {
        uint32_t r0[4], r1[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            r0[k] = pack2(oacc[4 * j + k][0] * i0, oacc[4 * j + k][1] * i0);
            r1[k] = pack2(oacc[4 * j + k][2] * i1, oacc[4 * j + k][3] * i1);
        }
        quad_transpose(r0, tq);
        quad_transpose(r1, tq);
        if (g8 < H) *reinterpret_cast<uint4 *>(ob + (size_t)g8 * ai.o_stride + j * 32) = make_uint4(r0[0], r0[1], r0[2], r0[3]);
        if (g8 + 8 < H) *reinterpret_cast<uint4 *>(ob + (size_t)(g8 + 8) * ai.o_stride + j * 32) = make_uint4(r1[0], r1[1], r1[2], r1[3]);
    }
    return 0;
}

// The epilogue of one 32-row x 128-column part of a tile, out of line for the same reason.
template <int EPI>
__device__ __noinline__ bool epilogue_part(const GemmArgs &g, const CUtensorMap *tmC, uint32_t tacc, int row0, int n0, float *stg,
                                           uint32_t tfull_bar, uint32_t parity, unsigned long long limit_ns, volatile int *abort_flag)
{
    auto acc_ready = [&] { return __all_sync(0xffffffffu, mbar_wait_relaxed(tfull_bar, parity, limit_ns, abort_flag)) != 0; };
    if constexpr (EPI == EPI_RESID) return epilogue_rows<EPI_RESID, 128, true>(g, tacc, row0, n0, stg, acc_ready);
    else return epilogue_store_tma<EPI, 128, true>(g, tmC, tacc, row0, n0, stg, acc_ready);
}

// The embedding / the head of 16 rows of a 128-row block (one worker warp's share), out of line likewise.
template <int AMAX>
__device__ __noinline__ void embed_part(const EmbedArgs &ea, int A, int row_first, int M, int lane)
{
    const __nv_bfloat16 *w_in = (const __nv_bfloat16 *)ea.w_in;
    for (int p = 0; p < 8; ++p) {
        const int row0 = row_first + p * 2;
        if (row0 < M)
            embed_row_pair<__nv_bfloat16, AMAX, true>(ea, row0, min(2, M - row0), lane, [&](int j, int c) {
                return make_float4(ldf(w_in + (size_t)c * A + j), ldf(w_in + (size_t)(c + 1) * A + j),
                                   ldf(w_in + (size_t)(c + 2) * A + j), ldf(w_in + (size_t)(c + 3) * A + j));
            });
    }
}
template <int AMAX>
__device__ __noinline__ void head_part(const HeadArgs &ha, int row_first, int M, int lane)
{
    const __nv_bfloat16 *w_out = (const __nv_bfloat16 *)ha.w_out;
    const int d = ha.d;
    for (int p = 0; p < 8; ++p) {
        const int row0 = row_first + p * 2;
        if (row0 < M)
            head_row_pair<__nv_bfloat16, AMAX, true>(ha, row0, min(2, M - row0), lane, [&](int j, int c) {
                const uint2 w = *reinterpret_cast<const uint2 *>(w_out + (size_t)j * d + c);
                const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162 *>(&w.x);
                const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162 *>(&w.y);
                return make_float4(__bfloat162float(lo.x), __bfloat162float(lo.y), __bfloat162float(hi.x), __bfloat162float(hi.y));
            });
    }
}

template <int HD, int AMAX>
__global__ void __launch_bounds__(THREADS, 1)
fused_steps_kernel(const __grid_constant__ FusedArgs f, unsigned long long limit_ns, int *status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t slots = smem_u32(smem);
    uint8_t *stg_base = smem + NST * SLOT_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(stg_base + WORKERS * STG_BYTES);
    const uint32_t bar0 = smem_u32(bars);
    // A slot serves projections (k-blocks, consumed by the MMA thread) and attention (key blocks, consumed by the
    // head warps) in turn.  Each kind has its own pair of barriers per slot, so that every waiter sees EVERY phase of
    // the barriers it waits on, in order: a waiter that skipped the other kind's uses of a shared barrier could fall
    // two phases behind, and a parity wait cannot tell phase k from phase k + 2.
    auto full_g = [&](int s) { return bar0 + 8u * s; };                 // projection k-block landed
    auto full_a = [&](int s) { return bar0 + 8u * (NST + s); };         // attention key block landed
    auto empty_g = [&](int s) { return bar0 + 8u * (2 * NST + s); };    // slot freed by the MMA thread
    auto empty_a = [&](int s) { return bar0 + 8u * (3 * NST + s); };    // slot freed by the attention consumers
    auto tfull = [&](int b) { return bar0 + 8u * (4 * NST + b); };
    auto tempty = [&](int b) { return bar0 + 8u * (4 * NST + 2 + b); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars + 4 * NST + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 4 * NST + 5);
    // Tasks of this CTA (in order, all kinds) whose dependency has been seen satisfied.  ONE thread per CTA -- the
    // producer -- polls the global counters; everybody else watches this word in shared memory.  (Acquiring loads and
    // fences drop the SM's L1, where the other warps keep their stack and spilled registers: nine pollers per CTA
    // made every inner loop of the kernel several times slower.)
    volatile int *dep_ready = reinterpret_cast<volatile int *>(bars + 4 * NST + 6);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    const int H = f.H, d = f.d, hpc = f.hpc, nslab = f.n_heads / hpc, EPB = BM / H;
    const int W = hpc * HD, NG = W / 64, KBk = slot_keys(W);
    const uint32_t box_bytes = (uint32_t)(NG * KBk * 128);

    if (threadIdx.x == 0) {
        for (int s = 0; s < NST; ++s) { mbar_init(full_g(s), 1); mbar_init(full_a(s), 1); mbar_init(empty_g(s), 1); mbar_init(empty_a(s), hpc); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull(b), 1); mbar_init(tempty(b), 4); }
        *abort_flag = 0;
        *dep_ready = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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

    auto first_task = [&](const OpDesc &o) { const int r = o.base % G; return cta >= r ? cta - r : cta - r + G; };
    // progress note per role (read by the host after a time-out): the global number of the task in hand
    auto note_task = [&](int role, const OpDesc &o, int t) { if (f.trace) f.trace[cta * 4 + role] = ((o.base + t) << 4) | (o.kind << 2) | (o.self & 1); };
    auto dep_counter = [&](const OpDesc &o, int m) { return f.done + (size_t)o.dep_step * f.mt_max + m; };
    auto dep_target = [&](const OpDesc &o, int m) { return o.dep_fixed + o.dep_attn * f.n_heads * envs_in_block(o.dep_ne, m, EPB); };

    if (warp == 0) {
        // ================= TMA producer and dependency watcher: one thread =================
        if (lane == 0) {
            int sc = 0;                                   // slots handed out so far (ring position = sc mod NST)
            int published = 0;                            // tasks of this CTA whose dependency has been announced
            uint32_t used = 0, kindm = 0, parg = 0, para = 0;   // per slot: ever used, last use was attention, next parity to wait for
            auto take_slot = [&](int sl, bool attn) -> bool {
                const uint32_t bit = 1u << sl;
                bool r = true;
                if (used & bit) {
                    if (kindm & bit) { r = mbar_wait_relaxed(empty_a(sl), (para >> sl) & 1u, limit_ns, abort_flag); para ^= bit; }
                    else { r = mbar_wait_relaxed(empty_g(sl), (parg >> sl) & 1u, limit_ns, abort_flag); parg ^= bit; }
                }
                used |= bit;
                kindm = attn ? (kindm | bit) : (kindm & ~bit);
                return r;
            };
            // waits until row block m holds everything the task reads, then tells the other roles
            auto dep_then_publish = [&](const OpDesc &o, int t, int m) -> bool {
                if (o.dep_step >= 0 && !wait_counter(dep_counter(o, m), dep_target(o, m), limit_ns, abort_flag, status)) {
                    note_failure(status, 2, o.kind, o.s, t, (ld_relaxed(dep_counter(o, m)) << 16) | dep_target(o, m));
                    return false;
                }
                PROF_EVT(1, o, t, m)
                fence_proxy_async_global();
                *dep_ready = ++published;
                return true;
            };
            ok = walk_ops(f, [&](const OpDesc &o) -> bool {
                if ((f.test_drop_copies == 1 && o.kind == OP_GEMM) || (f.test_drop_copies == 2 && o.kind == OP_ATTN))
                    return false;     // tests of the give-up path: the producer walks off, the other roles' waits run out
                if (o.kind == OP_GEMM) {
                    const int nt = o.N / BN, nkb = o.K / BK, pf = nkb < NST ? nkb : NST;
                    for (int t = first_task(o); t < o.ntasks; t += G) {
                        const int m = t / nt, n = t - m * nt;
                        note_task(0, o, t);
                        // the weight halves of the first stages do not depend on anything: request them before the wait
                        for (int i = 0; i < pf; ++i) {
                            const int sl = (sc + i) % NST;
                            if (!take_slot(sl, false)) { note_failure(status, 1, o.kind, o.s, t, sl); return false; }
                            mbar_expect_tx(full_g(sl), 2 * A_BYTES);
                            tma_load_2d(slots + sl * SLOT_BYTES + A_BYTES, o.tmW, full_g(sl), i * BK, n * BN);
                        }
                        if (!dep_then_publish(o, t, m)) return false;
                        for (int i = 0; i < pf; ++i) {
                            const int sl = (sc + i) % NST;
                            tma_load_2d(slots + sl * SLOT_BYTES, o.tmA, full_g(sl), i * BK, m * BM);
                        }
                        for (int kb = pf; kb < nkb; ++kb) {
                            const int sl = (sc + kb) % NST;
                            if (!take_slot(sl, false)) { note_failure(status, 3, o.kind, o.s, t, sl); return false; }
                            mbar_expect_tx(full_g(sl), 2 * A_BYTES);
                            tma_load_2d(slots + sl * SLOT_BYTES, o.tmA, full_g(sl), kb * BK, m * BM);
                            tma_load_2d(slots + sl * SLOT_BYTES + A_BYTES, o.tmW, full_g(sl), kb * BK, n * BN);
                        }
                        sc += nkb;
                    }
                } else if (o.kind == OP_ATTN) {
                    for (int t = first_task(o); t < o.ntasks; t += G) {
                        const int env = t / nslab, slab = t - env * nslab, m = env / EPB;
                        note_task(0, o, t);
                        const void *tm;
                        int P, krow, vrow, kgrp, vgrp;
                        if (o.self) {
                            // keys and values are this step's QKV rows: nothing can be requested before they exist
                            if (!dep_then_publish(o, t, m)) return false;
                            tm = f.attn_maps; P = H;
                            krow = vrow = env * H;
                            kgrp = (d + slab * W) / 64; vgrp = (2 * d + slab * W) / 64;
                        } else {
                            tm = f.attn_maps + 1 + env; P = f.meta[env].P;
                            const int pr = f.plane_rows ? f.plane_rows : P;
                            krow = (f.kv_layers == 1 ? 0 : o.layer) * 2 * pr; vrow = krow + pr;
                            kgrp = vgrp = slab * NG;
                            // descriptors are rewritten by the host between batches: drop any stale cached copy
                            asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(reinterpret_cast<uint64_t>(tm)) : "memory");
                        }
                        // cross-attention: the planes are inputs, so the first key blocks are requested ahead of the
                        // queries; the dependency is announced once as many blocks are on their way as the ring can
                        // hold beside the consumers (waiting for a free slot any earlier could wait for the very
                        // consumers that wait for the announcement)
                        const int nst = (P + KBk - 1) / KBk, announce_after = (nst < 3 ? nst : 3) - 1;
                        for (int j = 0; j < nst; ++j) {
                            int sl = sc % NST;
                            if (!take_slot(sl, true)) { note_failure(status, 5, o.kind, o.s, t, sl); return false; }
                            mbar_expect_tx(full_a(sl), box_bytes);
                            tma_load_3d(slots + sl * SLOT_BYTES, tm, full_a(sl), 0, krow + j * KBk, kgrp);
                            ++sc;
                            sl = sc % NST;
                            if (!take_slot(sl, true)) { note_failure(status, 6, o.kind, o.s, t, sl); return false; }
                            mbar_expect_tx(full_a(sl), box_bytes);
                            tma_load_3d(slots + sl * SLOT_BYTES, tm, full_a(sl), 0, vrow + j * KBk, vgrp);
                            ++sc;
                            if (!o.self && j == announce_after && !dep_then_publish(o, t, m)) return false;
                        }
                    }
                } else {
                    // embedding / head: nothing to copy, only the dependency to watch
                    for (int m = first_task(o); m < o.ntasks; m += G) {
                        note_task(0, o, m);
                        if (!dep_then_publish(o, m, m)) return false;
                    }
                }
                return true;
            });
        }
        __syncwarp();
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    } else if (warp == 1) {
        // ================= MMA issuer: one thread =================
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(BM, BN);
            int sc = 0, it = 0;
            uint32_t pg = 0;      // per slot: parity of the next projection k-block to wait for
            ok = walk_ops(f, [&](const OpDesc &o) -> bool {
                if (o.kind == OP_GEMM) {
                    const int nkb = o.K / BK;
                    for (int t = first_task(o); t < o.ntasks; t += G, ++it) {
                        const int buf = it & 1;
                        note_task(1, o, t);
                        if (!mbar_wait_relaxed(tempty(buf), (((uint32_t)(it >> 1)) & 1u) ^ 1u, limit_ns, abort_flag)) {
                            note_failure(status, 7, o.kind, o.s, t, it);
                            return false;
                        }
                        tc_fence_after();
                        const uint32_t d_tmem = tmem_base + (uint32_t)buf * BN;
                        for (int kb = 0; kb < nkb; ++kb, ++sc) {
                            const int sl = sc % NST;
                            // the first k-block of a task may be far away (its dependency): wait for it without
                            // taking issue slots from the workers that share this scheduler
                            const bool landed = kb == 0 ? mbar_wait_relaxed(full_g(sl), (pg >> sl) & 1u, limit_ns, abort_flag)
                                                        : mbar_wait(full_g(sl), (pg >> sl) & 1u, limit_ns, abort_flag);
                            if (!landed) { note_failure(status, 8, o.kind, o.s, t, (kb << 8) | sl); return false; }
                            if (kb == 0) { PROF_EVT(3, o, t, t / (o.N / BN)) }
                            pg ^= 1u << sl;
                            tc_fence_after();
                            const uint64_t ad = smem_desc(slots + sl * SLOT_BYTES), bd = smem_desc(slots + sl * SLOT_BYTES + A_BYTES);
                            tc_mma(d_tmem, ad, bd, idesc, kb != 0 ? 1u : 0u);
#pragma unroll
                            for (int k = 1; k < BK / UMMA_K; ++k)
                                tc_mma(d_tmem, ad + (uint64_t)(k * UMMA_K * 2 / 16), bd + (uint64_t)(k * UMMA_K * 2 / 16), idesc, 1u);
                            tc_commit(empty_g(sl));
                        }
                        tc_commit(tfull(buf));
                        PROF_EVT(4, o, t, t / (o.N / BN))
                    }
                } else if (o.kind == OP_ATTN) {
                    for (int t = first_task(o); t < o.ntasks; t += G) {
                        const int P = o.self ? H : f.meta[t / nslab].P;
                        sc += 2 * ((P + KBk - 1) / KBk);
                    }
                }
                return true;
            });
        }
        __syncwarp();
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    } else {
        // ================= workers: epilogue groups / attention consumers / row workers =================
        const int wi = warp - 2, grp = wi >> 2, q = warp & 3;
        float *stg = reinterpret_cast<float *>(stg_base + wi * STG_BYTES);
        const uint32_t myq = smem_u32(stg);
        int sc = 0, it = 0;
        int seen = 0;             // tasks of this CTA passed so far, of every kind (the producer announces them in this order)
        uint32_t pa = 0;          // per slot: parity of the next attention key block to wait for
        // waits until the producer has announced the dependency of this CTA's task number `seen`
        auto wait_dep = [&](const OpDesc &o, int t) -> bool {
            int r = 1;
            if (lane == 0 && *dep_ready <= seen) {
                const unsigned long long t0 = gtimer();
                for (;;) {
                    bool got = false;
                    for (int i = 0; i < 64 && !got; ++i) { got = *dep_ready > seen; if (!got) __nanosleep(40); }
                    if (got) break;
                    if (*abort_flag || gtimer() - t0 > limit_ns) { r = 0; note_failure(status, 9, o.kind, o.s, t, seen); break; }
                }
            }
            r = __shfl_sync(0xffffffffu, r, 0);
            __syncwarp();
            return r != 0;
        };
        const int bps_sh = KBk == 16 ? 0 : (KBk == 32 ? 1 : 2), bps_mask = (1 << bps_sh) - 1;   // 16-key blocks per slot
        ok = walk_ops(f, [&](const OpDesc &o) -> bool {
            int *done_s = f.done + (size_t)o.s * f.mt_max;
            if (o.kind == OP_EMBED) {
                EmbedArgs ea{f.meta, o.ne, H, f.A, d, o.s, f.a_state, f.w_in, f.temb, f.n_layers > 0 ? f.layers[0].g1 : f.g_final,
                             f.x, f.xg, f.ssq};
                for (int m = first_task(o); m < o.ntasks; m += G, ++seen) {
                    if (!wait_dep(o, m)) return false;
                    embed_part<AMAX>(ea, f.A, m * BM + wi * 16, o.M, lane);
                    signal_block(done_s + m, lane);
                }
            } else if (o.kind == OP_HEAD) {
                HeadArgs ha{f.meta, o.ne, H, f.A, d, o.s, f.K, f.a_state, f.x, f.g_final, f.w_out, f.b_out, f.eps, 0};
                for (int m = first_task(o); m < o.ntasks; m += G, ++seen) {
                    if (!wait_dep(o, m)) return false;
                    head_part<AMAX>(ha, m * BM + wi * 16, o.M, lane);
                    signal_block(done_s + m, lane);
                }
            } else if (o.kind == OP_GEMM) {
                const int nt = o.N / BN, nkb = o.K / BK;
                GemmArgs g{};
                g.M = o.M; g.N = o.N; g.K = o.K; g.epi = o.epi;
                g.ssq_in = f.ssq; g.n_ssq = d / SSQ_W; g.inv_d = f.inv_d; g.eps = f.eps;
                g.C = o.C; g.x = f.x; g.gain = o.gain; g.xg = f.xg; g.ssq_out = f.ssq;
                for (int t = first_task(o); t < o.ntasks; t += G, ++it, sc += nkb, ++seen) {
                    const int buf = it & 1;
                    if (grp != buf) continue;
                    const int m = t / nt, n = t - m * nt;
                    if (q == 0 && lane == 0) note_task(2 + grp, o, t);
                    if (!wait_dep(o, t)) return false;     // the residual rows / row scales this epilogue reads
                    if (q == 0 && lane == 0) { PROF_EVT(5, o, t, m) }
                    const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                    const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN);
                    const int row0 = m * BM + q * 32, n0 = n * BN;
                    bool done;
                    if (o.epi == EPI_RESID) done = epilogue_part<EPI_RESID>(g, o.tmC, tacc, row0, n0, stg, tfull(buf), acc_phase, limit_ns, abort_flag);
                    else if (o.epi == EPI_SCALE_GELU) done = epilogue_part<EPI_SCALE_GELU>(g, o.tmC, tacc, row0, n0, stg, tfull(buf), acc_phase, limit_ns, abort_flag);
                    else done = epilogue_part<EPI_SCALE_STORE>(g, o.tmC, tacc, row0, n0, stg, tfull(buf), acc_phase, limit_ns, abort_flag);
                    if (q == 0 && lane == 0) { PROF_EVT(6, o, t, m) }
                    if (!done) { if (lane == 0) note_failure(status, 10, o.kind, o.s, t, it); return false; }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(tempty(buf));
                        if (o.epi != EPI_RESID) epilogue_store_drain();    // the tile's stores have been written
                    }
                    signal_block(done_s + m, lane);
                    if (q == 0 && lane == 0) { PROF_EVT(7, o, t, m) }
                }
            } else {
                // ---- attention: worker = head within the slab (the per-operation kernel's consumer, on ring slots)
                for (int t = first_task(o); t < o.ntasks; t += G, ++seen) {
                    const int env = t / nslab, slab = t - env * nslab, m = env / EPB;
                    const int P = o.self ? H : f.meta[env].P;
                    const int nblk = (P + 15) >> 4, nslots = (nblk + bps_mask) >> bps_sh;
                    const int sc0 = sc;
                    sc += 2 * nslots;
                    if (wi >= hpc) continue;
                    if (wi == 0 && lane == 0) note_task(2, o, t);
                    if (!wait_dep(o, t)) return false;
                    const int head = slab * hpc + wi;
                    if (wi == 0 && lane == 0) { PROF_EVT(8, o, t, m) }
                    AttnItem ai;
                    ai.q_stride = o.self ? 3 * d : d;
                    ai.qb = (o.self ? (const __nv_bfloat16 *)f.qkv : (const __nv_bfloat16 *)f.qc) + (size_t)env * H * ai.q_stride + head * HD;
                    ai.ob = (__nv_bfloat16 *)f.att + (size_t)env * H * d + head * HD;
                    ai.o_stride = d; ai.H = H; ai.P = P; ai.KBk = KBk; ai.g0 = wi * (HD / 64); ai.sc0 = sc0;
                    ai.slots = slots; ai.full_a0 = full_a(0); ai.empty_a0 = empty_a(0); ai.myq = myq; ai.pa = pa;
                    ai.limit_ns = limit_ns; ai.abort_flag = abort_flag;
                    const int bad = attn_item<HD>(ai, lane);
                    pa = ai.pa;
                    if (bad) { if (lane == 0) note_failure(status, 11, o.kind, o.s, t, bad); return false; }
                    if (wi == 0 && lane == 0) { PROF_EVT(9, o, t, m) }
                    signal_block(done_s + m, lane);
                    if (wi == 0 && lane == 0) { PROF_EVT(10, o, t, m) }
                }
            }
            return true;
        });
        ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
    }

    // ---- teardown
    if (!ok) {
        *abort_flag = 1;
        if (lane == 0) atomicCAS(status, 0, 7 /* EBRL_ERR_TIMEOUT */);
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

}  // namespace fs

// Shapes the persistent kernel covers (beyond what the tensor-core GEMM and attention kernels need):
// H a divisor of 128 (environments never straddle a row block), A <= 16.
bool fused_supported(int H, int A, int d, int md, int n_heads, int hd)
{
    if (H < 1 || H > 16 || 128 % H != 0 || A > 16) return false;
    if (d % 128 || md % 128 || (hd != 64 && hd != 128)) return false;
    const int hpc = n_heads < fs::WORKERS ? n_heads : fs::WORKERS;
    return n_heads % hpc == 0;
}

template <int HD, int AMAX>
static cudaError_t fused_launch(const FusedArgs &f, int grid, unsigned long long limit_ns, int *status, cudaStream_t st)
{
    static bool attr_set[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(fs::fused_steps_kernel<HD, AMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, fs::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(fs::THREADS, 1, 1);
    cfg.dynamicSmemBytes = fs::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;     // all CTAs resident at once: tasks wait for one another
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fs::fused_steps_kernel<HD, AMAX>, f, limit_ns, status);
}

// grid = SM quota (at most one CTA per SM; fewer when no operation has that many tasks).
cudaError_t launch_fused_steps(const FusedArgs &f, int grid, unsigned long long limit_ns, int *status, cudaStream_t st)
{
    if (f.S < 1 || f.ne0 < 1) return cudaSuccess;
    const int mt = (f.ne0 * f.H + fs::BM - 1) / fs::BM;
    const int widest = std::max(mt * (std::max(f.md, 3 * f.d) / fs::BN), f.ne0 * (f.n_heads / f.hpc));
    const int g = widest < grid ? widest : grid;
    if (f.hd == 128) return f.A <= 8 ? fused_launch<128, 8>(f, g, limit_ns, status, st) : fused_launch<128, 16>(f, g, limit_ns, status, st);
    return f.A <= 8 ? fused_launch<64, 8>(f, g, limit_ns, status, st) : fused_launch<64, 16>(f, g, limit_ns, status, st);
}

}  // namespace ebrl
