// Softmax attention for the bf16 models: the H (<= 16) query tokens of one environment against
// its keys/values -- the cached prefix planes (cross-attention) or its own H rows of the QKV
// buffer (self-attention).  The kernel is bandwidth-shaped: every K/V element is used by only H
// queries, so the planes are streamed once through shared memory by 1-D bulk copies (one per
// key row, so that rows can be padded against bank conflicts) into a 3-stage ring, and the
// small contractions run on mma.sync (m16n8k16, bf16 in, fp32 accumulate) with the softmax
// statistics kept per row by quad shuffles.
//
// Work item = (environment, slab of up to 8 heads); one warp per head; a ninth warp issues the
// copies.  Keys are visited in blocks of 16 in index order with a running maximum and sum, so
// an environment's result does not depend on the grid size or on what else is in the batch.
// Every wait is bounded (status word, as in the GEMM).
#include "actgen_internal.h"
#include "ptx_helpers.cuh"

namespace ebrl {
namespace am {

using namespace ptx;

constexpr int NSTAGE = 3;
constexpr int MAXW = 8;                 // consumer warps = heads per slab
constexpr int THREADS = (MAXW + 1) * 32;
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
__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Keys per stage for a slab of W columns: a whole number of 16-key blocks within the stage budget.
__host__ __device__ inline int stage_keys(int W) { int k = STAGE_ROWS_BYTES / (W * 2); k &= ~15; return k < 16 ? 16 : (k > 64 ? 64 : k); }

template <int HD>
__global__ void __launch_bounds__(THREADS, 1) attn_mma_kernel(AttnArgs a, int hpc, unsigned long long limit_ns, int *status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const int W = hpc * HD;                       // slab width in columns
    const int pitch = W * 2 + 16;                 // bytes per staged key row (padded: conflict-free ldmatrix)
    const int KB = stage_keys(W);
    const int stage_bytes = KB * pitch;
    const uint32_t sK = smem_u32(smem), sV = sK + NSTAGE * stage_bytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + 2 * NSTAGE * stage_bytes);
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (NSTAGE + s); };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * NSTAGE);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int H = a.H, nslab = a.n_heads / hpc, items = a.n_envs * nslab;

    // zero the ring once: rows past a prefix's end are never copied, and 0 * stale bits must be 0
    for (int i = threadIdx.x; i < 2 * NSTAGE * stage_bytes / 16; i += blockDim.x)
        reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), hpc); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_proxy_async();
    __syncthreads();

    bool ok = true;
    int stage = 0;
    uint32_t phase = 0;

    if (warp == MAXW) {
        // ---- producer: one bulk copy per key row of K and of V
        for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
            const int env = item / nslab, slab = item - env * nslab;
            const __nv_bfloat16 *kbase, *vbase;
            int P, stride;
            if (a.self) {
                kbase = (const __nv_bfloat16 *)a.k_self + (size_t)env * H * a.kv_stride + slab * W;
                vbase = (const __nv_bfloat16 *)a.v_self + (size_t)env * H * a.kv_stride + slab * W;
                P = H; stride = a.kv_stride;
            } else {
                const EnvMeta m = a.meta[env];
                P = m.P; stride = a.d;
                kbase = (const __nv_bfloat16 *)m.kv + (size_t)a.kv_plane * 2 * P * a.d + slab * W;
                vbase = kbase + (size_t)P * a.d;
            }
            for (int j0 = 0; j0 < P; j0 += KB) {
                const int nrows = min(KB, P - j0);
                if (!__all_sync(0xffffffffu, mbar_wait(empty(stage), phase ^ 1u, limit_ns, abort_flag))) { ok = false; break; }
                if (lane == 0) mbar_expect_tx(full(stage), (uint32_t)(2 * nrows * W * 2));
                __syncwarp();
                for (int r = lane; r < 2 * nrows; r += 32) {
                    const int isv = r >= nrows, j = isv ? r - nrows : r;
                    const __nv_bfloat16 *src = (isv ? vbase : kbase) + (size_t)(j0 + j) * stride;
                    bulk_load((isv ? sV : sK) + stage * stage_bytes + j * pitch, src, (uint32_t)(W * 2), full(stage));
                }
                __syncwarp();
                if (++stage == NSTAGE) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp < hpc) {
        // ---- consumers: warp = head within the slab
        const int g = lane >> 2, t = lane & 3;
        const float sc = 1.4426950408889634f / sqrtf((float)HD);   // log2(e) / sqrt(hd): scores in base-2 units
        for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
            const int env = item / nslab, slab = item - env * nslab;
            const int P = a.self ? H : a.meta[env].P;
            const int head = slab * hpc + warp;
            // Q fragments (A operand, 16 x HD), rows >= H are zero
            uint32_t qf[HD / 16][4];
            {
                const __nv_bfloat16 *qb = (const __nv_bfloat16 *)a.q + (size_t)env * H * a.q_stride + head * HD;
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    const int c = ks * 16 + 2 * t;
                    qf[ks][0] = g < H ? *reinterpret_cast<const uint32_t *>(qb + (size_t)g * a.q_stride + c) : 0u;
                    qf[ks][1] = g + 8 < H ? *reinterpret_cast<const uint32_t *>(qb + (size_t)(g + 8) * a.q_stride + c) : 0u;
                    qf[ks][2] = g < H ? *reinterpret_cast<const uint32_t *>(qb + (size_t)g * a.q_stride + c + 8) : 0u;
                    qf[ks][3] = g + 8 < H ? *reinterpret_cast<const uint32_t *>(qb + (size_t)(g + 8) * a.q_stride + c + 8) : 0u;
                }
            }
            float o[HD / 8][4];
#pragma unroll
            for (int n = 0; n < HD / 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
            float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // rows g and g + 8
            const uint32_t kcol = (uint32_t)(warp * HD * 2);
            for (int j0 = 0; j0 < P; j0 += KB) {
                if (!__all_sync(0xffffffffu, mbar_wait(full(stage), phase, limit_ns, abort_flag))) { ok = false; break; }
                const int nrows = min(KB, P - j0);
                const uint32_t kst = sK + stage * stage_bytes + kcol, vst = sV + stage * stage_bytes + kcol;
                for (int jb = 0; jb < nrows; jb += 16) {
                    // S = Q K^T for 16 keys: two n-tiles of 8 keys
                    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
                    {
                        const uint32_t addr = kst + (uint32_t)((jb + (lane >> 4) * 8 + (lane & 7)) * pitch + ((lane >> 3) & 1) * 16);
#pragma unroll
                        for (int ks = 0; ks < HD / 16; ++ks) {
                            uint32_t b0, b1, b2, b3;
                            ldsm_x4(addr + ks * 32, b0, b1, b2, b3);
                            mma_bf16(s0, qf[ks], b0, b1);
                            mma_bf16(s1, qf[ks], b2, b3);
                        }
                    }
                    // mask keys past the prefix, running max / sum per row
                    const int kleft = nrows - jb;   // valid keys in this block (may exceed 16)
                    const int c0 = 2 * t, c1 = 2 * t + 1;
                    float v[8] = {s0[0], s0[1], s0[2], s0[3], s1[0], s1[1], s1[2], s1[3]};
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int key = (e >> 2) * 8 + ((e & 1) ? c1 : c0);
                        v[e] = key < kleft ? v[e] * sc : -INFINITY;
                    }
                    float mx0 = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[4], v[5]));
                    float mx1 = fmaxf(fmaxf(v[2], v[3]), fmaxf(v[6], v[7]));
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
                    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
                    const float al0 = exp2f(m0 - mn0), al1 = exp2f(m1 - mn1);
                    m0 = mn0; m1 = mn1;
                    float p[8];
                    p[0] = exp2f(v[0] - mn0); p[1] = exp2f(v[1] - mn0); p[4] = exp2f(v[4] - mn0); p[5] = exp2f(v[5] - mn0);
                    p[2] = exp2f(v[2] - mn1); p[3] = exp2f(v[3] - mn1); p[6] = exp2f(v[6] - mn1); p[7] = exp2f(v[7] - mn1);
                    l0 = l0 * al0 + ((p[0] + p[1]) + (p[4] + p[5]));
                    l1 = l1 * al1 + ((p[2] + p[3]) + (p[6] + p[7]));
                    uint32_t pf[4];
                    pf[0] = pack2(p[0], p[1]); pf[1] = pack2(p[2], p[3]); pf[2] = pack2(p[4], p[5]); pf[3] = pack2(p[6], p[7]);
                    // O = O * alpha + P V
                    const uint32_t vaddr = vst + (uint32_t)((jb + ((lane >> 3) & 1) * 8 + (lane & 7)) * pitch + (lane >> 4) * 16);
#pragma unroll
                    for (int n = 0; n < HD / 8; n += 2) {
                        uint32_t b0, b1, b2, b3;
                        ldsm_x4_t(vaddr + n * 16, b0, b1, b2, b3);
                        o[n][0] *= al0; o[n][1] *= al0; o[n][2] *= al1; o[n][3] *= al1;
                        o[n + 1][0] *= al0; o[n + 1][1] *= al0; o[n + 1][2] *= al1; o[n + 1][3] *= al1;
                        mma_bf16(o[n], pf, b0, b1);
                        mma_bf16(o[n + 1], pf, b2, b3);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty(stage));
                if (++stage == NSTAGE) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            // row sums across the quad, normalise, store
            l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
            const float i0 = 1.0f / l0, i1 = 1.0f / l1;
            __nv_bfloat16 *ob = (__nv_bfloat16 *)a.out + (size_t)env * H * a.o_stride + head * HD + 2 * t;
#pragma unroll
            for (int n = 0; n < HD / 8; ++n) {
                if (g < H) *reinterpret_cast<uint32_t *>(ob + (size_t)g * a.o_stride + n * 8) = pack2(o[n][0] * i0, o[n][1] * i0);
                if (g + 8 < H) *reinterpret_cast<uint32_t *>(ob + (size_t)(g + 8) * a.o_stride + n * 8) = pack2(o[n][2] * i1, o[n][3] * i1);
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

// Shapes the kernel covers: bf16, H <= 16, head_dim 64 or 128, heads a multiple of the slab.
bool attn_mma_supported(int H, int n_heads, int hd)
{
    if (H > 16 || (hd != 64 && hd != 128)) return false;
    const int hpc = n_heads < am::MAXW ? n_heads : am::MAXW;
    return n_heads % hpc == 0;
}

cudaError_t launch_attn_mma(const AttnArgs &a, int grid, unsigned long long limit_ns, int *status, cudaStream_t st)
{
    const int hpc = a.n_heads < am::MAXW ? a.n_heads : am::MAXW;
    const int items = a.n_envs * (a.n_heads / hpc);
    if (items == 0) return cudaSuccess;
    const int g = items < grid ? items : grid;
    const int W = hpc * a.hd;
    const size_t smem = (size_t)2 * am::NSTAGE * am::stage_keys(W) * (W * 2 + 16) + 64 + 128;
    cudaError_t e;
    if (a.hd == 128) {
        e = cudaFuncSetAttribute(am::attn_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        am::attn_mma_kernel<128><<<g, am::THREADS, smem, st>>>(a, hpc, limit_ns, status);
    } else {
        e = cudaFuncSetAttribute(am::attn_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        am::attn_mma_kernel<64><<<g, am::THREADS, smem, st>>>(a, hpc, limit_ns, status);
    }
    return cudaGetLastError();
}

}  // namespace ebrl
