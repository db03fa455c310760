// The fused GEMM epilogue shared by the tensor-core GEMM kernels: one thread owns one output
// row of the tile and walks its accumulator columns 32 at a time out of tensor memory.
#pragma once
#include "actgen_internal.h"
#include "split3.cuh"
#include "f32x2.cuh"

#include <cuda.h>

namespace ebrl {
namespace tc {

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// GELU in its erf form, 0.5 z (1 + erf(z / sqrt 2)), with erf from the five-term rational
// approximation erf(x) = 1 - (a1 t + ... + a5 t^5) exp(-x^2), t = 1 / (1 + p x), x >= 0
// (absolute error below 2e-7 -- four orders of magnitude under the bf16 rounding of the result),
// on the fast reciprocal and exponential units: about a dozen instructions per element, which
// keeps the GELU epilogue of the MLP-up GEMM shorter than its tile's mainloop.
__device__ __forceinline__ float gelu_erf(float z)
{
    // Phi(z) = 0.5 (1 + erf(z / sqrt 2)):  q = 0.5 (a1 t + ... + a5 t^5) exp(-z^2 / 2),  Phi = z >= 0 ? 1 - q : q
    const float az = fabsf(z);
    const float a1 = az * 0.84932180028801904f;           // |z| sqrt(log2(e) / 2): exp(-z^2/2) = 2^(-a1^2)
    float t, e;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(az, 0.23164189f, 1.0f)));   // p / sqrt 2
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-a1 * a1));
    float p = fmaf(0.5307027145f, t, -0.7265760135f);     // the five coefficients, halved
    p = fmaf(p, t, 0.7107068705f);
    p = fmaf(p, t, -0.142248368f);
    p = fmaf(p, t, 0.127414796f);
    const float q = p * t * e;
    return z * (z >= 0.f ? 1.0f - q : q);
}
// gelu_erf of two values at once: the same approximation with the polynomial and the products in packed
// form; only |z|, the reciprocal and the exponential stay scalar.  With q = 1/2 (a1 t + ... + a5 t^5) exp(-z^2/2),
// Phi(z) = 1/2 + sign(z) (1/2 - q), hence z Phi(z) = z / 2 + |z| (1/2 - q).
__device__ __forceinline__ void gelu_erf2(float &z0, float &z1)
{
    const uint64_t z = pk2(z0, z1), az = pk2(fabsf(z0), fabsf(z1));
    float t0, t1, e0, e1, a0, a1, r0, r1;
    upk2(mul2(mul2(z, z), pk2(-0.72134752044448170f, -0.72134752044448170f)), a0, a1);   // -z^2 log2(e) / 2
    upk2(fma2(az, pk2(0.23164189f, 0.23164189f), pk2(1.0f, 1.0f)), r0, r1);              // 1 + p |z|
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t0) : "f"(r0));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t1) : "f"(r1));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(a0));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(a1));
    const uint64_t t = pk2(t0, t1);
    uint64_t p = fma2(pk2(0.5307027145f, 0.5307027145f), t, pk2(-0.7265760135f, -0.7265760135f));
    p = fma2(p, t, pk2(0.7107068705f, 0.7107068705f));
    p = fma2(p, t, pk2(-0.142248368f, -0.142248368f));
    p = fma2(p, t, pk2(0.127414796f, 0.127414796f));
    const uint64_t q = mul2(mul2(p, t), pk2(e0, e1));
    const uint64_t h = fma2(q, pk2(-1.0f, -1.0f), pk2(0.5f, 0.5f));                      // 1/2 - q
    upk2(fma2(az, h, mul2(z, pk2(0.5f, 0.5f))), z0, z1);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}


constexpr int EPI_STAGE_FLOATS = 32 * 32;   // per-warp transpose buffer: 32 rows x 32 fp32 columns, 16-byte chunks swizzled

// Loads of data that another CTA of the SAME kernel may have written (the persistent step kernel):
// COH = true reads through L2 (ld.global.cg), because this SM's L1 may still hold the line from
// an earlier task; kernels whose inputs were complete before launch use plain loads.
template <bool COH> __device__ __forceinline__ float4 ld_f4(const float *p)
{
    if (COH) return __ldcg(reinterpret_cast<const float4 *>(p));
    return *reinterpret_cast<const float4 *>(p);
}
template <bool COH> __device__ __forceinline__ float ld_f1(const float *p)
{
    if (COH) return __ldcg(p);
    return *p;
}

// EPI_SCALE_STORE: C = acc * rowscale;  EPI_SCALE_GELU: C = gelu(acc * rowscale);
// EPI_RESID: x += acc, xg = x * gain, one sum-of-squares partial per 128 columns.
//
// Tensor memory hands each thread one ROW of the accumulator (32 columns at a time).  Global
// memory wants a warp instruction to touch few rows: the L1 handles one 128-byte line per cycle
// per instruction, so 32 threads x 16 bytes of 32 different rows cost 32 cycles.  Each 32 x 32
// chunk is therefore turned through shared memory: thread = row writes its 8 16-byte pieces
// (piece j of row r at position j ^ (r & 7): conflict-free), then lane l reads piece (l & 7) of
// rows 4 i + (l >> 3), i = 0..7, so that one instruction covers 4 rows x 128 contiguous bytes.
//
// `taddr` = tensor-memory address of this warp's lane quarter and of the first of the NCOLS
// accumulator columns this warp handles; n0 = their global column; row0 = global row of lane 0.
// All 32 lanes must call it.  `wait` blocks until the accumulator is complete (false on a
// time-out); the residual values of the first chunk are requested before it and those of each
// later chunk one chunk ahead.
// Four consecutive outputs of a row in the activations' type: bf16 (8 bytes) or fp32 (16 bytes).
template <typename OT> __device__ __forceinline__ void store_out4(OT *p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store_out4<__nv_bfloat16>(__nv_bfloat16 *p, float a, float b, float c, float d)
{
    *reinterpret_cast<uint2 *>(p) = make_uint2(pack_bf16(a, b), pack_bf16(c, d));
}
template <> __device__ __forceinline__ void store_out4<float>(float *p, float a, float b, float c, float d)
{
    *reinterpret_cast<float4 *>(p) = make_float4(a, b, c, d);
}

// SPLIT (fp32 models on the tensor cores): what feeds the next projection -- xg of the residual epilogue, C of the
// GELU epilogue -- is written as three bf16 term planes; the scale/store epilogue's C (queries, keys, values) stays fp32.
template <int EPI, int NCOLS, bool COH = false, typename OT = __nv_bfloat16, bool SPLIT = false, typename WaitF>
__device__ __forceinline__ bool epilogue_rows(const GemmArgs &g, uint32_t taddr, int row0, int n0, float *stg_generic, WaitF wait)
{
    constexpr int NC = NCOLS / 32;
    static_assert(NCOLS == SSQ_W, "one sum-of-squares segment per call");
    const int lane = threadIdx.x & 31;
    const uint32_t stg = (uint32_t)__cvta_generic_to_shared(stg_generic);
    const int nrows = g.M - row0;                   // rows of this warp that exist (may be <= 0 or > 32)
    const int sub = lane >> 3, piece = lane & 7;    // transposed domain: row 4 i + sub, columns 4 piece .. 4 piece + 3
    float *__restrict__ xg_x = g.x;
    float rs = 0.f;
    float4 xv[8];
    if (EPI == EPI_RESID) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (4 * i + sub < nrows) xv[i] = ld_f4<COH>(xg_x + (size_t)(row0 + 4 * i + sub) * g.N + n0 + 4 * piece);
    } else if (lane < nrows) {
        float s = 0.f;
        const int row = row0 + lane;
        for (int t = 0; t < g.n_ssq; ++t) s += ld_f1<COH>(g.ssq_in + (size_t)row * g.n_ssq + t);
        rs = 1.0f / sqrtf(s * g.inv_d + g.eps);
    }
    if (!wait()) return false;
    tc_fence_after();
    float ssp[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) ssp[i] = 0.f;
#pragma unroll 1
    for (int c = 0; c < NC; ++c) {
        uint32_t r[32];
        tc_ld32(taddr + (uint32_t)c * 32, r);
        tc_wait_ld();
        const int col = n0 + c * 32;
        // thread = row: 8 pieces of 16 bytes, swizzled
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float v[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                v[e] = __uint_as_float(r[4 * j + e]);
                if (EPI != EPI_RESID) {
                    v[e] *= rs;
                    if (EPI == EPI_SCALE_GELU) v[e] = gelu_erf(v[e]);
                }
            }
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stg + (uint32_t)(lane * 128 + ((j ^ (lane & 7)) << 4))),
                         "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]) : "memory");
        }
        __syncwarp();
        float4 acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int rr = 4 * i + sub;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(acc[i].x), "=f"(acc[i].y), "=f"(acc[i].z), "=f"(acc[i].w)
                         : "r"(stg + (uint32_t)(rr * 128 + ((piece ^ (rr & 7)) << 4))) : "memory");
        }
        __syncwarp();
        if (EPI == EPI_RESID) {
            const float4 gn = *reinterpret_cast<const float4 *>(g.gain + col + 4 * piece);
            OT *__restrict__ xg = (OT *)g.xg;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int rr = 4 * i + sub;
                if (rr < nrows) {
                    const size_t off = (size_t)(row0 + rr) * g.N + col + 4 * piece;
                    float4 xn;
                    xn.x = xv[i].x + acc[i].x; xn.y = xv[i].y + acc[i].y; xn.z = xv[i].z + acc[i].z; xn.w = xv[i].w + acc[i].w;
                    *reinterpret_cast<float4 *>(xg_x + off) = xn;
                    if (SPLIT) store_split4(g.xg, g.out_t1, g.out_t2, off, xn.x * gn.x, xn.y * gn.y, xn.z * gn.z, xn.w * gn.w);
                    else store_out4<OT>(xg + off, xn.x * gn.x, xn.y * gn.y, xn.z * gn.z, xn.w * gn.w);
                    ssp[i] = fmaf(xn.x, xn.x, ssp[i]); ssp[i] = fmaf(xn.y, xn.y, ssp[i]);
                    ssp[i] = fmaf(xn.z, xn.z, ssp[i]); ssp[i] = fmaf(xn.w, xn.w, ssp[i]);
                }
            }
            if (c + 1 < NC) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (4 * i + sub < nrows) xv[i] = ld_f4<COH>(xg_x + (size_t)(row0 + 4 * i + sub) * g.N + col + 32 + 4 * piece);
            }
        } else {
            OT *__restrict__ cp = (OT *)g.C;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int rr = 4 * i + sub;
                if (rr < nrows) {
                    const size_t off = (size_t)(row0 + rr) * g.N + col + 4 * piece;
                    if (SPLIT && EPI == EPI_SCALE_GELU) store_split4(g.C, g.out_t1, g.out_t2, off, acc[i].x, acc[i].y, acc[i].z, acc[i].w);
                    else store_out4<OT>(cp + off, acc[i].x, acc[i].y, acc[i].z, acc[i].w);
                }
            }
        }
    }
    if (EPI == EPI_RESID) {
        // a row's sum of squares over the segment: its 8 lanes' partial sums, added across the lanes
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float t = ssp[i];
            t += __shfl_xor_sync(0xffffffffu, t, 1);
            t += __shfl_xor_sync(0xffffffffu, t, 2);
            t += __shfl_xor_sync(0xffffffffu, t, 4);
            const int rr = 4 * i + sub;
            if (piece == 0 && rr < nrows) g.ssq_out[(size_t)(row0 + rr) * (g.N / SSQ_W) + n0 / SSQ_W] = t;
        }
    }
    return true;
}

// EPI_SCALE_STORE / EPI_SCALE_GELU through the copy engine: the thread that owns a row writes its bf16 values
// as 16-byte pieces into a [32 rows][128 B] staging tile in the 128-byte-swizzle layout (piece p of row r at
// p ^ (r & 7): conflict-free), and one lane hands the tile to a TMA store, which also clips rows past M.
// Per 64 columns that is 8 shared stores per thread and one copy instruction per warp, instead of 16 shared
// stores, 16 shared loads and 16 predicated global stores -- fewer issue slots taken from the single TMA and
// MMA threads that share the schedulers.  `stg_generic` must be 1024-byte aligned (4 KB).
template <int EPI, int NCOLS, bool COH = false, typename WaitF>
__device__ __forceinline__ bool epilogue_store_tma(const GemmArgs &g, const CUtensorMap *tmC, uint32_t taddr, int row0, int n0,
                                                   float *stg_generic, WaitF wait)
{
    static_assert(EPI != EPI_RESID && NCOLS % 64 == 0, "bf16 store epilogues only");
    const int lane = threadIdx.x & 31;
    const uint32_t stg = (uint32_t)__cvta_generic_to_shared(stg_generic);
    float rs = 0.f;
    if (row0 + lane < g.M) {
        float s = 0.f;
        const int row = row0 + lane;
        for (int t = 0; t < g.n_ssq; ++t) s += ld_f1<COH>(g.ssq_in + (size_t)row * g.n_ssq + t);
        rs = 1.0f / sqrtf(s * g.inv_d + g.eps);
    }
    if (!wait()) return false;
    tc_fence_after();
#pragma unroll 1
    for (int h = 0; h < NCOLS / 64; ++h) {
        // the staging tile is free once the previous copy has read it
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t r[32];
            tc_ld32(taddr + (uint32_t)((h * 2 + c) * 32), r);
            tc_wait_ld();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float lo, hi;
                    upk2(mul2(pk2(__uint_as_float(r[8 * j + 2 * e]), __uint_as_float(r[8 * j + 2 * e + 1])), pk2(rs, rs)), lo, hi);
                    if (EPI == EPI_SCALE_GELU) gelu_erf2(lo, hi);
                    w[e] = pack_bf16(lo, hi);
                }
                const int p = c * 4 + j;
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + (uint32_t)(lane * 128 + ((p ^ (lane & 7)) << 4))),
                             "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes before the copy engine reads them
        __syncwarp();
        if (lane == 0 && row0 < g.M) {
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(reinterpret_cast<uint64_t>(tmC)), "r"(n0 + h * 64), "r"(row0), "r"(stg) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
    }
    return true;
}
// Before a warp that used epilogue_store_tma leaves the kernel: its copies must have completed.
__device__ __forceinline__ void epilogue_store_drain()
{
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

}  // namespace tc
}  // namespace ebrl
