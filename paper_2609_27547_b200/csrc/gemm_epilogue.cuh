// The fused GEMM epilogue shared by the tensor-core GEMM kernels: one thread owns one output
// row of the tile and walks its accumulator columns 32 at a time out of tensor memory.
#pragma once
#include "actgen_internal.h"

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

__device__ __forceinline__ float gelu_erf(float z) { return 0.5f * z * (1.0f + erff(z * 0.70710678118654752440f)); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}


// EPI_SCALE_STORE: C = acc * rowscale;  EPI_SCALE_GELU: C = gelu(acc * rowscale);
// EPI_RESID: x += acc, xg = x * gain, one sum-of-squares partial per 128 columns.
// `taddr` = tensor-memory address of this warp's lane quarter and of the accumulator's first
// column; NCOLS columns starting at global column n0.  All 32 lanes must call it (tcgen05.ld is
// warp-collective); lanes with valid == false load and discard.
template <int EPI, int NCOLS>
__device__ __forceinline__ void epilogue_row(const GemmArgs &g, uint32_t taddr, int row, bool valid, int n0)
{
    float rs = 0.f;
    if (EPI != EPI_RESID && valid) {
        float s = 0.f;
        for (int t = 0; t < g.n_ssq; ++t) s += g.ssq_in[(size_t)row * g.n_ssq + t];
        rs = 1.0f / sqrtf(s * g.inv_d + g.eps);
    }
    float ss = 0.f;
#pragma unroll 1
    for (int c = 0; c < NCOLS / 32; ++c) {
        uint32_t r[32];
        tc_ld32(taddr + (uint32_t)c * 32, r);
        const int col = n0 + c * 32;
        if (EPI == EPI_RESID) {
            float4 xo[8];
            float *xp = g.x + (size_t)row * g.N + col;
            if (valid) {
#pragma unroll
                for (int j = 0; j < 8; ++j) xo[j] = *reinterpret_cast<const float4 *>(xp + 4 * j);
            }
            tc_wait_ld();
            if (valid) {
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float4 gn = *reinterpret_cast<const float4 *>(g.gain + col + 4 * j);
                    float4 xn;
                    xn.x = xo[j].x + __uint_as_float(r[4 * j + 0]);
                    xn.y = xo[j].y + __uint_as_float(r[4 * j + 1]);
                    xn.z = xo[j].z + __uint_as_float(r[4 * j + 2]);
                    xn.w = xo[j].w + __uint_as_float(r[4 * j + 3]);
                    *reinterpret_cast<float4 *>(xp + 4 * j) = xn;
                    ss = fmaf(xn.x, xn.x, ss); ss = fmaf(xn.y, xn.y, ss);
                    ss = fmaf(xn.z, xn.z, ss); ss = fmaf(xn.w, xn.w, ss);
                    pk[2 * j] = pack_bf16(xn.x * gn.x, xn.y * gn.y);
                    pk[2 * j + 1] = pack_bf16(xn.z * gn.z, xn.w * gn.w);
                }
                uint4 *xg = reinterpret_cast<uint4 *>((__nv_bfloat16 *)g.xg + (size_t)row * g.N + col);
#pragma unroll
                for (int j = 0; j < 4; ++j) xg[j] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                if ((c & 3) == 3) {
                    g.ssq_out[(size_t)row * (g.N / SSQ_W) + (col + 32 - SSQ_W) / SSQ_W] = ss;
                    ss = 0.f;
                }
            }
        } else {
            tc_wait_ld();
            if (valid) {
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    float a = __uint_as_float(r[2 * j]) * rs, b = __uint_as_float(r[2 * j + 1]) * rs;
                    if (EPI == EPI_SCALE_GELU) { a = gelu_erf(a); b = gelu_erf(b); }
                    pk[j] = pack_bf16(a, b);
                }
                uint4 *cp = reinterpret_cast<uint4 *>((__nv_bfloat16 *)g.C + (size_t)row * g.N + col);
#pragma unroll
                for (int j = 0; j < 4; ++j) cp[j] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
            }
        }
    }
}

}  // namespace tc
}  // namespace ebrl
