// Row-wise pieces of the path that are not contractions: the input embedding with the timestep
// term, and the final RMSNorm + velocity head + Euler update.  One warp owns a pair of rows.
// Shared by the per-operation kernels and the persistent step kernel, so that both produce the
// same bits: a row's result is one fixed sequence of operations whoever calls it.
#pragma once
#include "actgen_internal.h"
#include "split3.cuh"

namespace ebrl {

template <typename T> __device__ __forceinline__ float ldf(const T *p);
template <> __device__ __forceinline__ float ldf<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T *p, float v);
template <> __device__ __forceinline__ void stf<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

template <typename T> __device__ __forceinline__ void store4(T *p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float *p, float a, float b, float c, float d)
{
    *reinterpret_cast<float4 *>(p) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16 *p, float a, float b, float c, float d)
{
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    *reinterpret_cast<uint2 *>(p) = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
}

// COH: the action state may have been written by another CTA of the same kernel -- read it through L2.
template <bool COH> __device__ __forceinline__ float row_ld(const float *p) { return COH ? __ldcg(p) : *p; }
template <bool COH> __device__ __forceinline__ float4 row_ld4(const float *p)
{
    return COH ? __ldcg(reinterpret_cast<const float4 *>(p)) : *reinterpret_cast<const float4 *>(p);
}

// x = W_in a + temb(t_k); xg = x * gain; sum-of-squares partials -- rows row0 and row0 + 1 (nr of them
// exist).  Each lane takes four consecutive columns of a 128-column segment at a time; the rows' action
// vectors live in the lanes and are broadcast by shuffles.  w4(j, c) returns W_in[c .. c+3][j] as fp32.
template <typename T, int AMAX, bool COH, typename W4>
__device__ __forceinline__ void embed_row_pair(const EmbedArgs &a, int row0, int nr, int lane, W4 w4)
{
    const int nseg = a.d / SSQ_W;
    T *xg = (T *)a.xg;
    float aj[2][AMAX];
    int kk[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = row0 + (r < nr ? r : 0);
        const int env = row / a.H, h = row - env * a.H;
        const EnvMeta m = a.meta[env];
        kk[r] = m.k0 + a.s;
        const float *av = (a.s == 0) ? m.noise + (size_t)h * a.A : a.a_state + (size_t)row * a.A;
        const float mine = lane < a.A ? row_ld<COH>(av + lane) : 0.f;
#pragma unroll
        for (int j = 0; j < AMAX; ++j) aj[r][j] = __shfl_sync(0xffffffffu, mine, j);
    }
    for (int seg = 0; seg < nseg; ++seg) {
        const int c = seg * SSQ_W + 4 * lane;
        float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int j = 0; j < AMAX; ++j) {
            if (j < a.A) {
                const float4 w = w4(j, c);
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    acc[r][0] = fmaf(w.x, aj[r][j], acc[r][0]); acc[r][1] = fmaf(w.y, aj[r][j], acc[r][1]);
                    acc[r][2] = fmaf(w.z, aj[r][j], acc[r][2]); acc[r][3] = fmaf(w.w, aj[r][j], acc[r][3]);
                }
            }
        }
        const float4 gn = *reinterpret_cast<const float4 *>(a.gain + c);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            if (r < nr) {
                const int row = row0 + r;
                const float4 te = *reinterpret_cast<const float4 *>(a.temb + (size_t)kk[r] * a.d + c);
                const float v0 = acc[r][0] + te.x, v1 = acc[r][1] + te.y, v2 = acc[r][2] + te.z, v3 = acc[r][3] + te.w;
                *reinterpret_cast<float4 *>(a.x + (size_t)row * a.d + c) = make_float4(v0, v1, v2, v3);
                if (a.split_xg) store_split4(a.xg, a.xg_t1, a.xg_t2, (size_t)row * a.d + c, v0 * gn.x, v1 * gn.y, v2 * gn.z, v3 * gn.w);
                else store4<T>(xg + (size_t)row * a.d + c, v0 * gn.x, v1 * gn.y, v2 * gn.z, v3 * gn.w);
                float ss = v0 * v0;
                ss = fmaf(v1, v1, ss); ss = fmaf(v2, v2, ss); ss = fmaf(v3, v3, ss);
                ss = warp_sum(ss);
                if (lane == 0) a.ssq[(size_t)row * nseg + seg] = ss;
            }
        }
    }
}

// v = W_out RMSNorm(x; g_final) + b_out;  a += v / K -- rows row0 and row0 + 1.  Each lane takes four
// consecutive columns of a 128-column segment at a time, four segments per round so that the eight row
// loads of a round are in flight together.  w4(j, c) returns W_out[j][c .. c+3] as fp32.
template <typename T, int AMAX, bool COH, typename W4>
__device__ __forceinline__ void head_row_pair(const HeadArgs &a, int row0, int nr, int lane, W4 w4)
{
    float acc[2][AMAX];
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int j = 0; j < AMAX; ++j) acc[r][j] = 0.f;
    float ss[2] = {0.f, 0.f};
    if (!a.pull) {
        for (int c0 = lane * 4; c0 < a.d; c0 += 512) {
            float4 xv[4][2], gv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int c = c0 + u * 128;
                if (c < a.d) {
                    gv[u] = *reinterpret_cast<const float4 *>(a.gain + c);
#pragma unroll
                    for (int r = 0; r < 2; ++r)
                        xv[u][r] = row_ld4<COH>(a.x + (size_t)(row0 + (r < nr ? r : 0)) * a.d + c);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int c = c0 + u * 128;
                if (c < a.d) {
                    float t[2][4];
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        const float4 x4 = xv[u][r];
                        ss[r] = fmaf(x4.x, x4.x, ss[r]); ss[r] = fmaf(x4.y, x4.y, ss[r]);
                        ss[r] = fmaf(x4.z, x4.z, ss[r]); ss[r] = fmaf(x4.w, x4.w, ss[r]);
                        t[r][0] = x4.x * gv[u].x; t[r][1] = x4.y * gv[u].y; t[r][2] = x4.z * gv[u].z; t[r][3] = x4.w * gv[u].w;
                    }
#pragma unroll
                    for (int j = 0; j < AMAX; ++j) {
                        if (j < a.A) {
                            const float4 w = w4(j, c);
#pragma unroll
                            for (int r = 0; r < 2; ++r) {
                                acc[r][j] = fmaf(t[r][0], w.x, acc[r][j]); acc[r][j] = fmaf(t[r][1], w.y, acc[r][j]);
                                acc[r][j] = fmaf(t[r][2], w.z, acc[r][j]); acc[r][j] = fmaf(t[r][3], w.w, acc[r][j]);
                            }
                        }
                    }
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        if (r < nr) {   // warp-uniform
            const int row = row0 + r;
            const int env = row / a.H, h = row - env * a.H;
            const EnvMeta m = a.meta[env];
            const float ssr = a.pull ? 0.f : warp_sum(ss[r]);
            const float inv = 1.0f / sqrtf(ssr / (float)a.d + a.eps);
            const float *a_old = (a.s == 0) ? m.noise + (size_t)h * a.A : a.a_state + (size_t)row * a.A;
#pragma unroll
            for (int j = 0; j < AMAX; ++j) {
                if (j < a.A) {
                    const float dot = warp_sum(acc[r][j]);
                    if (lane == 0) {
                        const float ao = row_ld<COH>(a_old + j);
                        const float v = a.pull ? (a.b_out[j] - ao) : (dot * inv + a.b_out[j]);
                        const float an = ao + v / (float)a.K;
                        a.a_state[(size_t)row * a.A + j] = an;
                        if (a.s == m.nsteps - 1) m.out[(size_t)h * a.A + j] = an;
                    }
                }
            }
        }
    }
}

}  // namespace ebrl
