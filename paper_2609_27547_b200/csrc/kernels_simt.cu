// Plain-ALU (FFMA) kernels of the action-generation path: input embedding, velocity head with
// the Euler update, a tiled GEMM with the fused epilogues, and softmax attention (self and
// cross).  They serve the fp32 models, whose 1e-4 accuracy bound rules out tensor cores, and
// they are the fall-back kernels of the bf16 models for shapes the tensor-core kernels do not
// cover.  Every kernel is a persistent grid of at most `grid` CTAs (the SM quota), and every
// output element is computed by a fixed sequence of operations that does not depend on the
// grid size or on which other rows share a tile.
#include "actgen_internal.h"
#include "rowops.cuh"
#include "split3.cuh"

namespace ebrl {

__device__ __forceinline__ float gelu_erf(float z) { return 0.5f * z * (1.0f + erff(z * 0.70710678118654752440f)); }

// ---------------------------------------------------------------------------------------
// x = W_in a + temb(t_k); xg = x * gain; sum-of-squares partials.  W_in is staged once per CTA
// in shared memory as fp32 [A][d]; one warp per row, each lane four consecutive columns of a
// 128-column segment at a time; the row's action vector lives in the lanes and is broadcast by
// shuffles.
// ---------------------------------------------------------------------------------------
template <typename T, int AMAX>
__global__ void __launch_bounds__(1024) embed_kernel(EmbedArgs a)
{
    extern __shared__ float wT[];   // [A][d]
    const int rows = a.n_envs * a.H;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const T *w_in = (const T *)a.w_in;
    pdl_launch_dependents();
    for (int c = threadIdx.x; c < a.d; c += blockDim.x)   // weights do not depend on the previous kernel
        for (int j = 0; j < a.A; ++j) wT[j * a.d + c] = ldf(w_in + (size_t)c * a.A + j);
    __syncthreads();
    pdl_wait();
    // two rows per warp pass: each staged weight is used for both
    for (int row0 = (blockIdx.x * 32 + warp) * 2; row0 < rows; row0 += gridDim.x * 64)
        embed_row_pair<T, AMAX, false>(a, row0, min(2, rows - row0), lane,
                                       [&](int j, int c) { return *reinterpret_cast<const float4 *>(wT + j * a.d + c); });
}

// ---------------------------------------------------------------------------------------
// v = W_out RMSNorm(x; g_final) + b_out;  a += v / K.  W_out is staged once per CTA in shared
// memory as fp32 [A][d]; one warp handles two rows per pass (each staged weight serves both),
// each lane four consecutive columns of a 128-column segment at a time.
// ---------------------------------------------------------------------------------------
constexpr int HEAD_WARPS = 16;

template <typename T, int AMAX>
__global__ void __launch_bounds__(HEAD_WARPS * 32) head_kernel(HeadArgs a)
{
    extern __shared__ float wO[];   // [A][d]
    const int rows = a.n_envs * a.H;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const T *w_out = (const T *)a.w_out;
    pdl_launch_dependents();
    if (!a.pull) {
        for (int e = threadIdx.x; e < a.A * a.d; e += blockDim.x) wO[e] = ldf(w_out + e);   // weights: no dependency
    }
    __syncthreads();
    pdl_wait();
    for (int row0 = (blockIdx.x * HEAD_WARPS + warp) * 2; row0 < rows; row0 += gridDim.x * HEAD_WARPS * 2)
        head_row_pair<T, AMAX, false>(a, row0, min(2, rows - row0), lane,
                                      [&](int j, int c) { return *reinterpret_cast<const float4 *>(wO + j * a.d + c); });
}

// ---------------------------------------------------------------------------------------
// C = A W^T with fused epilogues.  128 x 128 tile, 1024 threads, 4 x 4 outputs per thread;
// each output is one FMA chain over k = 0 .. K-1 in order.
// ---------------------------------------------------------------------------------------
constexpr int GT = 128, GK = 16, GPAD = 4;

template <typename T>
__device__ __forceinline__ void load2(const T *p, float &a, float &b);
template <> __device__ __forceinline__ void load2<float>(const float *p, float &a, float &b)
{
    const float2 v = *reinterpret_cast<const float2 *>(p); a = v.x; b = v.y;
}
template <> __device__ __forceinline__ void load2<__nv_bfloat16>(const __nv_bfloat16 *p, float &a, float &b)
{
    const __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162 *>(p);
    a = __bfloat162float(v.x); b = __bfloat162float(v.y);
}

template <typename T, int EPI>
__global__ void __launch_bounds__(1024) gemm_simt_kernel(GemmArgs g)
{
    __shared__ __align__(16) float As[2][GK][GT + GPAD];
    __shared__ __align__(16) float Ws[2][GK][GT + GPAD];
    const int tid = threadIdx.x, tx = tid & 31, ty = tid >> 5;
    const int lr = tid >> 3, lk = (tid & 7) * 2;
    const T *A = (const T *)g.A;
    const T *W = (const T *)g.W;
    const int ntm = (g.M + GT - 1) / GT, ntn = g.N / GT, ntiles = ntm * ntn, nk = g.K / GK;
    pdl_launch_dependents();
    pdl_wait();
    for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int m0 = (tile / ntn) * GT, n0 = (tile % ntn) * GT;
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
        const bool arow_ok = (m0 + lr) < g.M;
        const T *ap = A + (size_t)(m0 + lr) * g.K + lk;
        const T *wp = W + (size_t)(n0 + lr) * g.K + lk;
        float pa0 = 0.f, pa1 = 0.f, pw0, pw1;
        if (arow_ok) load2(ap, pa0, pa1);
        load2(wp, pw0, pw1);
        __syncthreads();   // previous tile's readers are done with both buffers
        As[0][lk][lr] = pa0; As[0][lk + 1][lr] = pa1;
        Ws[0][lk][lr] = pw0; Ws[0][lk + 1][lr] = pw1;
        __syncthreads();
        for (int kb = 0; kb < nk; ++kb) {
            const int buf = kb & 1;
            if (kb + 1 < nk) {
                if (arow_ok) load2(ap + (size_t)(kb + 1) * GK, pa0, pa1);
                load2(wp + (size_t)(kb + 1) * GK, pw0, pw1);
            }
#pragma unroll
            for (int k = 0; k < GK; ++k) {
                const float4 av = *reinterpret_cast<const float4 *>(&As[buf][k][ty * 4]);
                const float4 wv = *reinterpret_cast<const float4 *>(&Ws[buf][k][tx * 4]);
                const float aa[4] = {av.x, av.y, av.z, av.w};
                const float ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(aa[i], ww[j], acc[i][j]);
            }
            if (kb + 1 < nk) {
                As[buf ^ 1][lk][lr] = pa0; As[buf ^ 1][lk + 1][lr] = pa1;
                Ws[buf ^ 1][lk][lr] = pw0; Ws[buf ^ 1][lk + 1][lr] = pw1;
            }
            __syncthreads();
        }
        // ---- epilogue
        const int col = n0 + tx * 4;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = m0 + ty * 4 + i;
            const bool ok = row < g.M;
            if (EPI == EPI_RESID) {
                float ss = 0.f;
                float xn[4] = {0.f, 0.f, 0.f, 0.f};
                if (ok) {
                    const float4 xo = *reinterpret_cast<const float4 *>(g.x + (size_t)row * g.N + col);
                    xn[0] = xo.x + acc[i][0]; xn[1] = xo.y + acc[i][1];
                    xn[2] = xo.z + acc[i][2]; xn[3] = xo.w + acc[i][3];
                    *reinterpret_cast<float4 *>(g.x + (size_t)row * g.N + col) = make_float4(xn[0], xn[1], xn[2], xn[3]);
                    T *xg = (T *)g.xg + (size_t)row * g.N + col;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        stf(xg + j, xn[j] * g.gain[col + j]);
                        ss = fmaf(xn[j], xn[j], ss);
                    }
                }
                ss = warp_sum(ss);
                if (ok && tx == 0) g.ssq_out[(size_t)row * (g.N / SSQ_W) + n0 / SSQ_W] = ss;
            } else if (ok) {
                float s = 0.f;
                for (int t = 0; t < g.n_ssq; ++t) s += g.ssq_in[(size_t)row * g.n_ssq + t];
                const float rs = 1.0f / sqrtf(s * g.inv_d + g.eps);
                T *c = (T *)g.C + (size_t)row * g.N + col;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float v = acc[i][j] * rs;
                    if (EPI == EPI_SCALE_GELU) v = gelu_erf(v);
                    stf(c + j, v);
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// Softmax attention for one (environment, head) per 128-thread group, four groups per CTA.
// Keys are visited in blocks of 32 in index order with a running maximum and sum.
// ---------------------------------------------------------------------------------------
constexpr int AKB = 32;   // keys per block: a constant, so the arithmetic is the same at any quota

__device__ __forceinline__ void group_sync(int g) { asm volatile("bar.sync %0, 128;" ::"r"(g + 1) : "memory"); }

template <typename T> __device__ __forceinline__ void load4(const T *p, float (&v)[4]);
template <> __device__ __forceinline__ void load4<float>(const float *p, float (&v)[4])
{
    const float4 x = *reinterpret_cast<const float4 *>(p);
    v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
}
template <> __device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16 *p, float (&v)[4])
{
    const uint2 x = *reinterpret_cast<const uint2 *>(p);
    const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162 *>(&x.x), hi = *reinterpret_cast<const __nv_bfloat162 *>(&x.y);
    v[0] = __bfloat162float(lo.x); v[1] = __bfloat162float(lo.y); v[2] = __bfloat162float(hi.x); v[3] = __bfloat162float(hi.y);
}

// GROUPS items are in flight per CTA (one per 128 threads).  With head_dim <= 64 a thread's share of the next key
// block (four 16-byte pieces of K and of V) is requested into registers while the current block is computed, so the
// global-memory latency of a block hides behind the arithmetic of the one before it.
template <typename T, int RMAX, int GROUPS>
__global__ void __launch_bounds__(GROUPS * 128) attn_simt_kernel(AttnArgs a)
{
    extern __shared__ __align__(16) float smem[];
    const int grp = threadIdx.x >> 7, t = threadIdx.x & 127, warp = t >> 5, lane = t & 31;
    const int H = a.H, hd = a.hd;
    const int per_group = (H * hd + AKB * (hd + 4) + AKB * hd + H * AKB + 2 * H + 3) & ~3;   // 16-byte multiples: rows are read as float4
    float *q = smem + (size_t)grp * per_group;
    float *kb = q + H * hd;
    float *vb = kb + AKB * (hd + 4);   // key rows padded by four floats: float4 reads of 32 different rows do not collide
    float *p = vb + AKB * hd;
    float *alpha = p + H * AKB;
    float *lsum = alpha + H;
    const int hd_sh = hd == 32 ? 5 : (hd == 64 ? 6 : 7);   // head_dim is 32, 64 or 128: shifts, not divisions
    const int ncg = 128 >> hd_sh, c = t & (hd - 1), rg = t >> hd_sh;
    const float scale = 1.0f / sqrtf((float)hd);
    const int items = a.n_envs * a.n_heads;
    pdl_launch_dependents();
    pdl_wait();
    const bool ahead = hd <= 64;     // 32 * (hd / 4) / 128 <= 4 pieces per thread and plane
    for (int item = blockIdx.x * GROUPS + grp; item < items; item += gridDim.x * GROUPS) {
        const int env = item / a.n_heads, h = item - env * a.n_heads;
        const T *kbase, *vbase;
        int P, kvs;
        if (a.self) {
            kbase = (const T *)a.k_self + (size_t)env * H * a.kv_stride + h * hd;
            vbase = (const T *)a.v_self + (size_t)env * H * a.kv_stride + h * hd;
            P = H; kvs = a.kv_stride;
        } else {
            const EnvMeta m = a.meta[env];
            P = m.P; kvs = a.d;
            const int pr = a.plane_rows ? a.plane_rows : P;
            kbase = (const T *)m.kv + (size_t)a.kv_plane * 2 * pr * a.d + h * hd;
            vbase = kbase + (size_t)pr * a.d;
        }
        const T *qg = (const T *)a.q + (size_t)env * H * a.q_stride + h * hd;
        for (int e = t; e < H * hd; e += 128) {
            const int i = e >> hd_sh, cc = e & (hd - 1);
            q[e] = ldf(qg + (size_t)i * a.q_stride + cc) * scale;
        }
        float acc[RMAX];
#pragma unroll
        for (int r = 0; r < RMAX; ++r) acc[r] = 0.f;
        float mrun[8], lrun[8];   // rows warp, warp+4, ... (H <= 32)
#pragma unroll
        for (int r = 0; r < 8; ++r) { mrun[r] = -INFINITY; lrun[r] = 0.f; }
        // this thread's pieces of a key block: piece u is key j = e >> (hd_sh - 2), columns cc .. cc + 3, e = t + 128 u
        float kreg[4][4], vreg[4][4];
        auto fetch_block = [&](int j0) {
            const int nk = min(AKB, P - j0);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int e = t + 128 * u;
                const int j = e >> (hd_sh - 2), cc = (e & ((hd >> 2) - 1)) << 2;
#pragma unroll
                for (int x = 0; x < 4; ++x) kreg[u][x] = vreg[u][x] = 0.f;
                if (e < AKB * (hd >> 2) && j < nk) {
                    load4(kbase + (size_t)(j0 + j) * kvs + cc, kreg[u]);
                    load4(vbase + (size_t)(j0 + j) * kvs + cc, vreg[u]);
                }
            }
        };
        if (ahead) fetch_block(0);
        for (int j0 = 0; j0 < P; j0 += AKB) {
            group_sync(grp);   // q ready; previous block's readers done
            const int nkeys = min(AKB, P - j0);
            if (ahead) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int e = t + 128 * u;
                    if (e < AKB * (hd >> 2)) {
                        const int j = e >> (hd_sh - 2), cc = (e & ((hd >> 2) - 1)) << 2;
                        *reinterpret_cast<float4 *>(kb + j * (hd + 4) + cc) = make_float4(kreg[u][0], kreg[u][1], kreg[u][2], kreg[u][3]);
                        *reinterpret_cast<float4 *>(vb + j * hd + cc) = make_float4(vreg[u][0], vreg[u][1], vreg[u][2], vreg[u][3]);
                    }
                }
                if (j0 + AKB < P) fetch_block(j0 + AKB);   // lands while this block is computed
            } else {
                for (int e = t; e < AKB * (hd >> 2); e += 128) {   // four columns per thread and turn
                    const int j = e >> (hd_sh - 2), cc = (e & ((hd >> 2) - 1)) << 2;
                    float kv[4] = {0.f, 0.f, 0.f, 0.f}, vv[4] = {0.f, 0.f, 0.f, 0.f};
                    if (j < nkeys) {
                        load4(kbase + (size_t)(j0 + j) * kvs + cc, kv);
                        load4(vbase + (size_t)(j0 + j) * kvs + cc, vv);
                    }
                    *reinterpret_cast<float4 *>(kb + j * (hd + 4) + cc) = make_float4(kv[0], kv[1], kv[2], kv[3]);
                    *reinterpret_cast<float4 *>(vb + j * hd + cc) = make_float4(vv[0], vv[1], vv[2], vv[3]);
                }
            }
            group_sync(grp);
            // scores and running softmax statistics: lane = key, each warp owns rows warp + 4 r
#pragma unroll
            for (int r0 = 0; r0 < 8; r0 += 4) {
                if (warp + 4 * r0 >= H) continue;   // no query row in this pass (warp-uniform)
                float s[4] = {0.f, 0.f, 0.f, 0.f};
                // four columns at a time: one 16-byte read of the key row and one broadcast read per query row
                // feed 16 FMAs (the chain per score still runs over the columns in order)
                const float4 *krow = reinterpret_cast<const float4 *>(kb + lane * (hd + 4));
                for (int c4 = 0; c4 < (hd >> 2); ++c4) {
                    const float4 k4 = krow[c4];
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        const int i = warp + 4 * (r0 + r);
                        if (i < H) {
                            const float4 q4 = *reinterpret_cast<const float4 *>(q + i * hd + 4 * c4);
                            s[r] = fmaf(q4.x, k4.x, s[r]); s[r] = fmaf(q4.y, k4.y, s[r]);
                            s[r] = fmaf(q4.z, k4.z, s[r]); s[r] = fmaf(q4.w, k4.w, s[r]);
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int i = warp + 4 * (r0 + r);
                    if (i < H) {
                        const float sv = (lane < nkeys) ? s[r] : -INFINITY;
                        const float mnew = fmaxf(mrun[r0 + r], warp_max(sv));
                        const float pv = expf(sv - mnew);
                        const float al = expf(mrun[r0 + r] - mnew);
                        lrun[r0 + r] = lrun[r0 + r] * al + warp_sum(pv);
                        mrun[r0 + r] = mnew;
                        p[i * AKB + lane] = pv;
                        if (lane == 0) alpha[i] = al;
                    }
                }
            }
            group_sync(grp);
            // out += p v
#pragma unroll
            for (int r = 0; r < RMAX; ++r) {
                const int i = rg + ncg * r;
                if (i < H) acc[r] *= alpha[i];
            }
            // four keys at a time (weights and values of keys past the prefix are exact zeros: they add nothing)
            for (int j = 0; j < ((nkeys + 3) & ~3); j += 4) {
                const float v0 = vb[j * hd + c], v1 = vb[(j + 1) * hd + c], v2 = vb[(j + 2) * hd + c], v3 = vb[(j + 3) * hd + c];
#pragma unroll
                for (int r = 0; r < RMAX; ++r) {
                    const int i = rg + ncg * r;
                    if (i < H) {
                        const float4 p4 = *reinterpret_cast<const float4 *>(p + i * AKB + j);
                        acc[r] = fmaf(p4.x, v0, acc[r]); acc[r] = fmaf(p4.y, v1, acc[r]);
                        acc[r] = fmaf(p4.z, v2, acc[r]); acc[r] = fmaf(p4.w, v3, acc[r]);
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const int i = warp + 4 * r;
            if (i < H && lane == 0) lsum[i] = lrun[r];
        }
        group_sync(grp);
        T *og = (T *)a.out + (size_t)env * H * a.o_stride + h * hd + c;
#pragma unroll
        for (int r = 0; r < RMAX; ++r) {
            const int i = rg + ncg * r;
            if (i < H) {
                const float val = acc[r] / lsum[i];
                if (a.split_out) {   // the three bf16 terms of the result, for the tensor-core projection that follows
                    const size_t off = (size_t)env * H * a.o_stride + h * hd + c + (size_t)i * a.o_stride;
                    __nv_bfloat16 t0, t1, t2;
                    split3(val, t0, t1, t2);
                    ((__nv_bfloat16 *)a.out)[off] = t0; ((__nv_bfloat16 *)a.out_t1)[off] = t1; ((__nv_bfloat16 *)a.out_t2)[off] = t2;
                } else {
                    stf(og + (size_t)i * a.o_stride, val);
                }
            }
        }
        group_sync(grp);   // lsum, q are reused by the next item
    }
}

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------
template <typename T, int AMAX>
static cudaError_t embed_launch(const EmbedArgs &a, int g, size_t smem, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(embed_kernel<T, AMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_kernel(embed_kernel<T, AMAX>, g, 1024, smem, st, 1, a);
}

template <typename T>
static cudaError_t embed_dispatch(const EmbedArgs &a, int g, size_t smem, cudaStream_t st)
{
    if (a.A <= 8) return embed_launch<T, 8>(a, g, smem, st);
    if (a.A <= 16) return embed_launch<T, 16>(a, g, smem, st);
    return embed_launch<T, 32>(a, g, smem, st);
}

// Hidden-state prefixes: copy every environment's [P][d_ctx] rows to its place in the packed matrix.
// Items are (environment, 64-row slice) over a fixed number of slices per environment (the longest
// prefix of the batch); slices past an environment's own length are skipped.
__global__ void __launch_bounds__(512) pack_prefix_kernel(PackArgs a)
{
    pdl_launch_dependents();
    pdl_wait();
    const int vec_per_row = a.row_bytes >> 4;
    const int items = a.n_envs * a.slices;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int env = item / a.slices, r0 = (item - env * a.slices) << 6;
        const EnvMeta m = a.meta[env];
        if (r0 >= m.P) continue;
        const int nr = min(64, m.P - r0);
        const uint4 *src = reinterpret_cast<const uint4 *>((const char *)m.hid + (size_t)r0 * a.row_bytes);
        uint4 *dst = reinterpret_cast<uint4 *>((char *)a.dst + (size_t)(m.row0 + r0) * a.row_bytes);
        const int nvec = nr * vec_per_row;
        for (int v = threadIdx.x; v < nvec; v += blockDim.x) dst[v] = src[v];
    }
}

cudaError_t launch_pack_prefix(const PackArgs &a, int grid, cudaStream_t st)
{
    if (a.n_envs == 0) return cudaSuccess;
    return launch_kernel(pack_prefix_kernel, grid, 512, 0, st, 1, a);
}

cudaError_t launch_embed(const EmbedArgs &a, int bf16, int grid, cudaStream_t st)
{
    const int rows = a.n_envs * a.H;
    if (rows == 0) return cudaSuccess;
    const int need = (rows + 63) / 64;
    const int g = need < grid ? need : grid;
    const size_t smem = (size_t)a.d * a.A * sizeof(float);
    return bf16 ? embed_dispatch<__nv_bfloat16>(a, g, smem, st) : embed_dispatch<float>(a, g, smem, st);
}

template <typename T, int AMAX>
static cudaError_t head_launch(const HeadArgs &a, int g, size_t smem, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(head_kernel<T, AMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_kernel(head_kernel<T, AMAX>, g, HEAD_WARPS * 32, smem, st, 1, a);
}

template <typename T>
static cudaError_t head_dispatch(const HeadArgs &a, int g, size_t smem, cudaStream_t st)
{
    if (a.A <= 8) return head_launch<T, 8>(a, g, smem, st);
    if (a.A <= 16) return head_launch<T, 16>(a, g, smem, st);
    return head_launch<T, 32>(a, g, smem, st);
}

cudaError_t launch_head(const HeadArgs &a, int bf16, int grid, cudaStream_t st)
{
    const int rows = a.n_envs * a.H;
    if (rows == 0) return cudaSuccess;
    const int need = (rows + 2 * HEAD_WARPS - 1) / (2 * HEAD_WARPS);
    const int g = need < grid ? need : grid;
    const size_t smem = (size_t)a.d * a.A * sizeof(float);
    return bf16 ? head_dispatch<__nv_bfloat16>(a, g, smem, st) : head_dispatch<float>(a, g, smem, st);
}

template <typename T>
static cudaError_t gemm_simt_dispatch(const GemmArgs &a, int g, cudaStream_t st)
{
    switch (a.epi) {
    case EPI_SCALE_STORE: return launch_kernel(gemm_simt_kernel<T, EPI_SCALE_STORE>, g, 1024, 0, st, 1, a);
    case EPI_SCALE_GELU: return launch_kernel(gemm_simt_kernel<T, EPI_SCALE_GELU>, g, 1024, 0, st, 1, a);
    default: return launch_kernel(gemm_simt_kernel<T, EPI_RESID>, g, 1024, 0, st, 1, a);
    }
}

cudaError_t launch_gemm_simt(const GemmArgs &a, int bf16, int grid, cudaStream_t st)
{
    if (a.M == 0) return cudaSuccess;
    const int tiles = ((a.M + GT - 1) / GT) * (a.N / GT);
    const int g = tiles < grid ? tiles : grid;
    return bf16 ? gemm_simt_dispatch<__nv_bfloat16>(a, g, st) : gemm_simt_dispatch<float>(a, g, st);
}

template <typename T, int RMAX, int GROUPS>
static cudaError_t attn_launch(const AttnArgs &a, int grid, cudaStream_t st)
{
    const int items = a.n_envs * a.n_heads;
    const int need = (items + GROUPS - 1) / GROUPS;
    const int g = need < grid ? need : grid;
    const size_t per_group = ((size_t)a.H * a.hd + AKB * (a.hd + 4) + AKB * a.hd + a.H * AKB + 2 * a.H + 3) & ~(size_t)3;
    const size_t smem = GROUPS * per_group * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(attn_simt_kernel<T, RMAX, GROUPS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_kernel(attn_simt_kernel<T, RMAX, GROUPS>, g, GROUPS * 128, smem, st, 1, a);
}

template <typename T>
static cudaError_t attn_dispatch(const AttnArgs &a, int grid, cudaStream_t st)
{
    const int ncg = 128 / a.hd;
    const int R = (a.H + ncg - 1) / ncg;
    if (R <= 4) return attn_launch<T, 4, 4>(a, grid, st);
    if (R <= 8) return attn_launch<T, 8, 4>(a, grid, st);
    if (R <= 16) return attn_launch<T, 16, 4>(a, grid, st);
    return attn_launch<T, 32, 4>(a, grid, st);
}

cudaError_t launch_attn_simt(const AttnArgs &a, int bf16, int grid, cudaStream_t st)
{
    if (a.n_envs * a.n_heads == 0) return cudaSuccess;
    return bf16 ? attn_dispatch<__nv_bfloat16>(a, grid, st) : attn_dispatch<float>(a, grid, st);
}

}  // namespace ebrl
