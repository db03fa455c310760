// Internal declarations shared by the translation units of libebrl_actgen (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace ebrl {

// Width (columns) of one sum-of-squares partial of the residual stream.  Every kernel that
// writes the residual stream x also writes, per row, sum(x^2) over each SSQ_W-column segment;
// consumers add the d/SSQ_W partials of a row in index order to get the RMSNorm scale.  The
// segment width is a constant of the library so that the value never depends on tile shapes.
constexpr int SSQ_W = 128;

// Per-environment record of one submitted group, in packed order (sorted by step count,
// longest first, so that the rows still active at inner step s are a prefix).
struct EnvMeta {
    const void *kv;    // device: [kv_layers][2][P][d]
    int32_t P;         // prefix length
    int32_t k0;        // Euler step index the environment starts from
    int32_t nsteps;    // steps to run in this submit
    int32_t row0;      // hidden-state prefixes: first row of the environment in the batch's packed prefix rows
    const float *noise;  // device: the environment's [H][A] state on entry
    float *out;          // device: where its [H][A] result goes
    const void *hid;   // hidden-state prefixes: device [P][d_ctx] as given by the caller (kv then points into the projected planes)
};

// Opaque storage of a CUtensorMap (the driver's 128-byte TMA descriptor).
struct alignas(64) TensorMap128 { uint64_t opaque[16]; };

enum Epilogue : int {
    EPI_SCALE_STORE = 0,   // C = acc * rowscale
    EPI_SCALE_GELU = 1,    // C = gelu(acc * rowscale)
    EPI_RESID = 2          // x += acc; xg = x * gain; ssq partials
};

struct GemmArgs {
    const void *A;         // [M][K] activations (T)
    const void *W;         // [N][K] weights (TW)
    int M, N, K;
    int epi;
    // EPI_SCALE_*: input row scale from ssq partials of the producer
    const float *ssq_in;   // [M][d/SSQ_W]
    int n_ssq;             // d / SSQ_W
    float inv_d, eps;
    void *C;               // [M][N] (T)
    // EPI_RESID
    float *x;              // [M][N] fp32 residual stream (N == d)
    const float *gain;     // [N] gain of the next RMSNorm
    void *xg;              // [M][N] (T)
    float *ssq_out;        // [M][N/SSQ_W]
    int test_drop_copies;  // tests of the give-up path: the copy-issuing thread issues nothing, every consumer's bounded wait runs out
    // fp32 models on the tensor cores: outputs that are the next projection's A operand (xg of the residual epilogue, C of
    // the GELU epilogue) are written as three bf16 term planes instead of one fp32 array; xg / C then name plane 0
    void *out_t1, *out_t2;
};

struct AttnArgs {
    const void *q;         // [rows][q_stride] (T), head h at columns h*hd
    int q_stride;
    void *out;             // [rows][o_stride] (T)
    int o_stride;
    int H, n_heads, hd;
    int n_envs;            // active environments
    // cross attention: keys/values from the environment's prefix planes
    const EnvMeta *meta;   // used when self == 0
    int d;                 // plane row length
    int kv_plane;          // plane pair index (layer index when kv_layers > 1, else 0)
    int plane_rows;        // rows from one plane of an environment to its next: 0 = the environment's own P
                           // (planes given by the caller), else the batch's packed prefix rows (projected planes)
    // self attention: keys/values are the environment's own rows
    int self;
    const void *k_self;    // [rows][kv_stride]
    const void *v_self;
    int kv_stride;
    // tensor-core kernel: TMA descriptors (device memory)
    const TensorMap128 *kv_maps;   // [n_envs]: the environment's planes as [kv_layers*2*P][d]
    const TensorMap128 *self_map;  // the QKV buffer as [rows][3d]
    int test_drop_copies;          // tests of the give-up path (see GemmArgs)
    void *out_t1, *out_t2;         // fp32 models on the tensor cores: out, out_t1, out_t2 = the three bf16 term planes of the result
    int split_out;
};

struct EmbedArgs {
    const EnvMeta *meta;
    int n_envs, H, A, d, s;        // s = inner step of this batch
    const float *a_state;          // [rows][A]
    const void *w_in;              // [d][A] (TW)
    const float *temb;             // [K][d]
    const float *gain;             // [d] gain of layer 0's first norm
    float *x;                      // [rows][d]
    void *xg;                      // [rows][d] (T)
    float *ssq;                    // [rows][d/SSQ_W]
    void *xg_t1, *xg_t2;           // fp32 models on the tensor cores: xg, xg_t1, xg_t2 = the three bf16 term planes of x * gain
    int split_xg;
};

struct HeadArgs {
    const EnvMeta *meta;
    int n_envs, H, A, d, s, K;
    float *a_state;
    const float *x;                // [rows][d]
    const float *gain;             // g_final
    const void *w_out;             // [A][d] (TW)
    const float *b_out;            // [A]
    float eps;
    int pull;                      // v = b_out - a
};

// Tensor-core GEMM (bf16 operands, fp32 accumulation in tensor memory).
int make_tmap_bf16(TensorMap128 *out, const void *base, uint64_t inner, uint64_t rows, uint32_t box_rows);
bool gemm_tc_supported(int N, int K);
int gemm_tc_box_rows_a();
int gemm_tc_box_rows_w();
cudaError_t launch_gemm_tc(const TensorMap128 &ta, const TensorMap128 &tw, const GemmArgs &a, int grid, int bn,
                           unsigned long long limit_ns, int *status, cudaStream_t st);

// The same GEMM on CTA pairs (tcgen05 cta_group::2, 256 x 256 tiles); needs grid >= 2.
cudaError_t launch_gemm_tc2(const TensorMap128 &ta, const TensorMap128 &tw, const GemmArgs &a, int grid,
                            unsigned long long limit_ns, int *status, cudaStream_t st);

// Tensor-core (mma.sync) attention over bulk-copied K/V rows, bf16 models.
bool attn_mma_supported(int H, int n_heads, int hd);
int attn_mma_slab_heads(int n_heads, int hd, bool wide);   // heads per slab: up to 16 x 64 or 8 x 128 columns when wide, else up to 8 heads
int attn_mma_make_map(TensorMap128 *out, const void *base, uint64_t rows, uint64_t width, int slab_heads, int hd);
cudaError_t launch_attn_mma(const AttnArgs &a, int grid, int slab_heads, int lookahead_blocks, unsigned long long limit_ns, int *status,
                            cudaStream_t st);

// fp32 GEMM on the tensor cores by splitting each operand into three bf16 terms (six products per k-slice).
bool gemm_tc3_supported(int N, int K);
cudaError_t launch_split3(const float *src, void *p0, void *p1, void *p2, size_t n, int grid, cudaStream_t st);
cudaError_t launch_gemm_tc3(const TensorMap128 *ta, const TensorMap128 *tw, const GemmArgs &a, int grid, unsigned long long limit_ns,
                            int *status, cudaStream_t st);
// the same on CTA pairs (256 x 256 tiles; N a multiple of 256, grid >= 2): bit-identical results (gemm_tc3p.cu)
bool gemm_tc3p_supported(int N, int K);
cudaError_t launch_gemm_tc3p(const TensorMap128 *ta, const TensorMap128 *tw, const GemmArgs &a, int grid, unsigned long long limit_ns,
                             int *status, cudaStream_t st);

// ---- the persistent step kernel (one resident grid for all Euler steps of a small batch) ----
// Per-layer table in device memory: TMA descriptors of the six matrices (128-row boxes) and the gains.
struct alignas(64) FusedLayerTab {
    TensorMap128 t_qkv, t_o, t_qc, t_oc, t_1, t_2;
    const float *g1, *g2, *g3;
};
// Per-slot table in device memory: descriptors of the activation buffers as A operands (128-row boxes)
// and as store targets of the epilogues (32-row x 64-column boxes).
struct alignas(64) FusedMaps {
    TensorMap128 a_xg, a_att, a_u, c_qkv, c_qc, c_u;
};
struct FusedArgs {
    int H, A, d, md, n_layers, n_heads, hd, hpc, K;
    int S, ne0;                    // inner steps of the batch, environments active at the first
    int kv_layers, plane_rows;
    float eps, inv_d;
    const EnvMeta *meta;           // packed order: environments still active at inner step s are a prefix
    const int *n_active;           // device [S]
    int *done;                     // device [S][mt_max] completion counters, zero on entry
    int mt_max;
    int *trace;                    // device [#CTAs][4] progress notes (task in hand per role), or NULL
    int test_drop_copies;          // tests of the give-up path: 1 = projections' copies, 2 = attention's copies are not issued
    float *a_state, *x, *ssq;
    void *xg, *qkv, *att, *qc, *u;
    const FusedMaps *maps;
    const TensorMap128 *attn_maps; // [0] = the QKV buffer, [1 + j] = environment j's planes
    const FusedLayerTab *layers;
    const void *w_in, *w_out;
    const float *b_out, *g_final, *temb;
};
bool fused_supported(int H, int A, int d, int md, int n_heads, int hd);
cudaError_t launch_fused_steps(const FusedArgs &f, int grid, unsigned long long limit_ns, int *status, cudaStream_t st);

// An SM partition (green context) with a stream inside it.
struct GreenPartition {
    void *ctx = nullptr;
    cudaStream_t stream = nullptr;
    int sm_count = 0;
    void *rest_ctx = nullptr;          // the complementary partition: every SM not in `ctx`
    cudaStream_t rest_stream = nullptr;
    int rest_sm_count = 0;
};
int green_partition_create(int device, int sm_quota, GreenPartition *out);
void green_partition_destroy(GreenPartition *p);

// Programmatic dependent launch: every kernel of a batch is launched with the attribute that lets
// its CTAs start (and run their on-chip set-up) while the previous kernel's last CTAs are still
// finishing; each kernel then calls pdl_wait() before it touches global memory of the batch, which
// blocks until the previous kernel has completed and its writes are visible.  Dependencies are
// unchanged; only the launch latency and the set-up move off the critical path.  The attribute is
// used only for batches whose grid fills every SM their stream can reach: under a smaller SM quota
// the early CTAs would park on SMs outside the quota (and measured slower).  pdl_set() states the
// choice for the calling thread's next launches (a handle created with EBRL_PDL=0 never turns it on).
void pdl_set(bool on);
bool pdl_enabled();
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kern)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, int cluster, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3((unsigned)block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (pdl_enabled()) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (cluster > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cluster;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (unsigned)n;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// Gathers the hidden-state prefixes of a batch into one [sum P][d_ctx] matrix (row0 of each
// environment from its record), the A operand of the K/V projections.
struct PackArgs {
    const EnvMeta *meta;
    int n_envs;
    int slices;            // 64-row slices per environment: ceil(longest prefix / 64)
    int row_bytes;         // d_ctx * sizeof(element), a multiple of 16
    void *dst;
};
cudaError_t launch_pack_prefix(const PackArgs &a, int grid, cudaStream_t st);

// Launchers (plain-ALU kernels).  bf16 != 0 selects bf16 activations/weights/planes.
// grid = number of persistent CTAs (the SM quota).
cudaError_t launch_embed(const EmbedArgs &a, int bf16, int grid, cudaStream_t st);
cudaError_t launch_head(const HeadArgs &a, int bf16, int grid, cudaStream_t st);
cudaError_t launch_gemm_simt(const GemmArgs &a, int bf16, int grid, cudaStream_t st);
cudaError_t launch_attn_simt(const AttnArgs &a, int bf16, int grid, cudaStream_t st);
// fp32 models, head_dim 64, H <= 8: one warp per (environment, head), operands in registers (attn_f32.cu)
bool attn_f32_supported(int H, int hd);
cudaError_t launch_attn_f32(const AttnArgs &a, int grid, cudaStream_t st);

}  // namespace ebrl
