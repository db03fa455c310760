// An entry point for callers that must not allocate: one Euler step of a layer-less action head
// (embedding + timestep term, final RMSNorm, velocity head, a += v/K) whose intermediate
// residual stream lives in a fixed device array compiled into the library instead of in
// memory obtained with cudaMalloc.
//
// Who needs this: code that runs where device allocation is forbidden or would stall -- inside
// a latency-critical control loop that may not take the allocator's lock or trigger an implicit
// device synchronisation, inside a process whose memory budget was handed out in full at
// start-up (a generation worker sharing a GPU with training under a fixed memory descriptor),
// or in a plug-in that is only given pointers and a stream.  Such a caller passes every input
// and output itself; the library brings its own scratch.
#include "../../include/ebrl_actgen.h"
#include "actgen_internal.h"

#include <mutex>

namespace {

constexpr int NA_MAX_ROWS = 512;     // rows (environments x action tokens) per call
constexpr int NA_MAX_D = 1024;       // model width
constexpr int NA_MAX_A = 32;

// The scratch: the fp32 residual stream x [rows][d] of one call.  Lives in every GPU that loads
// the library until the process exits (2 MiB).  Every call uses it from the start, so calls
// that overlap on the GPU would overwrite each other's rows.
static __device__ __align__(256) float g_noalloc_x[NA_MAX_ROWS * NA_MAX_D];

constexpr int MAX_DEVICES = 64;
float *g_scratch_addr[MAX_DEVICES];   // device address of g_noalloc_x on each device, once known
std::mutex g_setup_mu;

__device__ __forceinline__ float na_warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// x[row][c] = sum_j W_in[c][j] a[row][j] + temb[c]   (one warp per (row, 128-column segment))
__global__ void __launch_bounds__(1024) na_embed_kernel(const float *a_in, const float *w_in, const float *temb, float *x,
                                                        int rows, int A, int d)
{
    const int nseg = d / ebrl::SSQ_W, units = rows * nseg;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int u = blockIdx.x * 32 + warp; u < units; u += gridDim.x * 32) {
        const int row = u / nseg, seg = u - row * nseg;
        const float mine = lane < A ? a_in[(size_t)row * A + lane] : 0.f;
#pragma unroll
        for (int i = 0; i < ebrl::SSQ_W / 32; ++i) {
            const int c = seg * ebrl::SSQ_W + i * 32 + lane;
            float acc = 0.f;
            for (int j = 0; j < A; ++j) acc = fmaf(w_in[(size_t)c * A + j], __shfl_sync(0xffffffffu, mine, j), acc);
            x[(size_t)row * d + c] = acc + temb[c];
        }
    }
}

// v = W_out (g x / rms(x)) + b;  a_out = a_in + v / K   (one warp per row)
__global__ void __launch_bounds__(256) na_head_kernel(const float *a_in, float *a_out, const float *x, const float *gain,
                                                      const float *w_out, const float *b_out, int rows, int A, int d, int K, float eps)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int row = blockIdx.x * 8 + warp; row < rows; row += gridDim.x * 8) {
        const float *xr = x + (size_t)row * d;
        float acc[NA_MAX_A];
#pragma unroll
        for (int j = 0; j < NA_MAX_A; ++j) acc[j] = 0.f;
        float ss = 0.f;
        for (int c = lane; c < d; c += 32) {
            const float xv = xr[c];
            ss = fmaf(xv, xv, ss);
            const float t = xv * gain[c];
#pragma unroll
            for (int j = 0; j < NA_MAX_A; ++j)
                if (j < A) acc[j] = fmaf(t, w_out[(size_t)j * d + c], acc[j]);
        }
        ss = na_warp_sum(ss);
        const float inv = 1.0f / sqrtf(ss / (float)d + eps);
#pragma unroll
        for (int j = 0; j < NA_MAX_A; ++j) {
            if (j < A) {
                const float dot = na_warp_sum(acc[j]);
                if (lane == 0) {
                    const float ao = a_in[(size_t)row * A + j];
                    a_out[(size_t)row * A + j] = ao + (dot * inv + b_out[j]) / (float)K;
                }
            }
        }
    }
}

}  // namespace

extern "C" ebrl_status_t ebrl_actgen_l0_step_noalloc(const float *a_in, float *a_out, const float *w_in, const float *w_out,
                                                     const float *b_out, const float *g_final, const float *temb_row,
                                                     int32_t n_rows, int32_t A, int32_t d, int32_t K_steps, float rms_eps,
                                                     int32_t sm_quota, void *stream)
{
    if (!a_in || !a_out || !w_in || !w_out || !b_out || !g_final || !temb_row) return EBRL_ERR_INVALID_ARG;
    if (n_rows < 0 || A < 1 || d < 1 || K_steps < 1 || sm_quota < 0 || !(rms_eps >= 0.f)) return EBRL_ERR_INVALID_ARG;
    if (n_rows > NA_MAX_ROWS || d > NA_MAX_D || A > NA_MAX_A || d % ebrl::SSQ_W) return EBRL_ERR_UNSUPPORTED;   // beyond the fixed scratch
    if (n_rows == 0) return EBRL_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return EBRL_ERR_CUDA;
    float *x = nullptr;
    {
        // First call on this device: ask the runtime where g_noalloc_x lives on the CURRENT
        // device.  In host code the symbol's name is only a handle, never a device address.
        std::lock_guard<std::mutex> lk(g_setup_mu);
        if (!g_scratch_addr[dev]) {
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, g_noalloc_x) != cudaSuccess || !p) { cudaGetLastError(); return EBRL_ERR_CUDA; }
            g_scratch_addr[dev] = (float *)p;
        }
        x = g_scratch_addr[dev];
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return EBRL_ERR_CUDA;
    if (sm_quota > sms) return EBRL_ERR_QUOTA;
    const int grid = sm_quota == 0 ? sms : sm_quota;
    cudaStream_t st = (cudaStream_t)stream;
    const int units = n_rows * (d / ebrl::SSQ_W);
    const int g1 = (units + 31) / 32 < grid ? (units + 31) / 32 : grid;
    na_embed_kernel<<<g1, 1024, 0, st>>>(a_in, w_in, temb_row, x, n_rows, A, d);
    const int g2 = (n_rows + 7) / 8 < grid ? (n_rows + 7) / 8 : grid;
    na_head_kernel<<<g2, 256, 0, st>>>(a_in, a_out, x, g_final, w_out, b_out, n_rows, A, d, K_steps, rms_eps);
    return cudaGetLastError() == cudaSuccess ? EBRL_OK : EBRL_ERR_CUDA;
}
