// The C-ABI boundary of libebrl_actgen: argument validation, the ragged group batcher, the
// per-group launch sequence and completion tracking.  All arithmetic of the path runs in the
// kernels this file launches; nothing here computes on the host except the timestep-embedding
// table built once at create.
#include "../../include/ebrl_actgen.h"
#include "actgen_internal.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <unordered_set>
#include <vector>

using namespace ebrl;

namespace ebrl {
static thread_local bool t_pdl = false;
void pdl_set(bool on) { t_pdl = on; }
bool pdl_enabled() { return t_pdl; }
}  // namespace ebrl

namespace {

struct LayerDev {
    float *g1 = nullptr, *g2 = nullptr, *g3 = nullptr;
    void *w_qkv = nullptr, *w_o = nullptr, *w_qc = nullptr, *w_oc = nullptr, *w_1 = nullptr, *w_2 = nullptr;
    void *w_kc = nullptr, *w_vc = nullptr;           // hidden-state prefixes (cfg.d_ctx > 0): [d][d_ctx] each
    TensorMap128 t_qkv, t_o, t_qc, t_oc, t_1, t_2, t_kc, t_vc;   // TMA descriptors of the matrices (tensor-core path)
    // fp32 models on the tensor cores: the three bf16 terms of each matrix (0 qkv, 1 o, 2 qc, 3 oc, 4 w_1, 5 w_2) and their descriptors
    void *w3[6][3] = {};
    TensorMap128 t3[6][3];
};

// One complete copy of the policy's weights on the device.  The handle keeps two, so that a new
// policy version can be uploaded while batches launched under the previous one still run.
struct WeightSet {
    void *w_in = nullptr, *w_out = nullptr;
    float *b_out = nullptr, *g_final = nullptr;
    std::vector<LayerDev> layers;
    FusedLayerTab *ftab_d = nullptr;   // the persistent step kernel's per-layer table (descriptors + gains) in device memory
    bool allocated = false, ever_used = false;
    uint64_t version = 0;
    cudaEvent_t ready = nullptr;      // upload complete
    cudaEvent_t last_use = nullptr;   // last batch that reads this set
};

struct TimedLaunch {
    cudaEvent_t t0, t1;
    int cls;
    double flops, bytes;
};

struct HostCopy {
    void *dst;
    const void *src;
    size_t bytes;
};

struct Slot {
    float *a_state = nullptr, *x = nullptr, *ssq = nullptr;
    void *xg = nullptr, *qkv = nullptr, *att = nullptr, *qc = nullptr, *u = nullptr;
    EnvMeta *meta_d = nullptr, *meta_h = nullptr;
    TensorMap128 t_xg, t_att, t_u;                    // TMA descriptors of the A operands
    // fp32 models on the tensor cores: the projections' A operands as three bf16 term planes each, written by their producers
    void *xg3[3] = {}, *att3[3] = {}, *u3[3] = {};
    TensorMap128 t_xg3[3], t_att3[3], t_u3[3];
    FusedMaps *fmaps_d = nullptr;                     // persistent step kernel: the same plus the epilogues' store targets, in device memory
    int *fctl_d = nullptr, *fctl_h = nullptr;         // its control block: n_active[K] then the completion counters [K][mt_max]
    int mt_max = 0;
    TensorMap128 *maps_d = nullptr, *maps_h = nullptr; // attention descriptors: [0] = QKV buffer, [1 + j] = env j's planes
    cudaEvent_t done = nullptr;
    bool busy = false;
    int wset = 0;                                     // weight set the slot's batch in flight reads
    std::vector<int64_t> ids;
    // staging of the host-buffer entry point (allocated on first use)
    char *kv_stage = nullptr;
    size_t kv_stage_bytes = 0;
    float *noise_stage = nullptr, *out_stage = nullptr;
    std::vector<TimedLaunch> timed;
    size_t timed_used = 0;
    // groups queued in this slot and not yet launched
    std::vector<EnvMeta> pending;
    std::vector<TensorMap128> pending_maps;   // TMA descriptor of each pending environment's planes (encoded at submit)
    std::vector<HostCopy> copies_out;
    cudaStream_t stream = nullptr;
    int grid = 0, groups_pending = 0;
    size_t stage_used = 0, chunks_used = 0;
    cudaEvent_t h2d_done = nullptr, part_in = nullptr, part_out = nullptr;
    bool has_uploads = false;
    // hidden-state prefixes: the batch's packed hidden rows and the planes projected from them
    // ([n_layers][2][prefix_rows][d]); both grow to the largest batch seen
    void *hid_pack = nullptr, *planes = nullptr;
    size_t proj_cap_rows = 0;
    int prefix_rows = 0, prefix_slices = 0;   // of the batch being launched
    TensorMap128 t_hid;
};

thread_local std::string g_create_error;

}  // namespace

struct ebrl_actgen {
    ebrl_actgen_cfg_t cfg;
    int bf16 = 0, n_sms = 0, hd = 0, md = 0;
    bool use_tc = false;          // tensor-core GEMMs (bf16, d a multiple of 256)
    bool use_tc3 = false;         // fp32 models: projections on the tensor cores by three-term bf16 splitting
    bool use_pairs = true;        // CTA-pair GEMM allowed (EBRL_GEMM_PAIR=0 forbids it)
    int force_shape = 0;          // EBRL_GEMM_SHAPE = 2 (pairs), 256 or 128 forces one tile shape (tests, tuning)
    bool trace = false;           // EBRL_TRACE=1: the persistent kernel notes its progress; a time-out prints it to stderr
    Slot *trace_slot = nullptr;
    bool fused_ok = false;        // the persistent step kernel covers this model
    long fused_max_rows = 0;      // batches of at most this many rows take it by themselves (EBRL_FUSED_MAX_ROWS); 0: only when forced --
                                  // measured on B200 it is bit-identical to, but slower than, the per-operation kernels at every size tried
    bool pdl_allowed = true;      // EBRL_PDL=0 turns programmatic dependent launch off
    int attn_lookahead = 2;       // EBRL_ATTN_LOOKAHEAD: key blocks the attention producer asks L2 for ahead of its ring
    bool use_attn_mma = false;    // tensor-core attention (bf16, H <= 16, head_dim 64/128)
    int attn_hpc = 8;             // heads per slab of the tensor-core attention kernel and its descriptors
    bool use_attn_f32 = false;    // warp-per-item fp32 attention (head_dim 64, H <= 8)
    int *status_d = nullptr;      // device status word written by kernels whose waits ran out
    unsigned long long wait_ns = 0;
    size_t esz = 4;   // bytes per element of matrices / activations / planes
    WeightSet wset[2];
    int active = 0;               // the set new batches use
    uint64_t version = 1;         // policy version of wset[active]
    float *temb = nullptr;
    std::vector<Slot> slots;
    size_t fill = 0;              // slot collecting groups for the next batch
    size_t stage_hint = 0;        // plane staging a full batch has needed so far (bytes per slot)
    int host_depth = 1;           // groups per batch of host-staged submits: doubles per batch, back to 1 at sync
    std::unordered_set<int64_t> busy_ids;
    std::mutex mu;
    std::string err;
    ebrl_status_t sticky = EBRL_OK;
    ebrl_actgen_stats_t stats;
    std::vector<void *> owned;   // every device allocation, for destroy
    std::vector<std::pair<const char *, const char *>> canaries;   // EBRL_FLAG_DEBUG_CANARY: guard address and buffer name
    std::map<int, GreenPartition> partitions;   // SM partitions by quota (EBRL_FLAG_GREEN_CTX); ctx == nullptr: creation failed
    cudaStream_t copy_stream = nullptr;   // host-buffer entry point: uploads run here, beside the previous batch's kernels
};

namespace {

ebrl_status_t fail(ebrl_actgen *h, ebrl_status_t st, const char *fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (h) h->err = buf; else g_create_error = buf;
    return st;
}

// ---- pure host checks (also exported for tests that have no GPU) --------------------------

ebrl_status_t check_cfg(const ebrl_actgen_cfg_t *c, std::string *why)
{
    auto bad = [&](ebrl_status_t st, const char *m) { if (why) *why = m; return st; };
    if (!c) return bad(EBRL_ERR_INVALID_ARG, "cfg is NULL");
    if (c->abi_version != EBRL_ACTGEN_ABI_VERSION) return bad(EBRL_ERR_INVALID_ARG, "abi_version mismatch");
    if (c->H < 1 || c->A < 1 || c->d < 2 || c->n_layers < 0 || c->n_heads < 1 || c->mlp_mult < 1 || c->K_steps < 1)
        return bad(EBRL_ERR_INVALID_ARG, "H, A, d, n_heads, mlp_mult, K_steps must be positive and n_layers >= 0");
    if (c->d % 2) return bad(EBRL_ERR_INVALID_ARG, "d must be even (sin/cos halves of the timestep embedding)");
    if (c->d % c->n_heads) return bad(EBRL_ERR_INVALID_ARG, "d must be a multiple of n_heads");
    if (c->max_prefix_len < 1 || c->max_group_envs < 1 || c->max_inflight_groups < 1)
        return bad(EBRL_ERR_INVALID_ARG, "max_prefix_len, max_group_envs, max_inflight_groups must be >= 1");
    if ((c->param_dtype != EBRL_F32 && c->param_dtype != EBRL_BF16) || (c->kv_dtype != EBRL_F32 && c->kv_dtype != EBRL_BF16))
        return bad(EBRL_ERR_INVALID_ARG, "unknown dtype");
    if (c->kv_layers != 1 && c->kv_layers != c->n_layers) return bad(EBRL_ERR_INVALID_ARG, "kv_layers must be 1 or n_layers");
    if (!(c->rms_eps >= 0.f) || !(c->temb_max_period > 0.f)) return bad(EBRL_ERR_INVALID_ARG, "rms_eps >= 0 and temb_max_period > 0 required");
    if (c->H > 32 || c->A > 32) return bad(EBRL_ERR_UNSUPPORTED, "H and A up to 32 are supported");
    if (c->d % SSQ_W) return bad(EBRL_ERR_UNSUPPORTED, "d must be a multiple of 128");
    const int hd = c->d / c->n_heads;
    if (hd != 32 && hd != 64 && hd != 128) return bad(EBRL_ERR_UNSUPPORTED, "head_dim must be 32, 64 or 128");
    if (c->param_dtype != c->kv_dtype) return bad(EBRL_ERR_UNSUPPORTED, "param_dtype and kv_dtype must match");
    if ((int64_t)c->d * c->A * 4 > 200 * 1024) return bad(EBRL_ERR_UNSUPPORTED, "d * A is limited to 51200 (the input embedding is staged in shared memory)");
    if (c->d_ctx < 0) return bad(EBRL_ERR_INVALID_ARG, "d_ctx < 0");
    if (c->d_ctx > 0) {
        if (c->kv_layers != c->n_layers) return bad(EBRL_ERR_INVALID_ARG, "d_ctx > 0 (hidden-state prefixes) needs kv_layers == n_layers");
        if (c->d_ctx % 64) return bad(EBRL_ERR_UNSUPPORTED, "d_ctx must be a multiple of 64");
    }
    if ((int64_t)c->max_group_envs * c->max_inflight_groups * c->H > (int64_t)1 << 22)
        return bad(EBRL_ERR_UNSUPPORTED, "max_group_envs * max_inflight_groups * H is limited to 4M rows");
    return EBRL_OK;
}

ebrl_status_t check_submit(const ebrl_actgen_cfg_t *c, int n_sms, int32_t n, const int64_t *env_ids,
                           const void *const *prefix_kv, const void *noise, const void *out,
                           int32_t sm_quota, const ebrl_submit_ext_t *ext, std::string *why)
{
    auto bad = [&](ebrl_status_t st, const std::string &m) { if (why) *why = m; return st; };
    if (n < 0) return bad(EBRL_ERR_INVALID_ARG, "n_envs < 0");
    if (sm_quota < 0 || sm_quota > n_sms) return bad(EBRL_ERR_QUOTA, "sm_quota outside 0..#SMs");
    if (n == 0) return EBRL_OK;
    if (n > c->max_group_envs) return bad(EBRL_ERR_INVALID_ARG, "n_envs > max_group_envs");
    if (!env_ids || !noise || !out) return bad(EBRL_ERR_INVALID_ARG, "env_ids, noise and out must not be NULL");
    const bool pull = (c->flags & EBRL_FLAG_TEST_PULL) != 0;
    if (!pull && !prefix_kv) return bad(EBRL_ERR_INVALID_ARG, "prefix_kv is NULL");
    if (ext && ext->n_steps < 0) return bad(EBRL_ERR_INVALID_ARG, "n_steps < 0");
    std::unordered_set<int64_t> seen;
    for (int i = 0; i < n; ++i) {
        if (!seen.insert(env_ids[i]).second) return bad(EBRL_ERR_INVALID_ARG, "duplicate env id " + std::to_string(env_ids[i]));
        if (!pull) {
            if (!prefix_kv[i]) return bad(EBRL_ERR_INVALID_ARG, "prefix_kv[" + std::to_string(i) + "] is NULL");
            if (((uintptr_t)prefix_kv[i]) & 15) return bad(EBRL_ERR_INVALID_ARG, "prefix_kv[" + std::to_string(i) + "] is not 16-byte aligned");
        }
        if (ext && ext->prefix_len) {
            const int P = ext->prefix_len[i];
            if (P < 1 || P > c->max_prefix_len) return bad(EBRL_ERR_INVALID_ARG, "prefix_len[" + std::to_string(i) + "] outside 1..max_prefix_len");
        }
        if (ext && ext->step_index) {
            const int k = ext->step_index[i];
            if (k < 0 || k >= c->K_steps) return bad(EBRL_ERR_INVALID_ARG, "step_index[" + std::to_string(i) + "] outside [0, K)");
        }
    }
    return EBRL_OK;
}

// The ragged batcher's plan: environments sorted by the number of steps they run (longest
// first, ties in arrival order) so that the rows active at inner step s form a prefix.
// order[j] = caller index of packed position j; n_active[s] = environments with more than s
// steps.  Returns S = the largest step count.
int plan_group(const ebrl_actgen_cfg_t *c, int n, const ebrl_submit_ext_t *ext, int32_t *order,
               int32_t *nsteps, int32_t *n_active)
{
    const int K = c->K_steps;
    std::vector<int> steps(n);
    for (int i = 0; i < n; ++i) {
        const int k0 = (ext && ext->step_index) ? ext->step_index[i] : 0;
        int s = K - k0;
        if (ext && ext->n_steps > 0 && ext->n_steps < s) s = ext->n_steps;
        steps[i] = s;
    }
    for (int i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order, order + n, [&](int a, int b) { return steps[a] > steps[b]; });
    int S = 0;
    for (int j = 0; j < n; ++j) { nsteps[j] = steps[order[j]]; S = std::max(S, nsteps[j]); }
    for (int s = 0; s < K; ++s) {
        int cnt = 0;
        while (cnt < n && nsteps[cnt] > s) ++cnt;
        n_active[s] = cnt;
    }
    return S;
}

// ---- device helpers ---------------------------------------------------------------------

#define CK(call)                                                                              \
    do {                                                                                      \
        cudaError_t e_ = (call);                                                              \
        if (e_ != cudaSuccess)                                                                \
            return fail(h, EBRL_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));    \
    } while (0)

constexpr size_t CANARY_BYTES = 256;
constexpr int CANARY_BYTE = 0xA5;

// With EBRL_FLAG_DEBUG_CANARY every buffer gets a tail of CANARY_BYTES filled with a pattern that no kernel may
// touch; ebrl_actgen_sync checks the tails (a stand-in for a memory checker: a write past a buffer's end shows up
// as a changed tail, named in the error text).
ebrl_status_t dev_alloc(ebrl_actgen *h, void **p, size_t bytes, const char *what = "buffer")
{
    *p = nullptr;
    const bool canary = (h->cfg.flags & EBRL_FLAG_DEBUG_CANARY) != 0;
    const size_t body = (bytes ? bytes : 16);
    const size_t padded = (body + 15) & ~(size_t)15;
    cudaError_t e = cudaMalloc(p, canary ? padded + CANARY_BYTES : body);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(h, EBRL_ERR_NOMEM, "cudaMalloc of %zu bytes failed: %s", bytes, cudaGetErrorString(e));
    }
    h->owned.push_back(*p);
    if (canary) {
        if (cudaMemset((char *)*p + padded, CANARY_BYTE, CANARY_BYTES) != cudaSuccess) return fail(h, EBRL_ERR_CUDA, "cudaMemset of a canary failed");
        h->canaries.push_back({(const char *)*p + padded, what});
    }
    return EBRL_OK;
}

// Compares every canary tail with the pattern; names the first buffer whose tail changed.
ebrl_status_t check_canaries(ebrl_actgen *h)
{
    unsigned char buf[CANARY_BYTES];
    for (const auto &c : h->canaries) {
        if (cudaMemcpy(buf, c.first, CANARY_BYTES, cudaMemcpyDeviceToHost) != cudaSuccess) return fail(h, EBRL_ERR_CUDA, "reading a canary failed");
        for (size_t i = 0; i < CANARY_BYTES; ++i)
            if (buf[i] != CANARY_BYTE) {
                h->sticky = EBRL_ERR_CUDA;
                return fail(h, EBRL_ERR_CUDA, "memory past the end of %s was overwritten (byte %zu of its guard)", c.second, i);
            }
    }
    return EBRL_OK;
}

ebrl_status_t dev_copy_in(ebrl_actgen *h, void **dst, const void *src, size_t bytes)
{
    if (!src) return fail(h, EBRL_ERR_INVALID_ARG, "a weight pointer is NULL");
    ebrl_status_t st = dev_alloc(h, dst, bytes);
    if (st != EBRL_OK) return st;
    CK(cudaMemcpy(*dst, src, bytes, cudaMemcpyDefault));
    return EBRL_OK;
}

// Device buffers (and, on the tensor-core path, TMA descriptors) of one weight set.
ebrl_status_t alloc_weight_set(ebrl_actgen *h, WeightSet &ws)
{
    const ebrl_actgen_cfg_t &c = h->cfg;
    const size_t d = c.d, A = c.A, md = h->md, esz = h->esz;
    ebrl_status_t st;
    void *p = nullptr;
    if ((st = dev_alloc(h, &ws.w_in, d * A * esz)) != EBRL_OK) return st;
    if ((st = dev_alloc(h, &ws.w_out, A * d * esz)) != EBRL_OK) return st;
    if ((st = dev_alloc(h, &p, A * 4)) != EBRL_OK) return st; ws.b_out = (float *)p;
    if ((st = dev_alloc(h, &p, d * 4)) != EBRL_OK) return st; ws.g_final = (float *)p;
    ws.layers.resize(c.n_layers);
    for (LayerDev &o : ws.layers) {
        if ((st = dev_alloc(h, &p, d * 4)) != EBRL_OK) return st; o.g1 = (float *)p;
        if ((st = dev_alloc(h, &p, d * 4)) != EBRL_OK) return st; o.g2 = (float *)p;
        if ((st = dev_alloc(h, &p, d * 4)) != EBRL_OK) return st; o.g3 = (float *)p;
        if ((st = dev_alloc(h, &o.w_qkv, 3 * d * d * esz)) != EBRL_OK) return st;
        if ((st = dev_alloc(h, &o.w_o, d * d * esz)) != EBRL_OK) return st;
        if ((st = dev_alloc(h, &o.w_qc, d * d * esz)) != EBRL_OK) return st;
        if ((st = dev_alloc(h, &o.w_oc, d * d * esz)) != EBRL_OK) return st;
        if ((st = dev_alloc(h, &o.w_1, md * d * esz)) != EBRL_OK) return st;
        if ((st = dev_alloc(h, &o.w_2, d * md * esz)) != EBRL_OK) return st;
        if (c.d_ctx > 0) {
            if ((st = dev_alloc(h, &o.w_kc, d * (size_t)c.d_ctx * esz)) != EBRL_OK) return st;
            if ((st = dev_alloc(h, &o.w_vc, d * (size_t)c.d_ctx * esz)) != EBRL_OK) return st;
            if (h->use_tc) {
                const uint32_t bw = (uint32_t)gemm_tc_box_rows_w();
                if (make_tmap_bf16(&o.t_kc, o.w_kc, (uint64_t)c.d_ctx, d, bw) | make_tmap_bf16(&o.t_vc, o.w_vc, (uint64_t)c.d_ctx, d, bw))
                    return fail(h, EBRL_ERR_CUDA, "cuTensorMapEncodeTiled failed for a weight matrix");
            }
        }
        if (h->use_tc3) {
            const size_t rows_n[6] = {3 * d, d, d, d, md, d}, cols_k[6] = {d, d, d, d, d, md};
            for (int m = 0; m < 6; ++m)
                for (int t = 0; t < 3; ++t) {
                    if ((st = dev_alloc(h, &o.w3[m][t], rows_n[m] * cols_k[m] * 2)) != EBRL_OK) return st;
                    if (make_tmap_bf16(&o.t3[m][t], o.w3[m][t], cols_k[m], rows_n[m], 128))
                        return fail(h, EBRL_ERR_CUDA, "cuTensorMapEncodeTiled failed for a weight matrix");
                }
        }
        if (h->use_tc) {
            const uint32_t bw = (uint32_t)gemm_tc_box_rows_w();
            int bad = make_tmap_bf16(&o.t_qkv, o.w_qkv, d, 3 * d, bw) | make_tmap_bf16(&o.t_o, o.w_o, d, d, bw) |
                      make_tmap_bf16(&o.t_qc, o.w_qc, d, d, bw) | make_tmap_bf16(&o.t_oc, o.w_oc, d, d, bw) |
                      make_tmap_bf16(&o.t_1, o.w_1, d, md, bw) | make_tmap_bf16(&o.t_2, o.w_2, md, d, bw);
            if (bad) return fail(h, EBRL_ERR_CUDA, "cuTensorMapEncodeTiled failed for a weight matrix");
        }
    }
    if (h->fused_ok && c.n_layers > 0) {
        // descriptors and gain pointers refer to the set's buffers, not to their contents: built once per set
        std::vector<FusedLayerTab> tab(c.n_layers);
        for (int l = 0; l < c.n_layers; ++l) {
            const LayerDev &o = ws.layers[l];
            tab[l].t_qkv = o.t_qkv; tab[l].t_o = o.t_o; tab[l].t_qc = o.t_qc; tab[l].t_oc = o.t_oc; tab[l].t_1 = o.t_1; tab[l].t_2 = o.t_2;
            tab[l].g1 = o.g1; tab[l].g2 = o.g2; tab[l].g3 = o.g3;
        }
        if ((st = dev_alloc(h, &p, sizeof(FusedLayerTab) * tab.size())) != EBRL_OK) return st;
        ws.ftab_d = (FusedLayerTab *)p;
        CK(cudaMemcpy(ws.ftab_d, tab.data(), sizeof(FusedLayerTab) * tab.size(), cudaMemcpyHostToDevice));
    }
    if (cudaEventCreateWithFlags(&ws.ready, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ws.last_use, cudaEventDisableTiming) != cudaSuccess)
        return fail(h, EBRL_ERR_CUDA, "cudaEventCreate failed");
    ws.allocated = true;
    return EBRL_OK;
}

// Copies the caller's weights (host or device pointers) into a set, on `st` when async.
ebrl_status_t upload_weight_set(ebrl_actgen *h, WeightSet &ws, const ebrl_actgen_weights_t *wts, cudaStream_t st, bool async)
{
    const ebrl_actgen_cfg_t &c = h->cfg;
    const size_t d = c.d, A = c.A, md = h->md, esz = h->esz;
    if (!wts || !wts->w_in || !wts->w_out || !wts->b_out || !wts->g_final || (c.n_layers > 0 && !wts->layers))
        return fail(h, EBRL_ERR_INVALID_ARG, "a weight pointer is NULL");
    for (int l = 0; l < c.n_layers; ++l) {
        const ebrl_layer_weights_t &w = wts->layers[l];
        if (!w.g1 || !w.g2 || !w.g3 || !w.w_qkv || !w.w_o || !w.w_qc || !w.w_oc || !w.w_1 || !w.w_2)
            return fail(h, EBRL_ERR_INVALID_ARG, "a weight pointer of layer %d is NULL", l);
        if (c.d_ctx > 0 && (!w.w_kc || !w.w_vc))
            return fail(h, EBRL_ERR_INVALID_ARG, "w_kc / w_vc of layer %d is NULL although d_ctx > 0", l);
    }
    auto cp = [&](void *dst, const void *src, size_t bytes) {
        return async ? cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, st) : cudaMemcpy(dst, src, bytes, cudaMemcpyDefault);
    };
    cudaError_t e = cp(ws.w_in, wts->w_in, d * A * esz);
    if (e == cudaSuccess) e = cp(ws.w_out, wts->w_out, A * d * esz);
    if (e == cudaSuccess) e = cp(ws.b_out, wts->b_out, A * 4);
    if (e == cudaSuccess) e = cp(ws.g_final, wts->g_final, d * 4);
    for (int l = 0; l < c.n_layers && e == cudaSuccess; ++l) {
        const ebrl_layer_weights_t &w = wts->layers[l];
        LayerDev &o = ws.layers[l];
        e = cp(o.g1, w.g1, d * 4);
        if (e == cudaSuccess) e = cp(o.g2, w.g2, d * 4);
        if (e == cudaSuccess) e = cp(o.g3, w.g3, d * 4);
        if (e == cudaSuccess) e = cp(o.w_qkv, w.w_qkv, 3 * d * d * esz);
        if (e == cudaSuccess) e = cp(o.w_o, w.w_o, d * d * esz);
        if (e == cudaSuccess) e = cp(o.w_qc, w.w_qc, d * d * esz);
        if (e == cudaSuccess) e = cp(o.w_oc, w.w_oc, d * d * esz);
        if (e == cudaSuccess) e = cp(o.w_1, w.w_1, md * d * esz);
        if (e == cudaSuccess) e = cp(o.w_2, w.w_2, d * md * esz);
        if (e == cudaSuccess && c.d_ctx > 0) e = cp(o.w_kc, w.w_kc, d * (size_t)c.d_ctx * esz);
        if (e == cudaSuccess && c.d_ctx > 0) e = cp(o.w_vc, w.w_vc, d * (size_t)c.d_ctx * esz);
    }
    if (e != cudaSuccess) return fail(h, EBRL_ERR_CUDA, "copying the weights failed: %s", cudaGetErrorString(e));
    if (h->use_tc3) {
        // the three bf16 terms of every matrix, behind the copies on the same stream
        cudaStream_t ss = async ? st : nullptr;
        for (int l = 0; l < c.n_layers && e == cudaSuccess; ++l) {
            LayerDev &o = ws.layers[l];
            const void *src[6] = {o.w_qkv, o.w_o, o.w_qc, o.w_oc, o.w_1, o.w_2};
            const size_t n[6] = {3 * d * d, d * d, d * d, d * d, md * d, d * md};
            for (int m = 0; m < 6 && e == cudaSuccess; ++m)
                e = launch_split3((const float *)src[m], o.w3[m][0], o.w3[m][1], o.w3[m][2], n[m], h->n_sms, ss);
        }
        if (e == cudaSuccess && !async) e = cudaStreamSynchronize(ss);
        if (e != cudaSuccess) return fail(h, EBRL_ERR_CUDA, "splitting the weights failed: %s", cudaGetErrorString(e));
    }
    return EBRL_OK;
}

// Waits for a slot's group and folds its timing into the statistics.
ebrl_status_t retire(ebrl_actgen *h, Slot &s)
{
    if (!s.busy) return EBRL_OK;
    cudaError_t e = cudaEventSynchronize(s.done);
    s.busy = false;
    for (int64_t id : s.ids) h->busy_ids.erase(id);
    s.ids.clear();
    if (e != cudaSuccess) {
        if (h->sticky == EBRL_OK) h->sticky = EBRL_ERR_CUDA;
        return fail(h, EBRL_ERR_CUDA, "group failed: %s", cudaGetErrorString(e));
    }
    for (size_t i = 0; i < s.timed_used; ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, s.timed[i].t0, s.timed[i].t1) == cudaSuccess) {
            h->stats.class_ms[s.timed[i].cls] += ms;
            h->stats.class_launches[s.timed[i].cls] += 1;
            h->stats.class_flops[s.timed[i].cls] += s.timed[i].flops;
            h->stats.class_bytes[s.timed[i].cls] += s.timed[i].bytes;
        }
    }
    s.timed_used = 0;
    return EBRL_OK;
}

// The SM partition of a quota (created on first use, cached per quota); nullptr when the driver has none.
GreenPartition *partition_for(ebrl_actgen *h, int quota)
{
    auto it = h->partitions.find(quota);
    if (it == h->partitions.end()) {
        GreenPartition np;
        if (green_partition_create(h->cfg.device, quota, &np) != 0) np = GreenPartition();
        it = h->partitions.emplace(quota, np).first;
    }
    return it->second.ctx ? &it->second : nullptr;
}

struct Launcher {
    ebrl_actgen *h;
    Slot *slot;
    cudaStream_t st;
    int grid;
    bool timing;
    cudaError_t err = cudaSuccess;

    template <typename F> void run(int cls, double flops, double bytes, F &&f)
    {
        if (err != cudaSuccess) return;
        TimedLaunch *tl = nullptr;
        if (timing) {
            if (slot->timed_used == slot->timed.size()) {
                TimedLaunch n{};
                n.t0 = n.t1 = nullptr;
                if (cudaEventCreate(&n.t0) != cudaSuccess || cudaEventCreate(&n.t1) != cudaSuccess) { err = cudaGetLastError(); return; }
                slot->timed.push_back(n);
            }
            tl = &slot->timed[slot->timed_used++];
            tl->cls = cls; tl->flops = flops; tl->bytes = bytes;
            cudaEventRecord(tl->t0, st);
        }
        err = f();
        h->stats.kernel_launches += 1;
        if (tl) cudaEventRecord(tl->t1, st);
    }
};

// fp32 models: CTA pairs on 256 x 256 tiles or single CTAs on 128 x 128 tiles (bit-identical results).
static bool tc3_use_pairs(const ebrl_actgen *h, int M, int N, int K, int grid)
{
    if (grid < 2 || !gemm_tc3p_supported(N, K)) return false;
    if (h->force_shape == 2) return true;
    if (h->force_shape) return false;
    // rounds x time per round: a 128 x 128 tile takes about 5.5 us at K = 256, a 256 x 256 pair tile about 9.5 us (measured;
    // both scale with K).  Pairs win where a CTA gets several tiles -- small quotas, wide projections.
    const long rows128 = (M + 127) / 128, rows256 = (M + 255) / 256;
    const long r1 = (rows128 * (N / 128) + grid - 1) / grid, rp = (rows256 * (N / 256) + grid / 2 - 1) / (grid / 2);
    return rp * 19 <= r1 * 11;
}

cudaError_t launch_attn(ebrl_actgen *h, const AttnArgs &a, int grid, cudaStream_t st)
{
    if (h->use_attn_mma) return launch_attn_mma(a, grid, h->attn_hpc, h->attn_lookahead, h->wait_ns, h->status_d, st);
    if (h->use_attn_f32) return launch_attn_f32(a, grid, st);
    return launch_attn_simt(a, h->bf16, grid, st);
}

// Tile shape of a tensor-core GEMM by estimated time = waves x tile area / relative efficiency:
// 2 = CTA pairs (256 x 256), 256 = one CTA 128 x 256, 128 = one CTA 128 x 128.  The accumulation
// order per output element is the same for every shape, so the choice does not change a single
// bit of the result.
int pick_tile_shape(const ebrl_actgen *h, long M, int N, int grid)
{
    if (h->force_shape) return h->force_shape;
    const long mt = (M + 127) / 128, mp = (M + 255) / 256, pairs = grid / 2;
    const double t_pair = (h->use_pairs && pairs >= 1) ? (double)((mp * (N / 256) + pairs - 1) / pairs) * 32768.0 / 1.0 : 1e30;
    const double t_256 = (double)((mt * (N / 256) + grid - 1) / grid) * 32768.0 / 0.88;
    const double t_128 = (double)((mt * (N / 128) + grid - 1) / grid) * 16384.0 / 0.72;
    return (t_pair <= t_256 && t_pair <= t_128) ? 2 : (t_256 <= t_128 ? 256 : 128);
}

// Whether a batch of `rows` rows takes the persistent step kernel: the model must be covered, and the batch
// small enough that the per-operation grids would be mostly fill and drain (or the caller forces it).
bool use_fused_path(const ebrl_actgen *h, long rows, int grid)
{
    const ebrl_actgen_cfg_t &c = h->cfg;
    if (!h->fused_ok || (c.flags & (EBRL_FLAG_NO_FUSED | EBRL_FLAG_TEST_PULL)) || c.n_layers < 1 || grid < 1) return false;
    if (c.flags & EBRL_FLAG_FORCE_FUSED) return true;
    return rows <= h->fused_max_rows;
}

// Enqueues every kernel of one batch (the groups coalesced in one slot) on the stream.
cudaError_t enqueue_batch(ebrl_actgen *h, Slot &s, int S, const int32_t *n_active, const double *sum_P_active, int grid,
                          cudaStream_t st)
{
    const ebrl_actgen_cfg_t &c = h->cfg;
    const int d = c.d, H = c.H, L = c.n_layers, md = h->md, bf = h->bf16;
    const int nseg = d / SSQ_W;
    const bool pull = (c.flags & EBRL_FLAG_TEST_PULL) != 0;
    const double esz = (double)h->esz;
    Launcher ln{h, &s, st, grid, (c.flags & EBRL_FLAG_TIMING) != 0};
    const WeightSet &W = h->wset[h->active];
    if (c.d_ctx > 0 && !pull && L > 0) {
        // hidden-state prefixes: gather the batch's hidden rows, then every layer's K and V planes as
        // two dense GEMMs over all of them (once per batch: the planes do not change over the Euler steps)
        const int R = s.prefix_rows, dc = c.d_ctx;
        PackArgs pa{s.meta_d, n_active[0], s.prefix_slices, (int)(dc * h->esz), s.hid_pack};
        ln.run(EBRL_KC_PREFIX, 0.0, 2.0 * R * dc * esz, [&] { return launch_pack_prefix(pa, grid, st); });
        for (int l = 0; l < L; ++l)
            for (int j = 0; j < 2; ++j) {
                const LayerDev &w = W.layers[l];
                GemmArgs g{};
                g.A = s.hid_pack; g.W = j ? w.w_vc : w.w_kc; g.M = R; g.N = d; g.K = dc; g.epi = EPI_SCALE_STORE;
                g.ssq_in = s.ssq; g.n_ssq = 0; g.inv_d = 0.f; g.eps = 1.f;   // row scale 1 / sqrt(0 + 1) = 1: a plain store
                g.C = (char *)s.planes + (size_t)(l * 2 + j) * R * d * h->esz;
                const TensorMap128 &tW = j ? w.t_vc : w.t_kc;
                const double bytes = ((double)R * dc + (double)d * dc + (double)R * d) * esz, flops = 2.0 * R * d * dc;
                if (h->use_tc) {
                    const int shape = pick_tile_shape(h, R, d, grid);
                    if (shape == 2)
                        ln.run(EBRL_KC_PREFIX, flops, bytes, [&] { return launch_gemm_tc2(s.t_hid, tW, g, grid, h->wait_ns, h->status_d, st); });
                    else
                        ln.run(EBRL_KC_PREFIX, flops, bytes, [&] { return launch_gemm_tc(s.t_hid, tW, g, grid, shape, h->wait_ns, h->status_d, st); });
                } else {
                    ln.run(EBRL_KC_PREFIX, flops, bytes, [&] { return launch_gemm_simt(g, bf, grid, st); });
                }
            }
    }
    if (use_fused_path(h, (long)n_active[0] * H, grid) && S > 0 && n_active[0] > 0) {
        // small batch: ONE persistent kernel walks every Euler step
        for (int t = 0; t < c.K_steps; ++t) s.fctl_h[t] = t < S ? n_active[t] : 0;
        if ((ln.err = cudaMemcpyAsync(s.fctl_d, s.fctl_h, sizeof(int) * c.K_steps, cudaMemcpyHostToDevice, st)) != cudaSuccess) return ln.err;
        if ((ln.err = cudaMemsetAsync(s.fctl_d + c.K_steps, 0, sizeof(int) * ((size_t)c.K_steps * s.mt_max + 4 * 256 + 2 * 12 * 4 * 256 + 4 + 4 * 4000), st)) != cudaSuccess) return ln.err;
        FusedArgs f{};
        f.H = H; f.A = c.A; f.d = d; f.md = md; f.n_layers = L; f.n_heads = c.n_heads; f.hd = h->hd;
        f.hpc = h->attn_hpc; f.K = c.K_steps; f.S = S; f.ne0 = n_active[0];
        f.kv_layers = c.kv_layers; f.plane_rows = c.d_ctx > 0 ? s.prefix_rows : 0;
        f.eps = c.rms_eps; f.inv_d = 1.0f / (float)d;
        f.meta = s.meta_d; f.n_active = s.fctl_d; f.done = s.fctl_d + c.K_steps; f.mt_max = s.mt_max;
        f.test_drop_copies = (c.flags & EBRL_FLAG_TEST_DROP_GEMM_COPIES) ? 1 : ((c.flags & EBRL_FLAG_TEST_DROP_ATTN_COPIES) ? 2 : 0);
        f.trace = h->trace ? s.fctl_d + (size_t)c.K_steps * (1 + s.mt_max) : nullptr;
        h->trace_slot = &s;
        f.a_state = s.a_state; f.x = s.x; f.ssq = s.ssq; f.xg = s.xg; f.qkv = s.qkv; f.att = s.att; f.qc = s.qc; f.u = s.u;
        f.maps = s.fmaps_d; f.attn_maps = s.maps_d; f.layers = W.ftab_d;
        f.w_in = W.w_in; f.w_out = W.w_out; f.b_out = W.b_out; f.g_final = W.g_final; f.temb = h->temb;
        double flops = 0.0, bytes = 0.0;
        for (int step = 0; step < S; ++step) {
            const double M = (double)n_active[step] * H;
            flops += L * (M * (12.0 * d * d + 4.0 * d * md) + 4.0 * H * sum_P_active[step] * d + 4.0 * M * H * d) + 4.0 * M * d * c.A;
            bytes += L * (2.0 * sum_P_active[step] * d * esz + (6.0 * d * d + 2.0 * d * md) * esz);   // planes and weights once per layer-step
        }
        ln.run(EBRL_KC_FUSED, flops, bytes, [&] { return launch_fused_steps(f, grid, h->wait_ns, h->status_d, st); });
        return ln.err;
    }
    for (int step = 0; step < S; ++step) {
        const int ne = n_active[step], M = ne * H;
        if (ne == 0) break;
        if (!pull) {
            EmbedArgs ea{s.meta_d, ne, H, c.A, d, step, s.a_state, W.w_in, h->temb,
                         L > 0 ? W.layers[0].g1 : W.g_final, s.x, s.xg, s.ssq};
            if (h->use_tc3) { ea.xg = s.xg3[0]; ea.xg_t1 = s.xg3[1]; ea.xg_t2 = s.xg3[2]; ea.split_xg = 1; }
            ln.run(EBRL_KC_EMBED, 2.0 * M * d * c.A, (double)M * d * (4 + esz), [&] { return launch_embed(ea, bf, grid, st); });
            for (int l = 0; l < L; ++l) {
                const LayerDev &w = W.layers[l];
                auto gemm = [&](const void *A, const TensorMap128 &tA, const void *W, const TensorMap128 &tW, int N, int K, int epi,
                                void *C, const float *gain, const TensorMap128 *w3) {
                    GemmArgs g{};
                    g.A = A; g.W = W; g.M = M; g.N = N; g.K = K; g.epi = epi;
                    g.ssq_in = s.ssq; g.n_ssq = nseg; g.inv_d = 1.0f / (float)d; g.eps = c.rms_eps;
                    g.C = C; g.x = s.x; g.gain = gain; g.xg = s.xg; g.ssq_out = s.ssq;
                    g.test_drop_copies = (c.flags & EBRL_FLAG_TEST_DROP_GEMM_COPIES) ? 1 : 0;
                    const double bytes = ((double)M * K + (double)N * K + (double)M * N) * esz + (epi == EPI_RESID ? 8.0 * M * N : 0.0);
                    if (h->use_tc3) {
                        // the A operand exists as three bf16 term planes (its producer wrote them); the residual epilogue's xg and
                        // the GELU epilogue's C go out as term planes in turn; six tensor-core products per k-slice
                        const TensorMap128 *ta3 = A == s.xg ? s.t_xg3 : (A == s.att ? s.t_att3 : s.t_u3);
                        if (epi == EPI_RESID) { g.xg = s.xg3[0]; g.out_t1 = s.xg3[1]; g.out_t2 = s.xg3[2]; }
                        if (epi == EPI_SCALE_GELU) { g.C = s.u3[0]; g.out_t1 = s.u3[1]; g.out_t2 = s.u3[2]; }
                        if (tc3_use_pairs(h, M, N, K, grid))
                            ln.run(EBRL_KC_GEMM, 2.0 * M * N * K, bytes, [&] { return launch_gemm_tc3p(ta3, w3, g, grid, h->wait_ns, h->status_d, st); });
                        else
                            ln.run(EBRL_KC_GEMM, 2.0 * M * N * K, bytes, [&] { return launch_gemm_tc3(ta3, w3, g, grid, h->wait_ns, h->status_d, st); });
                    } else if (h->use_tc) {
                        const int shape = pick_tile_shape(h, M, N, grid);
                        if (shape == 2)
                            ln.run(EBRL_KC_GEMM, 2.0 * M * N * K, bytes, [&] { return launch_gemm_tc2(tA, tW, g, grid, h->wait_ns, h->status_d, st); });
                        else
                            ln.run(EBRL_KC_GEMM, 2.0 * M * N * K, bytes, [&] { return launch_gemm_tc(tA, tW, g, grid, shape, h->wait_ns, h->status_d, st); });
                    }
                    else
                        ln.run(EBRL_KC_GEMM, 2.0 * M * N * K, bytes, [&] { return launch_gemm_simt(g, bf, grid, st); });
                };
                // self-attention block
                gemm(s.xg, s.t_xg, w.w_qkv, w.t_qkv, 3 * d, d, EPI_SCALE_STORE, s.qkv, nullptr, w.t3[0]);
                {
                    AttnArgs a{};
                    a.q = s.qkv; a.q_stride = 3 * d; a.out = s.att; a.o_stride = d;
                    a.H = H; a.n_heads = c.n_heads; a.hd = h->hd; a.n_envs = ne; a.d = d;
                    a.self = 1;
                    a.test_drop_copies = (c.flags & EBRL_FLAG_TEST_DROP_ATTN_COPIES) ? 1 : 0;
                    a.k_self = (const char *)s.qkv + (size_t)d * h->esz;
                    a.v_self = (const char *)s.qkv + (size_t)2 * d * h->esz;
                    a.kv_stride = 3 * d;
                    a.self_map = s.maps_d; a.kv_maps = s.maps_d + 1;
                    if (h->use_tc3) { a.out = s.att3[0]; a.out_t1 = s.att3[1]; a.out_t2 = s.att3[2]; a.split_out = 1; }
                    ln.run(EBRL_KC_SELF_ATTN, 4.0 * M * H * d, 4.0 * M * d * esz, [&] { return launch_attn(h, a, grid, st); });
                }
                gemm(s.att, s.t_att, w.w_o, w.t_o, d, d, EPI_RESID, nullptr, w.g2, w.t3[1]);
                // cross-attention block
                gemm(s.xg, s.t_xg, w.w_qc, w.t_qc, d, d, EPI_SCALE_STORE, s.qc, nullptr, w.t3[2]);
                {
                    AttnArgs a{};
                    a.q = s.qc; a.q_stride = d; a.out = s.att; a.o_stride = d;
                    a.H = H; a.n_heads = c.n_heads; a.hd = h->hd; a.n_envs = ne; a.d = d;
                    a.meta = s.meta_d; a.kv_plane = (c.kv_layers == 1) ? 0 : l; a.self = 0;
                    a.test_drop_copies = (c.flags & EBRL_FLAG_TEST_DROP_ATTN_COPIES) ? 1 : 0;
                    a.plane_rows = c.d_ctx > 0 ? s.prefix_rows : 0;
                    a.self_map = s.maps_d; a.kv_maps = s.maps_d + 1;
                    if (h->use_tc3) { a.out = s.att3[0]; a.out_t1 = s.att3[1]; a.out_t2 = s.att3[2]; a.split_out = 1; }
                    ln.run(EBRL_KC_CROSS_ATTN, 4.0 * H * sum_P_active[step] * d,
                           2.0 * sum_P_active[step] * d * esz + 2.0 * M * d * esz, [&] { return launch_attn(h, a, grid, st); });
                }
                gemm(s.att, s.t_att, w.w_oc, w.t_oc, d, d, EPI_RESID, nullptr, w.g3, w.t3[3]);
                // MLP block
                gemm(s.xg, s.t_xg, w.w_1, w.t_1, md, d, EPI_SCALE_GELU, s.u, nullptr, w.t3[4]);
                gemm(s.u, s.t_u, w.w_2, w.t_2, d, md, EPI_RESID, nullptr, (l + 1 < L) ? W.layers[l + 1].g1 : W.g_final, w.t3[5]);
            }
        }
        HeadArgs ha{s.meta_d, ne, H, c.A, d, step, c.K_steps, s.a_state, s.x, W.g_final, W.w_out, W.b_out, c.rms_eps, pull ? 1 : 0};
        ln.run(EBRL_KC_HEAD, 2.0 * M * d * c.A, (double)M * d * 4, [&] { return launch_head(ha, bf, grid, st); });
    }
    return ln.err;
}

// Launches the groups waiting in a slot as ONE packed batch: their environments share the row
// space, so weights stream once per step for all of them.  Rows are independent in every
// kernel, hence the result of an environment does not depend on what it is batched with.
ebrl_status_t flush_slot(ebrl_actgen *h, Slot &s)
{
    if (s.pending.empty()) return EBRL_OK;
    const ebrl_actgen_cfg_t &c = h->cfg;
    const int n = (int)s.pending.size();
    cudaStream_t cs = s.stream;
    // the batcher's plan over the whole batch: longest-running environments first
    std::vector<int32_t> order(n);
    for (int i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return s.pending[a].nsteps > s.pending[b].nsteps; });
    std::vector<int32_t> n_active(c.K_steps, 0);
    std::vector<double> sum_P(c.K_steps, 0.0);
    int S = 0;
    std::vector<TensorMap128> maps_packed;
    const bool with_maps = h->use_attn_mma && !(c.flags & EBRL_FLAG_TEST_PULL);
    const bool hidden = c.d_ctx > 0 && !(c.flags & EBRL_FLAG_TEST_PULL) && c.n_layers > 0;
    if (with_maps) maps_packed.resize(n);
    long prefix_rows = 0;
    int longest = 0;
    for (int j = 0; j < n; ++j) {
        const EnvMeta &m = s.pending[order[j]];
        s.meta_h[j] = m;
        if (with_maps && !hidden) maps_packed[j] = s.pending_maps[order[j]];
        if (hidden) { s.meta_h[j].row0 = (int32_t)prefix_rows; prefix_rows += m.P; longest = std::max(longest, (int)m.P); }
        S = std::max(S, (int)m.nsteps);
        for (int t = 0; t < m.nsteps; ++t) { n_active[t] += 1; sum_P[t] += m.P; }
    }
    s.pending.clear();
    s.pending_maps.clear();
    if (hidden) {
        // scratch for the packed hidden rows and the planes projected from them; the slot's previous
        // batch has been retired, so a grow may free the old buffers
        if (prefix_rows > (long)INT32_MAX / (2 * c.n_layers)) return fail(h, EBRL_ERR_UNSUPPORTED, "a batch's prefixes hold too many rows");
        if ((size_t)prefix_rows > s.proj_cap_rows) {
            if (s.hid_pack) cudaFree(s.hid_pack);
            if (s.planes) cudaFree(s.planes);
            s.hid_pack = s.planes = nullptr; s.proj_cap_rows = 0;
            const size_t hb = (size_t)prefix_rows * c.d_ctx * h->esz, pb = (size_t)c.n_layers * 2 * prefix_rows * c.d * h->esz;
            if (cudaMalloc(&s.hid_pack, hb) != cudaSuccess || cudaMalloc(&s.planes, pb) != cudaSuccess) {
                cudaGetLastError();
                if (s.hid_pack) cudaFree(s.hid_pack);
                s.hid_pack = nullptr;
                for (int64_t id : s.ids) h->busy_ids.erase(id);   // the batch is dropped: nothing of it was enqueued
                s.ids.clear(); s.copies_out.clear(); s.groups_pending = 0;
                return fail(h, EBRL_ERR_NOMEM, "projected prefix planes of %ld rows (%zu bytes) do not fit on the device", prefix_rows, hb + pb);
            }
            s.proj_cap_rows = (size_t)prefix_rows;
        }
        s.prefix_rows = (int)prefix_rows;
        s.prefix_slices = (longest + 63) / 64;
        for (int j = 0; j < n; ++j) {
            EnvMeta &m = s.meta_h[j];
            m.hid = m.kv;
            m.kv = (const char *)s.planes + (size_t)m.row0 * c.d * h->esz;
            // the environment's view of the planes: from its first row to the end of the last plane
            if (with_maps && attn_mma_make_map(&maps_packed[j], m.kv, (uint64_t)2 * c.n_layers * prefix_rows - m.row0, c.d, h->attn_hpc, h->hd))
                return fail(h, EBRL_ERR_CUDA, "cuTensorMapEncodeTiled failed for projected prefix planes");
        }
        if (h->use_tc && make_tmap_bf16(&s.t_hid, s.hid_pack, (uint64_t)c.d_ctx, (uint64_t)prefix_rows, (uint32_t)gemm_tc_box_rows_a()))
            return fail(h, EBRL_ERR_CUDA, "cuTensorMapEncodeTiled failed for the packed hidden states");
    }
    // SM partition: the batch runs on the partition's stream, fenced against the caller's stream by events
    cudaStream_t user = cs;
    GreenPartition *gp = nullptr;
    if ((c.flags & EBRL_FLAG_GREEN_CTX) && s.grid < h->n_sms) gp = partition_for(h, s.grid);
    if (gp) {
        CK(cudaEventRecord(s.part_in, user));
        CK(cudaStreamWaitEvent(gp->stream, s.part_in, 0));
        cs = gp->stream;
    }
    h->stats.green_ctx_active = gp ? 1 : 0;
    h->stats.green_ctx_sms = gp ? gp->sm_count : 0;
    WeightSet &wsel = h->wset[h->active];
    if (wsel.version > 1) CK(cudaStreamWaitEvent(cs, wsel.ready, 0));   // a published version: its upload must have landed
    h->stats.weights_version = wsel.version;
    if (s.has_uploads) {   // the batch's kernels wait for the uploads issued on the copy stream
        CK(cudaEventRecord(s.h2d_done, h->copy_stream));
        CK(cudaStreamWaitEvent(cs, s.h2d_done, 0));
        s.has_uploads = false;
        h->host_depth = std::min(2 * h->host_depth, c.max_inflight_groups);
    }
    CK(cudaMemcpyAsync(s.meta_d, s.meta_h, sizeof(EnvMeta) * (size_t)n, cudaMemcpyHostToDevice, cs));
    if (h->use_attn_mma && !(c.flags & EBRL_FLAG_TEST_PULL)) {
        // one TMA descriptor per environment: its planes as a [kv_layers * 2 * P][d] matrix
        // (encoded when the group was submitted, so that the host work overlaps the previous batch)
        for (int j = 0; j < n; ++j) s.maps_h[j] = maps_packed[j];
        CK(cudaMemcpyAsync(s.maps_d + 1, s.maps_h, sizeof(TensorMap128) * (size_t)n, cudaMemcpyHostToDevice, cs));
    }
    pdl_set(h->pdl_allowed && s.grid >= (gp ? gp->sm_count : h->n_sms));
    cudaError_t e = enqueue_batch(h, s, S, n_active.data(), sum_P.data(), s.grid, cs);
    pdl_set(false);
    if (e != cudaSuccess) {
        h->sticky = EBRL_ERR_CUDA;
        return fail(h, EBRL_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
    }
    CK(cudaEventRecord(wsel.last_use, cs));
    wsel.ever_used = true;
    s.wset = h->active;
    if (gp) {
        CK(cudaEventRecord(s.part_out, cs));
        CK(cudaStreamWaitEvent(user, s.part_out, 0));
        cs = user;
    }
    for (const HostCopy &hc : s.copies_out) CK(cudaMemcpyAsync(hc.dst, hc.src, hc.bytes, cudaMemcpyDeviceToHost, cs));
    s.copies_out.clear();
    CK(cudaEventRecord(s.done, cs));
    s.busy = true;
    h->fill = (h->fill + 1) % h->slots.size();
    return EBRL_OK;
}

ebrl_status_t submit_impl(ebrl_actgen *h, int32_t n, const int64_t *env_ids, const void *const *prefix_kv,
                          const float *noise, float *out, int32_t sm_quota, void *stream,
                          const ebrl_submit_ext_t *ext, bool host_buffers,
                          const float *const *noise_ptrs = nullptr, float *const *out_ptrs = nullptr)
{
    if (noise_ptrs || out_ptrs) {   // per-environment state and result pointers instead of two [n][H][A] arrays
        if (!noise_ptrs || !out_ptrs || host_buffers || n < 1) return fail(h, EBRL_ERR_INVALID_ARG, "per-environment pointers: both arrays, device buffers, n >= 1");
        for (int i = 0; i < n; ++i)
            if (!noise_ptrs[i] || !out_ptrs[i] || (((uintptr_t)noise_ptrs[i] | (uintptr_t)out_ptrs[i]) & 3))
                return fail(h, EBRL_ERR_INVALID_ARG, "state or result pointer %d is NULL or not 4-byte aligned", i);
        noise = noise_ptrs[0];   // non-NULL stand-ins for the common checks
        out = out_ptrs[0];
    }
    std::string why;
    ebrl_status_t st = check_submit(&h->cfg, h->n_sms, n, env_ids, prefix_kv, noise, out, sm_quota, ext, &why);
    if (st != EBRL_OK) return fail(h, st, "%s", why.c_str());
    if (n == 0) return EBRL_OK;
    for (int i = 0; i < n; ++i)
        if (h->busy_ids.count(env_ids[i]))
            return fail(h, EBRL_ERR_ENV_BUSY, "env id %lld is in a group that has not been synced", (long long)env_ids[i]);
    if (h->sticky != EBRL_OK) return fail(h, h->sticky, "handle is in a failed state: %s", h->err.c_str());
    CK(cudaSetDevice(h->cfg.device));

    const ebrl_actgen_cfg_t &c = h->cfg;
    cudaStream_t cs = (cudaStream_t)stream;
    const int grid = sm_quota == 0 ? h->n_sms : sm_quota;
    // groups queue in the slot being filled; a group for another stream or quota closes the batch
    if (!h->slots[h->fill].pending.empty() && (h->slots[h->fill].stream != cs || h->slots[h->fill].grid != grid))
        if ((st = flush_slot(h, h->slots[h->fill])) != EBRL_OK) return st;
    Slot &s = h->slots[h->fill];
    if (s.pending.empty()) {
        // bounded queue: a slot is reused only after its previous batch has completed
        if ((st = retire(h, s)) != EBRL_OK) return st;
        s.stream = cs; s.grid = grid; s.groups_pending = 0; s.stage_used = 0; s.chunks_used = 0; s.has_uploads = false;
    }
    const bool pull = (c.flags & EBRL_FLAG_TEST_PULL) != 0;
    const size_t chunk = (size_t)c.H * c.A;
    const int K = c.K_steps;

    // bytes of one environment's prefix as the caller hands it over: its planes, or its hidden states
    auto prefix_bytes = [&](int P) {
        return c.d_ctx > 0 ? (size_t)P * c.d_ctx * h->esz : (size_t)c.kv_layers * 2 * P * c.d * h->esz;
    };
    const float *noise_d = noise;
    float *out_d = out;
    std::vector<const void *> kv_dev(n, nullptr);
    if (host_buffers) {
        // stage planes, noise and out on the device (staging belongs to the slot)
        size_t need = s.stage_used;
        std::vector<size_t> off(n);
        for (int i = 0; i < n; ++i) {
            const int P = (ext && ext->prefix_len) ? ext->prefix_len[i] : c.max_prefix_len;
            off[i] = need;
            need += (prefix_bytes(P) + 255) & ~(size_t)255;
        }
        if (!pull && s.stage_used != 0 && s.kv_stage_bytes < need) {
            // staging already referenced by queued groups: close the batch first, and remember how much
            // a whole batch of such groups would have taken so that the slots grow to it when next empty
            const size_t whole = need / (size_t)(s.groups_pending + 1) * (size_t)c.max_inflight_groups;
            h->stage_hint = std::max(h->stage_hint, std::max(need, whole));
            if ((st = flush_slot(h, s)) != EBRL_OK) return st;
            return submit_impl(h, n, env_ids, prefix_kv, noise, out, sm_quota, stream, ext, host_buffers);
        }
        if (!pull && (s.kv_stage_bytes < need || (s.stage_used == 0 && s.kv_stage_bytes < h->stage_hint))) {   // nothing staged in the slot: grow it
            if (s.kv_stage) cudaFree(s.kv_stage);
            s.kv_stage = nullptr; s.kv_stage_bytes = 0;
            const size_t want = std::max((size_t)c.max_inflight_groups * need, h->stage_hint);   // room for a whole batch of such groups
            cudaError_t e = cudaMalloc((void **)&s.kv_stage, want);
            if (e != cudaSuccess) {
                cudaGetLastError();
                h->stage_hint = 0;
                e = cudaMalloc((void **)&s.kv_stage, need);
                if (e != cudaSuccess) { cudaGetLastError(); return fail(h, EBRL_ERR_NOMEM, "staging of %zu bytes: %s", need, cudaGetErrorString(e)); }
                s.kv_stage_bytes = need;
            } else {
                s.kv_stage_bytes = want;
            }
        }
        if (!s.noise_stage) {
            void *p = nullptr;
            const size_t cap = (size_t)c.max_inflight_groups * c.max_group_envs * chunk * 4;
            if ((st = dev_alloc(h, &p, cap)) != EBRL_OK) return st;
            s.noise_stage = (float *)p;
            if ((st = dev_alloc(h, &p, cap)) != EBRL_OK) return st;
            s.out_stage = (float *)p;
        }
        if (!pull)
            for (int i = 0; i < n; ++i) {
                const int P = (ext && ext->prefix_len) ? ext->prefix_len[i] : c.max_prefix_len;
                CK(cudaMemcpyAsync(s.kv_stage + off[i], prefix_kv[i], prefix_bytes(P), cudaMemcpyHostToDevice, h->copy_stream));
                kv_dev[i] = s.kv_stage + off[i];
            }
        s.stage_used = need;
        noise_d = s.noise_stage + s.chunks_used * chunk;
        out_d = s.out_stage + s.chunks_used * chunk;
        CK(cudaMemcpyAsync((void *)noise_d, noise, (size_t)n * chunk * 4, cudaMemcpyHostToDevice, h->copy_stream));
        s.has_uploads = true;
        s.copies_out.push_back(HostCopy{out, out_d, (size_t)n * chunk * 4});
        s.chunks_used += (size_t)n;
    } else if (!pull) {
        for (int i = 0; i < n; ++i) kv_dev[i] = prefix_kv[i];
    }

    // descriptors of the group's planes first: a failure must leave nothing of the group queued
    std::vector<TensorMap128> group_maps;
    if (h->use_attn_mma && !pull && c.d_ctx == 0) {   // (projected planes get theirs when the batch is launched)
        group_maps.resize(n);
        for (int i = 0; i < n; ++i) {
            const int P = (ext && ext->prefix_len) ? ext->prefix_len[i] : c.max_prefix_len;
            if (attn_mma_make_map(&group_maps[i], kv_dev[i], (uint64_t)c.kv_layers * 2 * P, c.d, h->attn_hpc, h->hd))
                return fail(h, EBRL_ERR_CUDA, "cuTensorMapEncodeTiled failed for the prefix planes of environment %lld", (long long)env_ids[i]);
        }
    }
    uint64_t env_steps = 0;
    for (int i = 0; i < n; ++i) {
        EnvMeta m{};
        m.kv = kv_dev[i];
        m.P = (ext && ext->prefix_len) ? ext->prefix_len[i] : c.max_prefix_len;
        m.k0 = (ext && ext->step_index) ? ext->step_index[i] : 0;
        int ns = K - m.k0;
        if (ext && ext->n_steps > 0 && ext->n_steps < ns) ns = ext->n_steps;
        m.nsteps = ns;
        m.noise = noise_ptrs ? noise_ptrs[i] : noise_d + (size_t)i * chunk;
        m.out = out_ptrs ? out_ptrs[i] : out_d + (size_t)i * chunk;
        s.pending.push_back(m);
        if (!group_maps.empty()) s.pending_maps.push_back(group_maps[i]);
        env_steps += (uint64_t)ns;
        s.ids.push_back(env_ids[i]);
        h->busy_ids.insert(env_ids[i]);
    }
    s.groups_pending += 1;
    h->stats.groups += 1;
    h->stats.envs += (uint64_t)n;
    h->stats.env_steps += env_steps;
    h->stats.granted_sms = grid;
    // Batches of host-staged groups ramp up after a sync (1, 2, 4, ... groups, up to the configured
    // depth): the first uploads are the only ones nothing can hide, so the first batch is kept small
    // and every later batch uploads while the one before it computes.
    const int depth = host_buffers ? std::min(h->host_depth, c.max_inflight_groups) : c.max_inflight_groups;
    if (s.groups_pending >= depth) return flush_slot(h, s);
    return EBRL_OK;
}

void free_all(ebrl_actgen *h)
{
    for (Slot &s : h->slots) {
        if (s.done) cudaEventDestroy(s.done);
        if (s.h2d_done) cudaEventDestroy(s.h2d_done);
        if (s.part_in) cudaEventDestroy(s.part_in);
        if (s.part_out) cudaEventDestroy(s.part_out);
        if (s.meta_h) cudaFreeHost(s.meta_h);
        if (s.maps_h) cudaFreeHost(s.maps_h);
        if (s.fctl_h) cudaFreeHost(s.fctl_h);
        if (s.kv_stage) cudaFree(s.kv_stage);
        if (s.hid_pack) cudaFree(s.hid_pack);
        if (s.planes) cudaFree(s.planes);
        for (TimedLaunch &t : s.timed) { if (t.t0) cudaEventDestroy(t.t0); if (t.t1) cudaEventDestroy(t.t1); }
    }
    for (WeightSet &ws : h->wset) {
        if (ws.ready) cudaEventDestroy(ws.ready);
        if (ws.last_use) cudaEventDestroy(ws.last_use);
        ws.ready = ws.last_use = nullptr;
    }
    for (auto &kv : h->partitions) green_partition_destroy(&kv.second);
    h->partitions.clear();
    if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
    h->copy_stream = nullptr;
    for (void *p : h->owned) cudaFree(p);
    h->owned.clear();
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// exported
// ---------------------------------------------------------------------------------------------
extern "C" {

uint32_t ebrl_actgen_abi_version(void) { return EBRL_ACTGEN_ABI_VERSION; }

int32_t ebrl_actgen_k_steps(ebrl_actgen_t h) { return h ? h->cfg.K_steps : 0; }

uint64_t ebrl_actgen_struct_size(int32_t which)
{
    switch (which) {
    case 0: return sizeof(ebrl_actgen_cfg_t);
    case 1: return sizeof(ebrl_layer_weights_t);
    case 2: return sizeof(ebrl_actgen_weights_t);
    case 3: return sizeof(ebrl_submit_ext_t);
    case 4: return sizeof(ebrl_actgen_stats_t);
    default: return 0;
    }
}

// Host-only checks, exported so that the argument rules can be tested without a device.
ebrl_status_t ebrl_actgen_check_cfg(const ebrl_actgen_cfg_t *cfg)
{
    std::string why;
    ebrl_status_t st = check_cfg(cfg, &why);
    if (st != EBRL_OK) g_create_error = why;
    return st;
}

ebrl_status_t ebrl_actgen_check_submit(const ebrl_actgen_cfg_t *cfg, int32_t n_sms, int32_t n_envs,
                                       const int64_t *env_ids, const void *const *prefix_kv,
                                       const float *noise, const float *out, int32_t sm_quota,
                                       const ebrl_submit_ext_t *ext)
{
    std::string why;
    ebrl_status_t st = check_cfg(cfg, &why);
    if (st == EBRL_OK) st = check_submit(cfg, n_sms, n_envs, env_ids, prefix_kv, noise, out, sm_quota, ext, &why);
    if (st != EBRL_OK) g_create_error = why;
    return st;
}

// The batcher's plan for a group (host only): order[n], nsteps[n], n_active[K]; returns the
// number of inner steps, or -1 on bad arguments.
int32_t ebrl_actgen_plan_group(const ebrl_actgen_cfg_t *cfg, int32_t n_envs, const ebrl_submit_ext_t *ext,
                               int32_t *order, int32_t *nsteps, int32_t *n_active)
{
    if (check_cfg(cfg, nullptr) != EBRL_OK || n_envs < 0 || !order || !nsteps || !n_active) return -1;
    if (ext && ext->step_index)
        for (int i = 0; i < n_envs; ++i)
            if (ext->step_index[i] < 0 || ext->step_index[i] >= cfg->K_steps) return -1;
    return plan_group(cfg, n_envs, ext, order, nsteps, n_active);
}

ebrl_status_t ebrl_actgen_create(const ebrl_actgen_cfg_t *cfg, const ebrl_actgen_weights_t *wts, ebrl_actgen_t *out_handle)
{
    if (!out_handle) return fail(nullptr, EBRL_ERR_INVALID_ARG, "out_handle is NULL");
    *out_handle = nullptr;
    std::string why;
    ebrl_status_t st = check_cfg(cfg, &why);
    if (st != EBRL_OK) return fail(nullptr, st, "%s", why.c_str());
    if (!wts || (cfg->n_layers > 0 && !wts->layers)) return fail(nullptr, EBRL_ERR_INVALID_ARG, "weights is NULL");

    ebrl_actgen *h = new (std::nothrow) ebrl_actgen();
    if (!h) return fail(nullptr, EBRL_ERR_NOMEM, "out of host memory");
    h->cfg = *cfg;
    memset(&h->stats, 0, sizeof h->stats);
    h->bf16 = cfg->param_dtype == EBRL_BF16;
    h->esz = h->bf16 ? 2 : 4;
    h->hd = cfg->d / cfg->n_heads;
    h->md = cfg->mlp_mult * cfg->d;

    auto bail = [&](ebrl_status_t s) {
        g_create_error = h->err;
        free_all(h);
        delete h;
        return s;
    };
    cudaError_t e = cudaSetDevice(cfg->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->n_sms, cudaDevAttrMultiProcessorCount, cfg->device);
    if (e != cudaSuccess) {
        fail(h, EBRL_ERR_CUDA, "no usable CUDA device %d: %s", cfg->device, cudaGetErrorString(e));
        cudaGetLastError();
        return bail(EBRL_ERR_CUDA);
    }
    const int d = cfg->d, A = cfg->A, md = h->md;
    const size_t esz = h->esz;
    h->use_tc = h->bf16 && !(cfg->flags & EBRL_FLAG_FORCE_SIMT) && gemm_tc_supported(d, d) && gemm_tc_supported(md, d) &&
                gemm_tc_supported(d, md) && gemm_tc_supported(3 * d, d);
    if (const char *e2 = getenv("EBRL_GEMM_PAIR")) h->use_pairs = atoi(e2) != 0;
    if (const char *e3 = getenv("EBRL_GEMM_SHAPE")) { const int v = atoi(e3); if (v == 2 || v == 256 || v == 128) h->force_shape = v; }
    if (const char *e4 = getenv("EBRL_PDL")) h->pdl_allowed = atoi(e4) != 0;
    if (const char *e5 = getenv("EBRL_ATTN_LOOKAHEAD")) h->attn_lookahead = std::min(64, std::max(0, atoi(e5)));
    h->use_attn_mma = h->bf16 && !(cfg->flags & EBRL_FLAG_FORCE_SIMT) && attn_mma_supported(cfg->H, cfg->n_heads, h->hd);
    h->use_attn_f32 = !h->bf16 && !(cfg->flags & EBRL_FLAG_FORCE_SIMT) && attn_f32_supported(cfg->H, h->hd);
    h->use_tc3 = !h->bf16 && !(cfg->flags & EBRL_FLAG_FORCE_SIMT) && gemm_tc3_supported(d, d) && gemm_tc3_supported(md, d) &&
                 gemm_tc3_supported(d, md) && gemm_tc3_supported(3 * d, d);
    h->fused_ok = h->use_tc && h->use_attn_mma && fused_supported(cfg->H, cfg->A, d, md, cfg->n_heads, h->hd);
    if (const char *e6 = getenv("EBRL_FUSED_MAX_ROWS")) h->fused_max_rows = atol(e6);
    if (const char *e7 = getenv("EBRL_TRACE")) h->trace = atoi(e7) != 0;
    {   // the attention descriptors are shared with the persistent step kernel, whose slabs are at most 8 heads: wide slabs
        // only on handles that cannot take that path
        const bool fused_may_run = h->fused_ok && !(cfg->flags & EBRL_FLAG_NO_FUSED) &&
                                   ((cfg->flags & EBRL_FLAG_FORCE_FUSED) || h->fused_max_rows > 0);
        h->attn_hpc = attn_mma_slab_heads(cfg->n_heads, h->hd, !fused_may_run);
    }
    if ((st = alloc_weight_set(h, h->wset[0])) != EBRL_OK) return bail(st);
    if ((st = upload_weight_set(h, h->wset[0], wts, nullptr, false)) != EBRL_OK) return bail(st);
    h->wset[0].version = 1;
    {   // timestep-embedding table [K][d], evaluated in double on the host and rounded once
        std::vector<float> t((size_t)cfg->K_steps * d);
        const int half = d / 2;
        for (int k = 0; k < cfg->K_steps; ++k) {
            const double tau = (double)cfg->temb_scale * ((double)k / (double)cfg->K_steps);
            for (int j = 0; j < half; ++j) {
                const double w = std::pow((double)cfg->temb_max_period, -(double)j / (double)half);
                t[(size_t)k * d + j] = (float)std::sin(tau * w);
                t[(size_t)k * d + half + j] = (float)std::cos(tau * w);
            }
        }
        if ((st = dev_copy_in(h, (void **)&h->temb, t.data(), t.size() * 4)) != EBRL_OK) return bail(st);
    }
    // a batch holds up to max_inflight_groups groups; two batch slots let the host queue the
    // next batch while the previous one runs
    const size_t batch_envs = (size_t)cfg->max_inflight_groups * cfg->max_group_envs;
    const size_t rows = batch_envs * cfg->H;
    h->wait_ns = cfg->wait_limit_ns ? cfg->wait_limit_ns : 4000000000ull;
    {
        void *p = nullptr;
        if ((st = dev_alloc(h, &p, 16)) != EBRL_OK) return bail(st);
        h->status_d = (int *)p;
        if (cudaMemset(h->status_d, 0, 16) != cudaSuccess) { fail(h, EBRL_ERR_CUDA, "cudaMemset failed"); return bail(EBRL_ERR_CUDA); }
    }
    if (cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking) != cudaSuccess) {
        fail(h, EBRL_ERR_CUDA, "cudaStreamCreate failed");
        return bail(EBRL_ERR_CUDA);
    }
    h->slots.resize(2);
    for (Slot &s : h->slots) {
        void *p = nullptr;
        if ((st = dev_alloc(h, &p, rows * A * 4, "the action-state workspace")) != EBRL_OK) return bail(st); s.a_state = (float *)p;
        if ((st = dev_alloc(h, &p, rows * d * 4, "the residual-stream workspace x")) != EBRL_OK) return bail(st); s.x = (float *)p;
        if ((st = dev_alloc(h, &p, rows * (d / SSQ_W) * 4, "the sum-of-squares workspace")) != EBRL_OK) return bail(st); s.ssq = (float *)p;
        if ((st = dev_alloc(h, &s.xg, rows * d * esz, "the workspace xg")) != EBRL_OK) return bail(st);
        if ((st = dev_alloc(h, &s.qkv, rows * 3 * d * esz, "the workspace qkv")) != EBRL_OK) return bail(st);
        if ((st = dev_alloc(h, &s.att, rows * d * esz, "the workspace att")) != EBRL_OK) return bail(st);
        if ((st = dev_alloc(h, &s.qc, rows * d * esz, "the workspace qc")) != EBRL_OK) return bail(st);
        if ((st = dev_alloc(h, &s.u, rows * md * esz, "the workspace u")) != EBRL_OK) return bail(st);
        if ((st = dev_alloc(h, &p, sizeof(EnvMeta) * batch_envs)) != EBRL_OK) return bail(st); s.meta_d = (EnvMeta *)p;
        if (cudaMallocHost((void **)&s.meta_h, sizeof(EnvMeta) * batch_envs) != cudaSuccess) {
            cudaGetLastError();
            fail(h, EBRL_ERR_NOMEM, "pinned staging allocation failed");
            return bail(EBRL_ERR_NOMEM);
        }
        // stale workspace rows are read (never stored) as padding of tiles and boxes: keep them finite
        if (cudaMemset(s.x, 0, rows * d * 4) != cudaSuccess || cudaMemset(s.xg, 0, rows * d * esz) != cudaSuccess ||
            cudaMemset(s.qkv, 0, rows * 3 * d * esz) != cudaSuccess || cudaMemset(s.att, 0, rows * d * esz) != cudaSuccess ||
            cudaMemset(s.qc, 0, rows * d * esz) != cudaSuccess || cudaMemset(s.u, 0, rows * md * esz) != cudaSuccess ||
            cudaMemset(s.ssq, 0, rows * (d / SSQ_W) * 4) != cudaSuccess) {
            fail(h, EBRL_ERR_CUDA, "cudaMemset of the workspace failed");
            return bail(EBRL_ERR_CUDA);
        }
        if (h->use_attn_mma) {
            if ((st = dev_alloc(h, &p, sizeof(TensorMap128) * (batch_envs + 1))) != EBRL_OK) return bail(st);
            s.maps_d = (TensorMap128 *)p;
            if (cudaMallocHost((void **)&s.maps_h, sizeof(TensorMap128) * batch_envs) != cudaSuccess) {
                cudaGetLastError();
                fail(h, EBRL_ERR_NOMEM, "pinned staging allocation failed");
                return bail(EBRL_ERR_NOMEM);
            }
            TensorMap128 self_map;
            if (attn_mma_make_map(&self_map, s.qkv, rows, 3 * (uint64_t)d, h->attn_hpc, h->hd) ||
                cudaMemcpy(s.maps_d, &self_map, sizeof self_map, cudaMemcpyHostToDevice) != cudaSuccess) {
                fail(h, EBRL_ERR_CUDA, "building the TMA descriptor of the QKV buffer failed");
                return bail(EBRL_ERR_CUDA);
            }
        }
        if (h->use_tc) {
            // the row extent is the workspace capacity: rows past a group's M hold stale data
            // that only ever reaches output rows that are never stored (rows are independent)
            const uint32_t ba = (uint32_t)gemm_tc_box_rows_a();
            int bad = make_tmap_bf16(&s.t_xg, s.xg, d, rows, ba) | make_tmap_bf16(&s.t_att, s.att, d, rows, ba) |
                      make_tmap_bf16(&s.t_u, s.u, md, rows, ba);
            if (bad) { fail(h, EBRL_ERR_CUDA, "cuTensorMapEncodeTiled failed for a workspace"); return bail(EBRL_ERR_CUDA); }
        }
        if (h->use_tc3) {
            for (int t = 0; t < 3; ++t) {
                void **bufs[3] = {&s.xg3[t], &s.att3[t], &s.u3[t]};
                TensorMap128 *maps[3] = {&s.t_xg3[t], &s.t_att3[t], &s.t_u3[t]};
                const size_t width[3] = {(size_t)d, (size_t)d, (size_t)md};
                for (int b = 0; b < 3; ++b) {
                    if ((st = dev_alloc(h, bufs[b], rows * width[b] * 2, "a split-operand workspace")) != EBRL_OK) return bail(st);
                    if (cudaMemset(*bufs[b], 0, rows * width[b] * 2) != cudaSuccess) { fail(h, EBRL_ERR_CUDA, "cudaMemset of the workspace failed"); return bail(EBRL_ERR_CUDA); }
                    if (make_tmap_bf16(maps[b], *bufs[b], width[b], rows, 128)) {
                        fail(h, EBRL_ERR_CUDA, "cuTensorMapEncodeTiled failed for a workspace");
                        return bail(EBRL_ERR_CUDA);
                    }
                }
            }
        }
        if (h->fused_ok) {
            FusedMaps fm;
            fm.a_xg = s.t_xg; fm.a_att = s.t_att; fm.a_u = s.t_u;
            int bad = make_tmap_bf16(&fm.c_qkv, s.qkv, 3 * (uint64_t)d, rows, 32) | make_tmap_bf16(&fm.c_qc, s.qc, d, rows, 32) |
                      make_tmap_bf16(&fm.c_u, s.u, md, rows, 32);
            if (bad) { fail(h, EBRL_ERR_CUDA, "cuTensorMapEncodeTiled failed for a workspace"); return bail(EBRL_ERR_CUDA); }
            if ((st = dev_alloc(h, &p, sizeof fm)) != EBRL_OK) return bail(st);
            s.fmaps_d = (FusedMaps *)p;
            if (cudaMemcpy(s.fmaps_d, &fm, sizeof fm, cudaMemcpyHostToDevice) != cudaSuccess) { fail(h, EBRL_ERR_CUDA, "cudaMemcpy failed"); return bail(EBRL_ERR_CUDA); }
            s.mt_max = (int)((rows + 127) / 128);
            if ((st = dev_alloc(h, &p, sizeof(int) * ((size_t)cfg->K_steps * (1 + s.mt_max) + 4 * 256 + 2 * 12 * 4 * 256 + 4 + 4 * 4000))) != EBRL_OK) return bail(st);
            s.fctl_d = (int *)p;
            if (cudaMallocHost((void **)&s.fctl_h, sizeof(int) * (size_t)cfg->K_steps) != cudaSuccess) {
                cudaGetLastError();
                fail(h, EBRL_ERR_NOMEM, "pinned staging allocation failed");
                return bail(EBRL_ERR_NOMEM);
            }
        }
        if (cudaEventCreateWithFlags(&s.part_in, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&s.part_out, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&s.h2d_done, cudaEventDisableTiming) != cudaSuccess) {
            fail(h, EBRL_ERR_CUDA, "cudaEventCreate failed");
            return bail(EBRL_ERR_CUDA);
        }
        if (cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming) != cudaSuccess) {
            fail(h, EBRL_ERR_CUDA, "cudaEventCreate failed");
            return bail(EBRL_ERR_CUDA);
        }
    }
    *out_handle = h;
    return EBRL_OK;
}

ebrl_status_t ebrl_actgen_submit(ebrl_actgen_t h, int32_t n, const int64_t *env_ids, const void *const *prefix_kv,
                                 const float *noise, float *out, int32_t sm_quota, void *stream, const ebrl_submit_ext_t *ext)
{
    if (!h) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(h->mu);
    return submit_impl(h, n, env_ids, prefix_kv, noise, out, sm_quota, stream, ext, false);
}

ebrl_status_t ebrl_actgen_submit_scattered(ebrl_actgen_t h, int32_t n, const int64_t *env_ids, const void *const *prefix_kv,
                                           const float *const *state_ptrs, float *const *out_ptrs, int32_t sm_quota, void *stream,
                                           const ebrl_submit_ext_t *ext)
{
    if (!h) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(h->mu);
    if (n == 0) return EBRL_OK;
    if (n < 0 || !state_ptrs || !out_ptrs) return fail(h, EBRL_ERR_INVALID_ARG, "n_envs < 0, or state_ptrs / out_ptrs is NULL");
    return submit_impl(h, n, env_ids, prefix_kv, nullptr, nullptr, sm_quota, stream, ext, false, state_ptrs, out_ptrs);
}

ebrl_status_t ebrl_actgen_submit_host(ebrl_actgen_t h, int32_t n, const int64_t *env_ids, const void *const *prefix_kv_host,
                                      const float *noise_host, float *out_host, int32_t sm_quota, void *stream,
                                      const ebrl_submit_ext_t *ext)
{
    if (!h) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(h->mu);
    return submit_impl(h, n, env_ids, prefix_kv_host, noise_host, out_host, sm_quota, stream, ext, true);
}

ebrl_status_t ebrl_actgen_flush(ebrl_actgen_t h)
{
    if (!h) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(h->mu);
    if (cudaSetDevice(h->cfg.device) != cudaSuccess) return fail(h, EBRL_ERR_CUDA, "cudaSetDevice failed");
    return flush_slot(h, h->slots[h->fill]);
}

ebrl_status_t ebrl_actgen_sync(ebrl_actgen_t h)
{
    if (!h) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(h->mu);
    if (cudaSetDevice(h->cfg.device) != cudaSuccess) return fail(h, EBRL_ERR_CUDA, "cudaSetDevice failed");
    ebrl_status_t first = flush_slot(h, h->slots[h->fill]);
    for (size_t i = 0; i < h->slots.size(); ++i) {
        Slot &s = h->slots[(h->fill + i) % h->slots.size()];
        ebrl_status_t st = retire(h, s);
        if (st != EBRL_OK && first == EBRL_OK) first = st;
    }
    h->host_depth = 1;
    if (first == EBRL_OK && !h->canaries.empty()) first = check_canaries(h);
    if (first == EBRL_OK && h->status_d) {
        int word[4] = {0, 0, 0, 0};   // [0] status; [1..3] where the first wait gave up (persistent step kernel): site/kind/step, task, detail
        if (cudaMemcpy(word, h->status_d, sizeof word, cudaMemcpyDeviceToHost) == cudaSuccess && word[0] != 0) {
            h->sticky = (ebrl_status_t)word[0];
            if (word[1] != 0 && h->trace && h->trace_slot) {
                std::vector<int> tr(4 * 256), ctr((size_t)h->cfg.K_steps * h->trace_slot->mt_max);
                const Slot &ts = *h->trace_slot;
                if (cudaMemcpy(tr.data(), ts.fctl_d + (size_t)h->cfg.K_steps * (1 + ts.mt_max), tr.size() * 4, cudaMemcpyDeviceToHost) == cudaSuccess &&
                    cudaMemcpy(ctr.data(), ts.fctl_d + h->cfg.K_steps, ctr.size() * 4, cudaMemcpyDeviceToHost) == cudaSuccess) {
                    fprintf(stderr, "[ebrl trace] cta: producer mma workers0 workers1  (task<<4 | kind<<2 | self)\n");
                    for (int cta = 0; cta < 256; ++cta)
                        if (tr[4 * cta] | tr[4 * cta + 1] | tr[4 * cta + 2] | tr[4 * cta + 3])
                            fprintf(stderr, "[ebrl trace] %3d: %d/%d %d/%d %d/%d %d/%d\n", cta, tr[4 * cta] >> 4, tr[4 * cta] & 15, tr[4 * cta + 1] >> 4,
                                    tr[4 * cta + 1] & 15, tr[4 * cta + 2] >> 4, tr[4 * cta + 2] & 15, tr[4 * cta + 3] >> 4, tr[4 * cta + 3] & 15);
                    fprintf(stderr, "[ebrl trace] counters of inner step 0:");
                    for (int m = 0; m < ts.mt_max && m < 32; ++m) fprintf(stderr, " %d", ctr[m]);
                    fprintf(stderr, "\n");
                }
            }
            if (word[1] != 0)
                fail(h, h->sticky, "a device-side wait ran out of time (status %d; site %d, operation kind %d, inner step %d, task %d, detail 0x%x)",
                     word[0], word[1] & 0xff, (word[1] >> 8) & 0xf, (word[1] >> 12) & 0xffff, word[2], (unsigned)word[3]);
            else
                fail(h, h->sticky, "a device-side wait ran out of time (status %d)", word[0]);
        }
    }
    if (first == EBRL_OK && h->sticky != EBRL_OK) first = h->sticky;
    return first;
}

ebrl_status_t ebrl_actgen_destroy(ebrl_actgen_t h)
{
    if (!h) return EBRL_OK;
    ebrl_status_t st;
    {
        std::lock_guard<std::mutex> lk(h->mu);
        cudaSetDevice(h->cfg.device);
        st = flush_slot(h, h->slots[h->fill]);
        for (Slot &s : h->slots) { ebrl_status_t r = retire(h, s); if (r != EBRL_OK && st == EBRL_OK) st = r; }
        free_all(h);
    }
    delete h;
    return st;
}

const char *ebrl_actgen_last_error(ebrl_actgen_t h) { return h ? h->err.c_str() : g_create_error.c_str(); }

ebrl_status_t ebrl_actgen_get_stats(ebrl_actgen_t h, ebrl_actgen_stats_t *out)
{
    if (!h || !out) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(h->mu);
    *out = h->stats;
    return EBRL_OK;
}

ebrl_status_t ebrl_actgen_reset_stats(ebrl_actgen_t h)
{
    if (!h) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(h->mu);
    const int32_t g = h->stats.granted_sms, gc = h->stats.green_ctx_active, gs = h->stats.green_ctx_sms;
    const uint64_t wv = h->stats.weights_version;
    memset(&h->stats, 0, sizeof h->stats);
    h->stats.weights_version = wv;
    h->stats.granted_sms = g; h->stats.green_ctx_active = gc; h->stats.green_ctx_sms = gs;
    return EBRL_OK;
}

ebrl_status_t ebrl_actgen_update_weights(ebrl_actgen_t h, const ebrl_actgen_weights_t *weights, void *stream, uint64_t *out_version)
{
    if (!h) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(h->mu);
    if (h->sticky != EBRL_OK) return fail(h, h->sticky, "handle is in a failed state: %s", h->err.c_str());
    CK(cudaSetDevice(h->cfg.device));
    // groups queued so far were submitted under the current version: launch them with it
    ebrl_status_t st = flush_slot(h, h->slots[h->fill]);
    if (st != EBRL_OK) return st;
    WeightSet &t = h->wset[1 - h->active];
    if (!t.allocated && (st = alloc_weight_set(h, t)) != EBRL_OK) return st;
    cudaStream_t cs = (cudaStream_t)stream;
    // Batches still reading the set being replaced: the upload waits for every one of them on the device.  last_use
    // covers the most recent batch; batches in flight on other streams (two slots, partition streams) have their
    // own completion events.
    if (t.ever_used) CK(cudaStreamWaitEvent(cs, t.last_use, 0));
    for (Slot &sl : h->slots)
        if (sl.busy && sl.wset == 1 - h->active) CK(cudaStreamWaitEvent(cs, sl.done, 0));
    if ((st = upload_weight_set(h, t, weights, cs, true)) != EBRL_OK) return st;
    CK(cudaEventRecord(t.ready, cs));
    h->active = 1 - h->active;
    t.version = ++h->version;
    if (out_version) *out_version = t.version;
    return EBRL_OK;
}

uint64_t ebrl_actgen_weights_version(ebrl_actgen_t h)
{
    if (!h) return 0;
    std::lock_guard<std::mutex> lk(h->mu);
    return h->version;
}

ebrl_status_t ebrl_actgen_partition_info(ebrl_actgen_t h, int32_t sm_quota, int32_t *out_gen_sms, int32_t *out_rest_sms, void **out_rest_stream)
{
    if (!h) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(h->mu);
    if (out_gen_sms) *out_gen_sms = 0;
    if (out_rest_sms) *out_rest_sms = 0;
    if (out_rest_stream) *out_rest_stream = nullptr;
    if (sm_quota < 1 || sm_quota > h->n_sms) return fail(h, EBRL_ERR_QUOTA, "sm_quota outside 1..#SMs");
    if (!(h->cfg.flags & EBRL_FLAG_GREEN_CTX) || sm_quota >= h->n_sms) return EBRL_OK;   // no partition is used for such submits
    CK(cudaSetDevice(h->cfg.device));
    const GreenPartition *gp = partition_for(h, sm_quota);
    if (!gp) return EBRL_OK;
    if (out_gen_sms) *out_gen_sms = gp->sm_count;
    if (out_rest_sms) *out_rest_sms = gp->rest_sm_count;
    if (out_rest_stream) *out_rest_stream = (void *)gp->rest_stream;
    return EBRL_OK;
}

#ifdef EBRL_FUSED_PROF
// tuning builds only: the persistent kernel's event log of the last launch (read by fused_timeline.py)
ebrl_status_t ebrl_actgen_debug_events(ebrl_actgen_t h, long long *out, int32_t n_events, int32_t *count)
{
    if (!h || !out || !h->trace_slot) return EBRL_ERR_INVALID_ARG;
    const Slot &ts = *h->trace_slot;
    const int *base = ts.fctl_d + (size_t)h->cfg.K_steps * (1 + ts.mt_max) + 4 * 256 + 2 * 12 * 4 * 256;
    if (cudaMemcpy(count, base, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return EBRL_ERR_CUDA;
    return cudaMemcpy(out, base + 4, sizeof(long long) * 2 * (size_t)n_events, cudaMemcpyDeviceToHost) == cudaSuccess ? EBRL_OK : EBRL_ERR_CUDA;
}
#endif

ebrl_status_t ebrl_actgen_set_timing(ebrl_actgen_t h, int32_t on)
{
    if (!h) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(h->mu);
    if (on) h->cfg.flags |= EBRL_FLAG_TIMING; else h->cfg.flags &= ~EBRL_FLAG_TIMING;
    return EBRL_OK;
}

}  // extern "C"
