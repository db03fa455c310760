/*
 * ebrl_actgen -- batched action generation for independently progressing environments on one
 * NVIDIA B200 (sm_100a), behind a C ABI.
 *
 * The operation (paper section 2.1): a diffusion-style action head turns a random tensor into
 * an action chunk over several denoising steps, conditioned on a representation the backbone
 * has cached (here: per-environment prefix K/V planes).  Environments are independent and are
 * served in groups (section 4.2.2); generation runs under an SM quota smaller than the chip
 * so that other stages can share the GPU (sections 4.2.1 and 4.3.1).
 *
 * Per environment e, with action state a in R^{H x A}, prefix planes Kc, Vc in R^{P_e x d} and
 * step index k_e, the library computes, for k = k_e .. k_end-1 (t_k = k/K):
 *
 *     x_h   = W_in a_h + temb(t_k)                                   (h = 0..H-1)
 *     for each layer l:
 *         [q|k|v] = W_qkv RMSNorm(x; g1);  x += W_o  concat_heads softmax(q k^T / sqrt(hd)) v
 *         qc      = W_qc  RMSNorm(x; g2);  x += W_oc concat_heads softmax(qc Kc^T / sqrt(hd)) Vc
 *         x      += W_2 GELU(W_1 RMSNorm(x; g3))                      (GELU in its erf form)
 *     v     = W_out RMSNorm(x; g_final) + b_out
 *     a    += v / K                                                   (explicit Euler)
 *
 *     (variant cfg.d_ctx > 0, the prefix given as hidden states h in R^{P_e x d_ctx}: layer l uses
 *      Kc = h W_kc_l^T, Vc = h W_vc_l^T, computed once per batch and stored in kv_dtype)
 *
 *     temb(t)_j = sin(temb_scale * t * w_j), temb(t)_{d/2+j} = cos(temb_scale * t * w_j),
 *     w_j = temb_max_period^(-j/(d/2));   RMSNorm(x; g)_j = g_j x_j / sqrt(mean(x^2) + rms_eps).
 *
 * Matrices are row-major [out][in] (y = W x).  Accumulation is always fp32; the action state,
 * gains and b_out are fp32; matrices and prefix planes are fp32 or bf16 (param_dtype/kv_dtype).
 *
 * The result for an environment is a pure function of (weights, its planes, its state, its
 * step index, the step count): it does not depend on environment ids, on which group the
 * environment arrives in, on the order inside the group, or on the SM quota.  Results are
 * bit-identical across those choices.
 *
 * Error behaviour: every call returns a status; nothing throws, aborts or traps across this
 * boundary.  Invalid arguments are detected before anything is enqueued.  Asynchronous
 * failures (a CUDA error, a bounded device-side wait that ran out) are sticky and are returned
 * by ebrl_actgen_sync.  There is no CPU fallback: without a usable CUDA device the calls fail.
 */
#ifndef EBRL_ACTGEN_H_
#define EBRL_ACTGEN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define EBRL_ACTGEN_ABI_VERSION 3u

typedef struct ebrl_actgen *ebrl_actgen_t;

typedef enum {
    EBRL_OK = 0,
    EBRL_ERR_INVALID_ARG = 1,   /* bad pointer, size, dtype, step index, duplicate env id ...   */
    EBRL_ERR_UNSUPPORTED = 2,   /* valid but outside what the kernels cover (see create)        */
    EBRL_ERR_NOMEM = 3,         /* host or device allocation failed                             */
    EBRL_ERR_CUDA = 4,          /* a CUDA call or kernel failed; text in last_error             */
    EBRL_ERR_ENV_BUSY = 5,      /* an env id of this group is in a group not yet synced         */
    EBRL_ERR_QUOTA = 6,         /* sm_quota outside 0..#SMs                                     */
    EBRL_ERR_TIMEOUT = 7        /* a bounded device-side wait gave up                           */
} ebrl_status_t;

typedef enum { EBRL_F32 = 0, EBRL_BF16 = 1 } ebrl_dtype_t;

/* cfg.flags */
#define EBRL_FLAG_TEST_PULL   1u  /* replace the network by v = b_out - a (integrator check)    */
#define EBRL_FLAG_GREEN_CTX   2u  /* run each batch inside an SM partition (green context) of at
                                     least sm_quota SMs when the driver offers one; the grid cap
                                     of sm_quota CTAs applies either way                         */
#define EBRL_FLAG_TIMING      4u  /* record per-kernel-class device time (see get_stats)        */
#define EBRL_FLAG_FORCE_SIMT  8u  /* use the plain-ALU kernels, not tensor cores (bf16 models: for
                                     every operation; fp32 models: for the projections, which
                                     otherwise run on the tensor cores as six bf16 products per
                                     term pair of three-term operand splits, fp32-accurate)       */
#define EBRL_FLAG_NO_FUSED   16u  /* never use the persistent step kernel (one resident grid that
                                     walks all Euler steps of a small batch); always launch one
                                     kernel per operation                                        */
#define EBRL_FLAG_FORCE_FUSED 32u /* use the persistent step kernel for every batch the kernel
                                     covers (bf16 tensor-core models with H a divisor of 128 and
                                     A <= 16), whatever its size.  Without the flag no batch takes
                                     it: it delivers the same bits as the per-operation kernels
                                     but has measured slower on B200 at every batch size tried;
                                     EBRL_FUSED_MAX_ROWS=<rows> in the environment at create makes
                                     batches of up to that many rows take it                    */

#define EBRL_FLAG_TEST_DROP_GEMM_COPIES 64u   /* tests of the give-up path only: the copy-issuing threads of
                                     the projection kernels issue nothing, so every consumer's bounded
                                     wait (cfg.wait_limit_ns) runs out and ebrl_actgen_sync returns
                                     EBRL_ERR_TIMEOUT; the kernels return normally, the context stays usable */
#define EBRL_FLAG_TEST_DROP_ATTN_COPIES 128u  /* the same for the tensor-core attention kernels                */
#define EBRL_FLAG_DEBUG_CANARY 256u /* every device buffer the handle allocates at create gets a guard of
                                     256 pattern bytes behind it; ebrl_actgen_sync checks the guards and
                                     returns EBRL_ERR_CUDA naming the buffer when one was overwritten      */

/* Plain data, copied at create. */
typedef struct {
    uint32_t abi_version;        /* EBRL_ACTGEN_ABI_VERSION                                     */
    int32_t H, A, d;             /* action tokens, action dims, model width                     */
    int32_t n_layers, n_heads;   /* head_dim = d / n_heads                                      */
    int32_t mlp_mult;            /* MLP hidden width = mlp_mult * d                             */
    int32_t K_steps;             /* Euler steps from t = 0 to t = 1                             */
    int32_t max_prefix_len;      /* upper bound on any P_e                                      */
    int32_t max_group_envs;      /* upper bound on n_envs of one submit                         */
    int32_t max_inflight_groups; /* groups that may be submitted before a sync (>= 1)           */
    int32_t param_dtype;         /* ebrl_dtype_t of the matrices                                */
    int32_t kv_dtype;            /* ebrl_dtype_t of the prefix planes                           */
    int32_t kv_layers;           /* 1: one K/V plane pair for all layers; n_layers: per layer   */
    float rms_eps;               /* 1e-6                                                        */
    float temb_scale;            /* 1000                                                        */
    float temb_max_period;       /* 10000                                                       */
    uint32_t flags;              /* EBRL_FLAG_*                                                 */
    int32_t device;              /* CUDA device ordinal                                         */
    uint64_t wait_limit_ns;      /* bound for device-side waits; 0 = default                    */
    int32_t d_ctx;               /* 0: prefix_kv[i] holds the cached K/V planes themselves.
                                    > 0: prefix_kv[i] holds the backbone's hidden states
                                    [P_e][d_ctx] (kv_dtype) and every layer projects its own
                                    planes Kc = h W_kc^T, Vc = h W_vc^T once per batch, before
                                    the first Euler step; needs kv_layers == n_layers         */
    int32_t reserved_;
} ebrl_actgen_cfg_t;

typedef struct {
    const float *g1, *g2, *g3;   /* [d] fp32 RMSNorm gains                                      */
    const void *w_qkv;           /* [3d][d]: rows 0..d-1 Q, d..2d-1 K, 2d..3d-1 V;
                                    head h = rows h*hd..(h+1)*hd-1 of each third               */
    const void *w_o;             /* [d][d]   self-attention output projection                   */
    const void *w_qc;            /* [d][d]   cross-attention query projection                   */
    const void *w_oc;            /* [d][d]   cross-attention output projection                  */
    const void *w_1;             /* [mlp_mult*d][d]                                             */
    const void *w_2;             /* [d][mlp_mult*d]                                             */
    const void *w_kc;            /* [d][d_ctx] cross-attention key projection of the prefix's
                                    hidden states; read only when cfg.d_ctx > 0, else NULL     */
    const void *w_vc;            /* [d][d_ctx] value projection, likewise                       */
} ebrl_layer_weights_t;

/* Pointers may be host or device memory; everything is copied to the device at create and the
 * caller's buffers are not referenced afterwards. */
typedef struct {
    const void *w_in;            /* [d][A] param_dtype                                          */
    const void *w_out;           /* [A][d] param_dtype                                          */
    const float *b_out;          /* [A] fp32                                                    */
    const float *g_final;        /* [d] fp32                                                    */
    const ebrl_layer_weights_t *layers;   /* [n_layers]                                         */
} ebrl_actgen_weights_t;

/* Optional per-submit extension; NULL means the defaults. */
typedef struct {
    const int32_t *prefix_len;   /* host [n]; NULL: every P_e = cfg.max_prefix_len              */
    const int32_t *step_index;   /* host [n], k_e in [0, K); NULL: all 0                        */
    int32_t n_steps;             /* 0: run every env to step K; s > 0: advance by min(s, K-k_e) */
} ebrl_submit_ext_t;

/* Kernel classes of the per-class timing (EBRL_FLAG_TIMING). */
enum { EBRL_KC_EMBED = 0, EBRL_KC_GEMM = 1, EBRL_KC_SELF_ATTN = 2, EBRL_KC_CROSS_ATTN = 3,
       EBRL_KC_HEAD = 4, EBRL_KC_PREFIX = 5 /* packing and projecting hidden-state prefixes */,
       EBRL_KC_FUSED = 6 /* the persistent step kernel: every operation of every Euler step */,
       EBRL_KC_COUNT = 7 };

typedef struct {
    uint64_t groups, envs, env_steps;     /* submitted since create                            */
    uint64_t kernel_launches;             /* kernels of this library launched since create     */
    int32_t granted_sms;                  /* SMs of the last submit's quota actually used:
                                             CTAs of the persistent grids, or the green
                                             context's SM count when one is active             */
    int32_t green_ctx_active;             /* 1 if the last batch ran inside a green context    */
    int32_t green_ctx_sms;                /* SMs in that context's partition (the driver rounds
                                             the quota up to its granularity), else 0          */
    int32_t reserved_;
    double class_ms[EBRL_KC_COUNT];       /* device time per kernel class (EBRL_FLAG_TIMING),
                                             accumulated over synced groups                    */
    uint64_t class_launches[EBRL_KC_COUNT];
    double class_flops[EBRL_KC_COUNT];    /* algorithmic 2*m*n*k FLOPs of those launches       */
    double class_bytes[EBRL_KC_COUNT];    /* algorithmic bytes of those launches               */
    uint64_t weights_version;             /* policy version the last launched batch ran with   */
} ebrl_actgen_stats_t;

/* A generation worker for one policy (section 2.1: the action head that denoises a random tensor
 * into an action chunk; section 4.2.1: generation is a stage of its own with its own resources).
 * Validates cfg, copies the weights to the device (re-laid-out as the kernels want), builds
 * the timestep-embedding table, allocates max_inflight_groups workspaces of
 * max_group_envs * H rows.  Supported: d a multiple of 256 (tensor-core path) or of 64
 * (plain path), d even, H <= 32, A <= 32, head_dim in {32, 64, 128} ...; anything else
 * returns EBRL_ERR_UNSUPPORTED.  On failure *out_handle is NULL. */
ebrl_status_t ebrl_actgen_create(const ebrl_actgen_cfg_t *cfg, const ebrl_actgen_weights_t *weights,
                                 ebrl_actgen_t *out_handle);

/* Enqueues one group of n_envs environments on `stream`.
 *   env_ids    host [n]: unique within the group and among groups not yet synced.  Used only
 *              for these checks and for error text; they never enter the arithmetic.
 *   prefix_kv  host [n] of DEVICE pointers; env i: [kv_layers][2][P_i][d] in kv_dtype, plane 0
 *              = K, plane 1 = V, rows contiguous, 16-byte aligned.  With cfg.d_ctx > 0 env i's
 *              pointer is instead its hidden states [P_i][d_ctx] in kv_dtype; the projected
 *              planes live in scratch of the handle that grows to the largest batch seen
 *              (n_layers * 2 * sum(P_i) * d elements per batch in flight; EBRL_ERR_NOMEM when
 *              the device cannot hold it).
 *              Every value in an environment's planes must be finite.  The tensor-core attention
 *              reads keys and values in blocks of 16 rows; in the last block of a plane the rows
 *              past P_i are the first rows of what follows it INSIDE THE SAME ENVIRONMENT'S
 *              BUFFER (the V plane after K, the next layer's K plane after V when kv_layers > 1;
 *              past the end of the buffer the copy engine supplies zeros, never a neighbour's
 *              memory).  Their scores are masked and their values get weight exactly 0, which
 *              keeps any finite number out of the result -- but 0 x Inf or 0 x NaN is NaN.  So an
 *              Inf or NaN in layer l+1's keys can reach layer l's result of the same environment
 *              (whose layer l+1 would be spoiled by it anyway); no other environment is affected.
 *   noise      DEVICE [n][H][A] fp32: env i's action state at its step index (the initial
 *              noise when that is 0).
 *   out        DEVICE [n][H][A] fp32; may equal noise.
 *   sm_quota   1..#SMs; 0 = all SMs.  Every kernel of this group runs as a persistent grid of
 *              at most sm_quota CTAs (at most one CTA's worth of SMs each), inside a green
 *              context of that many SMs when EBRL_FLAG_GREEN_CTX is set and available.
 *   stream     cudaStream_t of the caller (NULL = the legacy default stream).
 * Queueing (the bounded queue between simulation and generation, section 4.2.2): a submitted
 * group waits in the handle until max_inflight_groups groups are queued, or a group for a
 * different stream or quota arrives, or ebrl_actgen_flush / ebrl_actgen_sync is called; the
 * queued groups are then launched on `stream` as ONE packed batch (their environments share
 * the row space, so the weights stream once per Euler step for all of them).  The batch is
 * ordered after everything on the stream at launch time, and every `out` of the batch is ready
 * for work enqueued on the stream after the launch.  With max_inflight_groups = 1 every submit
 * launches at once.  At most two batches are in flight; a further launch first waits for the
 * older one.  Batching never changes an environment's result.
 * Host arrays are copied before the call returns.  Device buffers must stay valid and
 * unmodified until the group has completed (ebrl_actgen_sync, or ebrl_actgen_flush followed by
 * a stream synchronisation).  n_envs = 0 is a no-op returning EBRL_OK. */
ebrl_status_t ebrl_actgen_submit(ebrl_actgen_t h, int32_t n_envs, const int64_t *env_ids,
                                 const void *const *prefix_kv, const float *noise, float *out,
                                 int32_t sm_quota, void *stream, const ebrl_submit_ext_t *ext);

/* The same as ebrl_actgen_submit with one DEVICE pointer per environment for its state and its
 * result ([H][A] fp32 each, 4-byte aligned; out_ptrs[i] may equal state_ptrs[i]) instead of two
 * [n][H][A] arrays: for callers whose environments keep their buffers apart (the queue of
 * ebrl_queue.h).  state_ptrs and out_ptrs are host arrays, copied before the call returns. */
ebrl_status_t ebrl_actgen_submit_scattered(ebrl_actgen_t h, int32_t n_envs, const int64_t *env_ids,
                                           const void *const *prefix_kv, const float *const *state_ptrs,
                                           float *const *out_ptrs, int32_t sm_quota, void *stream,
                                           const ebrl_submit_ext_t *ext);

/* The same with HOST buffers: prefix_kv[i], noise and out point to host memory (pinned memory
 * makes the copies asynchronous).  The planes and the noise are copied to device staging
 * owned by the handle when the call is made -- on a copy stream of the handle, so that the
 * upload of one batch overlaps the kernels of the previous one -- the group runs with its batch
 * on `stream` once its uploads are done, and `out` is copied back after the batch on `stream`;
 * `out` is valid after ebrl_actgen_sync.  The host buffers must stay valid until then.  Needs
 * prefix_len in ext, or every P_e = max_prefix_len.
 * Batches of host-staged groups ramp up: after create and after every sync the first batch
 * closes at 1 group, the next at 2, then 4, ... up to max_inflight_groups, so that only the first
 * group's upload is exposed and every later batch uploads behind the previous one's kernels. */
ebrl_status_t ebrl_actgen_submit_host(ebrl_actgen_t h, int32_t n_envs, const int64_t *env_ids,
                                      const void *const *prefix_kv_host, const float *noise_host,
                                      float *out_host, int32_t sm_quota, void *stream,
                                      const ebrl_submit_ext_t *ext);

/* Non-blocking weight publication (paper section 4.2.1: training publishes updated weights to
 * the generation workers while rollout continues; the policy version a group ran with is the
 * staleness bookkeeping of section 6).  The handle keeps two weight sets.  The call first
 * launches the groups queued so far (they were submitted under the current version), then
 * copies `weights` (host or device pointers, layout as at create) into the spare set
 * asynchronously on `stream` and makes it the set every later batch uses; batches already
 * launched keep running on the old set.  If the spare set is still being read by an earlier
 * batch, the copy waits for it on the device, not on the host.  The caller's weight buffers
 * must stay valid until `stream` has passed the copy (or until ebrl_actgen_sync).  Versions
 * count from 1 (the weights given at create); *out_version (may be NULL) receives the new one.
 * Pending uploads are device work: ebrl_actgen_sync does not wait for an update that no batch
 * uses yet. */
ebrl_status_t ebrl_actgen_update_weights(ebrl_actgen_t h, const ebrl_actgen_weights_t *weights, void *stream,
                                         uint64_t *out_version);
uint64_t ebrl_actgen_weights_version(ebrl_actgen_t h);

/* Launches the queued groups now, without blocking. */
ebrl_status_t ebrl_actgen_flush(ebrl_actgen_t h);

/* The point where the consumer of the action chunks (the simulation stage of section 4.2.2, which
 * needs an environment's chunk before it can step that environment) waits for generation: launches
 * the queued groups, then blocks until every submitted group has completed; returns the first
 * sticky error. */
ebrl_status_t ebrl_actgen_sync(ebrl_actgen_t h);

/* Ends the generation worker (section 4.2.1: stages are created and retired by the scheduler as
 * resources are re-divided): syncs, then frees everything the handle owns. */
ebrl_status_t ebrl_actgen_destroy(ebrl_actgen_t h);

/* Library-owned, NUL-terminated text of the last error on this handle (or of the last failed
 * create when h is NULL); valid until the next call on the same handle. */
const char *ebrl_actgen_last_error(ebrl_actgen_t h);

/* Counters and per-kernel-class device time since create or the last reset: the measurements the
 * generation profile P_gen(s_g, B_g) of section 4.3.2 is built from (throughput per SM quota and
 * batch size).  A single device_ns total is not kept; class_ms splits it by kernel class. */
ebrl_status_t ebrl_actgen_get_stats(ebrl_actgen_t h, ebrl_actgen_stats_t *out_stats);
ebrl_status_t ebrl_actgen_reset_stats(ebrl_actgen_t h);

/* SM partitions behind the quota (sections 4.2.1 and 4.3.1: stages share a GPU under separate logical
 * SM quotas).  With EBRL_FLAG_GREEN_CTX a submit with 0 < sm_quota < #SMs runs inside a driver
 * partition of *out_gen_sms SMs -- the quota rounded UP to the driver's granularity (8 SMs on B200:
 * 74 -> 80, 37 -> 40) -- while its grids stay capped at exactly sm_quota CTAs: "quota" is the number of
 * SMs the generator keeps busy, the partition is the fence around them.  The SMs outside it form the
 * complementary partition of *out_rest_sms SMs; *out_rest_stream is a cudaStream_t owned by the handle
 * (valid until destroy) whose kernels can only run there, which is where a co-running stage (the
 * simulator stand-in of the bench) belongs so that the driver keeps the two apart in both directions.
 * All three are 0 / NULL when the flag is off, the quota is the whole chip or the driver offers no
 * partitions; any of the out pointers may be NULL.  The partition of a quota is created on first use. */
ebrl_status_t ebrl_actgen_partition_info(ebrl_actgen_t h, int32_t sm_quota, int32_t *out_gen_sms, int32_t *out_rest_sms,
                                         void **out_rest_stream);

/* Switches the per-kernel-class timing (EBRL_FLAG_TIMING) on or off for later submits. */
ebrl_status_t ebrl_actgen_set_timing(ebrl_actgen_t h, int32_t on);

uint32_t ebrl_actgen_abi_version(void);

/* K_steps of the handle's configuration (0 for NULL). */
int32_t ebrl_actgen_k_steps(ebrl_actgen_t h);

/* sizeof of an ABI struct as this library was compiled: 0 ebrl_actgen_cfg_t, 1 ebrl_layer_weights_t,
 * 2 ebrl_actgen_weights_t, 3 ebrl_submit_ext_t, 4 ebrl_actgen_stats_t; 0 for any other index.  For
 * bindings that mirror the structs by hand. */
uint64_t ebrl_actgen_struct_size(int32_t which);

/* ---- an entry point that allocates nothing ---------------------------------------------
 * (The paper has no counterpart; this serves callers that cannot call cudaMalloc.)
 * One Euler step of a layer-less action head on n_rows action tokens:
 *     x = W_in a + temb_row;  v = W_out RMSNorm(x; g_final) + b_out;  a_out = a_in + v / K_steps
 * -- what ebrl_actgen_submit computes for an n_layers = 0, fp32 model advanced by one step --
 * for callers that may not allocate device memory at this point: a control loop that must not
 * take the allocator's lock or risk its implicit synchronisation, a worker whose whole memory
 * budget was handed out at start-up, a plug-in that is only given pointers and a stream.
 * All pointers are DEVICE memory owned by the caller, fp32: a_in/a_out [n_rows][A] (may be the
 * same buffer), w_in [d][A], w_out [A][d], b_out [A], g_final [d], temb_row [d] (the timestep
 * embedding of this step).  The intermediate x is kept in a fixed 2 MiB array that is part of
 * the library image on every GPU that loads it, so the call never calls cudaMalloc, cudaFree
 * or any allocating routine.  Limits: n_rows <= 512, d <= 1024 and a multiple of 128, A <= 32;
 * larger sizes return EBRL_ERR_UNSUPPORTED.  sm_quota as in submit (0 = all SMs).
 * The first call on a device looks up the array's device address (with that device current,
 * which must be the device of `stream`); make that first call outside any stream capture.
 * All calls share the one array and it keeps the previous call's contents: nothing in it needs
 * clearing (every row used is written before it is read), but two calls whose kernels overlap
 * on the GPU (different streams) race on it -- order them on one stream or with events.
 * The work is asynchronous on `stream`. */
ebrl_status_t ebrl_actgen_l0_step_noalloc(const float *a_in, float *a_out, const float *w_in, const float *w_out,
                                          const float *b_out, const float *g_final, const float *temb_row,
                                          int32_t n_rows, int32_t A, int32_t d, int32_t K_steps, float rms_eps,
                                          int32_t sm_quota, void *stream);

/* ---- host-only helpers (no device needed): the argument rules and the batcher's plan ------
 * ebrl_actgen_check_cfg / check_submit apply exactly the checks create / submit apply before
 * touching the device (n_sms = the SM count to check the quota against) and return the same
 * status; the reason is available from ebrl_actgen_last_error(NULL).
 * ebrl_actgen_plan_group returns how the ragged batcher packs a group (sections 4.2.2-4.2.3:
 * environments of a group progress independently): environments are ordered by the number of
 * steps they run, longest first and ties in arrival order, so that the rows still active at
 * inner step s are a prefix.  order[n] = caller index of packed position j, nsteps[n] = steps
 * of packed position j, n_active[K] = environments with more than s steps.  Returns the number
 * of inner steps, or -1 on bad arguments. */
ebrl_status_t ebrl_actgen_check_cfg(const ebrl_actgen_cfg_t *cfg);
ebrl_status_t ebrl_actgen_check_submit(const ebrl_actgen_cfg_t *cfg, int32_t n_sms, int32_t n_envs,
                                       const int64_t *env_ids, const void *const *prefix_kv,
                                       const float *noise, const float *out, int32_t sm_quota,
                                       const ebrl_submit_ext_t *ext);
int32_t ebrl_actgen_plan_group(const ebrl_actgen_cfg_t *cfg, int32_t n_envs, const ebrl_submit_ext_t *ext,
                               int32_t *order, int32_t *nsteps, int32_t *n_active);

/* ---- failure detection without a fault -------------------------------------------------
 * Every device-side wait of the library is bounded (cfg.wait_limit_ns): a producer that never
 * arrives makes the waiting kernel record EBRL_ERR_TIMEOUT and return normally.  This call runs
 * that wait once on `device` in a one-warp kernel: with signal_it = 0 nothing arrives and
 * *out_status becomes EBRL_ERR_TIMEOUT after about limit_ns (1 ns .. 2 s); with signal_it = 1
 * the barrier is signalled and *out_status is EBRL_OK.  *out_waited_ns (may be NULL) is the time
 * the wait took on the device.  The context stays usable either way. */
ebrl_status_t ebrl_actgen_wait_probe(int32_t device, uint64_t limit_ns, int32_t signal_it, int32_t *out_status,
                                     uint64_t *out_waited_ns);

/* ---- bench utility: the synthetic "simulation" co-runner --------------------------------
 * A memory-bound stand-in for a GPU simulator sharing the device with generation (sections
 * 2.2 and 4.2.1): n_steps passes of x[i] = x[i]*alpha + beta over a DEVICE fp32 buffer of
 * n_floats elements, as a persistent grid of n_ctas CTAs on `stream`.  Bounded by
 * construction (no flag to wait for). */
ebrl_status_t ebrl_sim_corunner_launch(float *buf, uint64_t n_floats, int32_t n_steps,
                                       int32_t n_ctas, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* EBRL_ACTGEN_H_ */
