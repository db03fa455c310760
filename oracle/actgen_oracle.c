/*
 * fp64 CPU oracle for batched action generation (TEST INFRASTRUCTURE ONLY).
 *
 * This file is the slow, plain statement of what the action-generation path computes.  It is
 * used by the tests, by the smoke check and by the bench's CPU-baseline leg; the product path
 * never calls it and shares no code, header, table or constant with it.
 *
 * What it follows.  The paper (section 2.1) describes the operation only in outline: a
 * diffusion-style action head turns a random tensor into an action chunk over several
 * denoising steps, conditioned on a representation cached by the backbone (a KV cache).
 * Section 4.2.2 adds that every environment depends only on its own observations and actions,
 * so environments are processed here one at a time, each by the same plain sequence.  The
 * concrete head (pre-RMSNorm blocks of self-attention over the H action tokens,
 * cross-attention to the cached prefix K/V, GELU MLP, linear embedding plus sinusoidal
 * timestep embedding, linear velocity output, explicit Euler update a += v/K) is the one the
 * benchmark configurations state; the paper fixes none of it.  That this architecture is the
 * one the paper's policies use is therefore "parity unpinned" by the paper; every arithmetic
 * piece below is pinned by closed forms, invariants, brute force and library cross-checks in
 * the CPU test-suite.
 *
 * Arithmetic: every stored input (fp32 values; bf16 inputs arrive already rounded and widened
 * to fp32) is widened to fp64 and nothing is rounded afterwards.  No blocking, no fusion, no
 * reordering: loops run in the order of the formulas.  Threads split the work across
 * environments only, so each environment's arithmetic is one sequential chain.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t H;          /* action tokens per chunk                         */
    int32_t A;          /* action dimensions                               */
    int32_t d;          /* model width (even)                              */
    int32_t n_layers;   /* L                                               */
    int32_t n_heads;    /* heads; head_dim = d / n_heads                   */
    int32_t mlp_mult;   /* hidden width of the MLP = mlp_mult * d          */
    int32_t K_steps;    /* K Euler steps from t = 0 (noise) to t = 1       */
    int32_t kv_layers;  /* 1: one K/V plane pair for all layers; L: per-layer planes */
    double rms_eps;
    double temb_scale;
    double temb_max_period;
    int32_t d_ctx;      /* 0: the prefix is the cached K/V planes.  > 0: the prefix is the backbone's
                           hidden states [P][d_ctx] and every layer projects its own keys and values
                           from them (the cross-attention form of heads that attend to backbone
                           features rather than to a ready-made cache, section 2.1)               */
} ebrl_oracle_cfg;

typedef struct {
    const float *w_in;    /* [d][A]  */
    const float *w_out;   /* [A][d]  */
    const float *b_out;   /* [A]     */
    const float *g_final; /* [d]     */
    /* one pointer per layer in each array */
    const float *const *g1;    /* [d]      */
    const float *const *g2;    /* [d]      */
    const float *const *g3;    /* [d]      */
    const float *const *w_qkv; /* [3d][d]  rows 0..d-1 = Q, d..2d-1 = K, 2d..3d-1 = V */
    const float *const *w_o;   /* [d][d]   */
    const float *const *w_qc;  /* [d][d]   */
    const float *const *w_oc;  /* [d][d]   */
    const float *const *w_1;   /* [md][d]  */
    const float *const *w_2;   /* [d][md]  */
    const float *const *w_kc;  /* [d][d_ctx]  key projection of the hidden-state prefix (d_ctx > 0)   */
    const float *const *w_vc;  /* [d][d_ctx]  value projection, likewise                              */
} ebrl_oracle_weights;

/* ------------------------------------------------------------------------------------------
 * Elementary pieces.  Each is exported so that the tests can pin it on its own.
 * ---------------------------------------------------------------------------------------- */

/* Sinusoidal timestep embedding of Euler step k (t = k/K, tau = temb_scale * t):
 *   temb[j]       = sin(tau * w_j),  temb[d/2 + j] = cos(tau * w_j),
 *   w_j = temb_max_period^(-j / (d/2)),  j = 0 .. d/2-1.                                     */
void ebrl_oracle_timestep_embedding(const ebrl_oracle_cfg *c, int k, double *temb)
{
    const int half = c->d / 2;
    const double tau = c->temb_scale * ((double)k / (double)c->K_steps);
    for (int j = 0; j < half; ++j) {
        const double w = pow(c->temb_max_period, -(double)j / (double)half);
        temb[j] = sin(tau * w);
        temb[half + j] = cos(tau * w);
    }
}

/* RMSNorm(x; g)_j = g_j * x_j / sqrt(mean_i(x_i^2) + eps). */
void ebrl_oracle_rmsnorm(const double *x, const float *g, int d, double eps, double *y)
{
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += x[i] * x[i];
    const double r = sqrt(ss / (double)d + eps);
    for (int j = 0; j < d; ++j) y[j] = (double)g[j] * x[j] / r;
}

/* GELU in its exact form: z/2 * (1 + erf(z / sqrt 2)). */
double ebrl_oracle_gelu(double z)
{
    return 0.5 * z * (1.0 + erf(z / sqrt(2.0)));
}

/* In-place softmax of one row: subtract the maximum, exponentiate, divide by the sum. */
void ebrl_oracle_softmax_row(double *s, int n)
{
    double m = s[0];
    for (int j = 1; j < n; ++j) if (s[j] > m) m = s[j];
    double z = 0.0;
    for (int j = 0; j < n; ++j) { s[j] = exp(s[j] - m); z += s[j]; }
    for (int j = 0; j < n; ++j) s[j] /= z;
}

/* y[n] = W[n][k] x[k]  (y = W x; W row-major [n_out][n_in]), optionally y += instead of y =. */
static void matvec(const float *W, const double *x, int n_out, int n_in, double *y, int accumulate)
{
    for (int o = 0; o < n_out; ++o) {
        double acc = 0.0;
        const float *row = W + (size_t)o * (size_t)n_in;
        for (int i = 0; i < n_in; ++i) acc += (double)row[i] * x[i];
        if (accumulate) y[o] += acc; else y[o] = acc;
    }
}

/* One softmax-attention head, no mask:
 *   out[i][:] = sum_j softmax_j( q[i].k[j] / sqrt(hd) ) v[j][:]
 * q rows have stride q_stride doubles; keys/values are given either as doubles (kd/vd) or as
 * floats (kf/vf) with row stride kv_stride; out rows have stride o_stride.                   */
static void attention_head(const double *q, int q_stride, int nq,
                           const double *kd, const double *vd, const float *kf, const float *vf,
                           int kv_stride, int nk, int hd, double *out, int o_stride, double *scores)
{
    const double scale = 1.0 / sqrt((double)hd);
    for (int i = 0; i < nq; ++i) {
        for (int j = 0; j < nk; ++j) {
            double s = 0.0;
            for (int c = 0; c < hd; ++c) {
                const double kv = kd ? kd[(size_t)j * kv_stride + c] : (double)kf[(size_t)j * kv_stride + c];
                s += q[(size_t)i * q_stride + c] * kv;
            }
            scores[j] = s * scale;
        }
        ebrl_oracle_softmax_row(scores, nk);
        for (int c = 0; c < hd; ++c) {
            double o = 0.0;
            for (int j = 0; j < nk; ++j) {
                const double vv = vd ? vd[(size_t)j * kv_stride + c] : (double)vf[(size_t)j * kv_stride + c];
                o += scores[j] * vv;
            }
            out[(size_t)i * o_stride + c] = o;
        }
    }
}

/* Exported wrapper of one attention head on float keys/values (for the pins). */
void ebrl_oracle_attention_head(const double *q, int nq, const float *k, const float *v, int nk,
                                int hd, double *out)
{
    double *scores = (double *)malloc(sizeof(double) * (size_t)nk);
    attention_head(q, hd, nq, NULL, NULL, k, v, hd, nk, hd, out, hd, scores);
    free(scores);
}

/* ------------------------------------------------------------------------------------------
 * The velocity network for one environment at Euler step k:  v = f(a, t_k; prefix K/V).
 * a, v: [H][A] doubles.  kv: [kv_layers][2][P][d] floats (plane 0 = K, plane 1 = V); with
 * d_ctx > 0 it is the hidden states [P][d_ctx] and layer l attends to Kc = h W_kc_l^T,
 * Vc = h W_vc_l^T (nothing rounded in between).
 * ---------------------------------------------------------------------------------------- */
int ebrl_oracle_velocity(const ebrl_oracle_cfg *c, const ebrl_oracle_weights *w,
                         const float *kv, int P, const double *a, int k, double *v)
{
    const int H = c->H, A = c->A, d = c->d, L = c->n_layers, nh = c->n_heads;
    const int hd = d / nh, md = c->mlp_mult * d;
    const int smax = (P > H ? P : H);
    double *temb = (double *)malloc(sizeof(double) * (size_t)d);
    double *x = (double *)malloc(sizeof(double) * (size_t)H * d);
    double *y = (double *)malloc(sizeof(double) * (size_t)d);
    double *qkv = (double *)malloc(sizeof(double) * (size_t)H * 3 * d);
    double *att = (double *)malloc(sizeof(double) * (size_t)H * d);
    double *qc = (double *)malloc(sizeof(double) * (size_t)H * d);
    double *u = (double *)malloc(sizeof(double) * (size_t)md);
    double *scores = (double *)malloc(sizeof(double) * (size_t)smax);
    if (!temb || !x || !y || !qkv || !att || !qc || !u || !scores) return 1;

    /* input embedding: x_h = W_in a_h + temb(t_k); no bias, no positional term over h */
    ebrl_oracle_timestep_embedding(c, k, temb);
    for (int h = 0; h < H; ++h) {
        matvec(w->w_in, a + (size_t)h * A, d, A, x + (size_t)h * d, 0);
        for (int j = 0; j < d; ++j) x[(size_t)h * d + j] += temb[j];
    }

    for (int l = 0; l < L; ++l) {
        /* self-attention over the H action tokens of this environment */
        for (int h = 0; h < H; ++h) {
            ebrl_oracle_rmsnorm(x + (size_t)h * d, w->g1[l], d, c->rms_eps, y);
            matvec(w->w_qkv[l], y, 3 * d, d, qkv + (size_t)h * 3 * d, 0);
        }
        for (int hh = 0; hh < nh; ++hh)
            attention_head(qkv + (size_t)hh * hd, 3 * d, H,
                           qkv + d + (size_t)hh * hd, qkv + 2 * d + (size_t)hh * hd, NULL, NULL,
                           3 * d, H, hd, att + (size_t)hh * hd, d, scores);
        for (int h = 0; h < H; ++h)
            matvec(w->w_o[l], att + (size_t)h * d, d, d, x + (size_t)h * d, 1);

        /* cross-attention to the cached prefix: keys/values are used as cached, unprojected */
        for (int h = 0; h < H; ++h) {
            ebrl_oracle_rmsnorm(x + (size_t)h * d, w->g2[l], d, c->rms_eps, y);
            matvec(w->w_qc[l], y, d, d, qc + (size_t)h * d, 0);
        }
        if (c->d_ctx > 0) {
            /* keys and values of this layer from the prefix's hidden states, row by row */
            const int dc = c->d_ctx;
            double *Kd = (double *)malloc(sizeof(double) * (size_t)P * d);
            double *Vd = (double *)malloc(sizeof(double) * (size_t)P * d);
            double *hrow = (double *)malloc(sizeof(double) * (size_t)dc);
            if (!Kd || !Vd || !hrow) return 1;
            for (int p = 0; p < P; ++p) {
                for (int j = 0; j < dc; ++j) hrow[j] = (double)kv[(size_t)p * dc + j];
                matvec(w->w_kc[l], hrow, d, dc, Kd + (size_t)p * d, 0);
                matvec(w->w_vc[l], hrow, d, dc, Vd + (size_t)p * d, 0);
            }
            for (int hh = 0; hh < nh; ++hh)
                attention_head(qc + (size_t)hh * hd, d, H, Kd + (size_t)hh * hd, Vd + (size_t)hh * hd,
                               NULL, NULL, d, P, hd, att + (size_t)hh * hd, d, scores);
            free(Kd); free(Vd); free(hrow);
        } else {
            const int pl = (c->kv_layers == 1) ? 0 : l;
            const float *Kc = kv + (size_t)pl * 2 * (size_t)P * d;
            const float *Vc = Kc + (size_t)P * d;
            for (int hh = 0; hh < nh; ++hh)
                attention_head(qc + (size_t)hh * hd, d, H, NULL, NULL,
                               Kc + (size_t)hh * hd, Vc + (size_t)hh * hd, d, P, hd,
                               att + (size_t)hh * hd, d, scores);
        }
        for (int h = 0; h < H; ++h)
            matvec(w->w_oc[l], att + (size_t)h * d, d, d, x + (size_t)h * d, 1);

        /* MLP */
        for (int h = 0; h < H; ++h) {
            ebrl_oracle_rmsnorm(x + (size_t)h * d, w->g3[l], d, c->rms_eps, y);
            matvec(w->w_1[l], y, md, d, u, 0);
            for (int j = 0; j < md; ++j) u[j] = ebrl_oracle_gelu(u[j]);
            matvec(w->w_2[l], u, d, md, x + (size_t)h * d, 1);
        }
    }

    /* velocity head: v_h = W_out RMSNorm(x_h; g_final) + b_out */
    for (int h = 0; h < H; ++h) {
        ebrl_oracle_rmsnorm(x + (size_t)h * d, w->g_final, d, c->rms_eps, y);
        matvec(w->w_out, y, A, d, v + (size_t)h * A, 0);
        for (int j = 0; j < A; ++j) v[(size_t)h * A + j] += (double)w->b_out[j];
    }

    free(temb); free(x); free(y); free(qkv); free(att); free(qc); free(u); free(scores);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Explicit Euler integration of da/dt = v(a, t) from step k0 to step k1 (t_k = k/K,
 * step size 1/K):  a <- a + v(a, t_k) / K.   The velocity is a callback so that the
 * integrator can be pinned on a velocity field with a known solution.
 * ---------------------------------------------------------------------------------------- */
typedef int (*ebrl_oracle_velocity_fn)(void *ctx, const double *a, int k, double *v);

int ebrl_oracle_euler(int n, int K, int k0, int k1, double *a,
                      ebrl_oracle_velocity_fn f, void *ctx)
{
    double *v = (double *)malloc(sizeof(double) * (size_t)n);
    if (!v) return 1;
    for (int k = k0; k < k1; ++k) {
        const int rc = f(ctx, a, k, v);
        if (rc) { free(v); return rc; }
        for (int i = 0; i < n; ++i) a[i] += v[i] / (double)K;
    }
    free(v);
    return 0;
}

typedef struct {
    const ebrl_oracle_cfg *c;
    const ebrl_oracle_weights *w;
    const float *kv;
    int P;
    int pull;   /* 1: the linear test field v = b_out - a instead of the network */
} env_ctx;

static int env_velocity(void *p, const double *a, int k, double *v)
{
    const env_ctx *e = (const env_ctx *)p;
    if (e->pull) {
        for (int h = 0; h < e->c->H; ++h)
            for (int j = 0; j < e->c->A; ++j)
                v[h * e->c->A + j] = (double)e->w->b_out[j] - a[h * e->c->A + j];
        return 0;
    }
    return ebrl_oracle_velocity(e->c, e->w, e->kv, e->P, a, k, v);
}

/* ------------------------------------------------------------------------------------------
 * A group of environments.  Environment i starts from noise[i] (its current action state at
 * step step_index[i]; the initial noise when that is 0) and advances to step K, or by
 * n_steps steps if n_steps > 0 (never beyond K).  out[i] = the state reached.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
    const ebrl_oracle_cfg *c;
    const ebrl_oracle_weights *w;
    int n_envs;
    const float *const *prefix_kv;
    const int32_t *prefix_len;
    const int32_t *step_index;
    int n_steps;
    const float *noise;
    double *out;
    int pull;
    pthread_mutex_t mu;
    int next;
    int err;
} job_t;

static void *worker(void *p)
{
    job_t *job = (job_t *)p;
    const int n = job->c->H * job->c->A;
    for (;;) {
        pthread_mutex_lock(&job->mu);
        const int i = job->next++;
        pthread_mutex_unlock(&job->mu);
        if (i >= job->n_envs) break;
        double *a = job->out + (size_t)i * n;
        for (int j = 0; j < n; ++j) a[j] = (double)job->noise[(size_t)i * n + j];
        const int k0 = job->step_index ? job->step_index[i] : 0;
        int k1 = job->c->K_steps;
        if (job->n_steps > 0 && k0 + job->n_steps < k1) k1 = k0 + job->n_steps;
        env_ctx e = { job->c, job->w, job->prefix_kv ? job->prefix_kv[i] : NULL,
                      job->prefix_len ? job->prefix_len[i] : 0, job->pull };
        const int rc = ebrl_oracle_euler(n, job->c->K_steps, k0, k1, a, env_velocity, &e);
        if (rc) { pthread_mutex_lock(&job->mu); job->err = rc; pthread_mutex_unlock(&job->mu); }
    }
    return NULL;
}

int ebrl_oracle_actgen(const ebrl_oracle_cfg *c, const ebrl_oracle_weights *w, int n_envs,
                       const float *const *prefix_kv, const int32_t *prefix_len,
                       const int32_t *step_index, int n_steps, const float *noise, double *out,
                       int n_threads, int pull)
{
    if (!c || !w || n_envs < 0 || !noise || !out) return 2;
    if (c->d % 2 || c->n_heads < 1 || c->d % c->n_heads || c->K_steps < 1) return 2;
    job_t job;
    memset(&job, 0, sizeof job);
    job.c = c; job.w = w; job.n_envs = n_envs; job.prefix_kv = prefix_kv;
    job.prefix_len = prefix_len; job.step_index = step_index; job.n_steps = n_steps;
    job.noise = noise; job.out = out; job.pull = pull;
    pthread_mutex_init(&job.mu, NULL);
    if (n_threads < 1) n_threads = 1;
    if (n_threads > n_envs) n_threads = n_envs > 0 ? n_envs : 1;
    if (n_threads == 1) {
        worker(&job);
    } else {
        pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)n_threads);
        int started = 0;
        for (int t = 0; t < n_threads; ++t)
            if (pthread_create(&th[t], NULL, worker, &job) == 0) ++started; else break;
        if (started == 0) worker(&job);
        for (int t = 0; t < started; ++t) pthread_join(th[t], NULL);
        free(th);
    }
    pthread_mutex_destroy(&job.mu);
    return job.err;
}
