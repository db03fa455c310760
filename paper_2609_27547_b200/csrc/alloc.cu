// Host-only: the elastic resource allocator (section 4.3.2: Algorithm 1 and Eq. 2) and the runtime
// re-balance trigger of the same section.  No device code; lives in the library so that a scheduler
// written in any language can call it next to the generation entry points.
//
// The allocation problem: the simulator keeps the smallest profiled quota at which its rate is within
// a tolerance of its best (more SMs buy it nothing); the rest of the chip is divided between generation
// and training so that the pipeline rate Theta = min(min(T_s, T_g), T_t) is largest.  T_g grows and T_t
// shrinks as generation's share grows, so the division is found by bisecting on "is rollout already
// faster than training?", with the best batch-size pair that fits the memory budget chosen at every
// probe, and the better end of the final bracket returned.
#include "../../include/ebrl_alloc.h"

#include <algorithm>
#include <deque>
#include <new>

namespace {

bool grid_ok(int n, const int32_t *q, int lo)
{
    if (n < 1 || !q) return false;
    for (int i = 0; i < n; ++i) {
        if (q[i] < lo || q[i] > 100) return false;
        if (i && q[i] <= q[i - 1]) return false;
    }
    return true;
}

bool profile_ok(const ebrl_profile_t &p)
{
    if (!grid_ok(p.n_quota, p.quota_pct, 1) || p.n_batch < 1 || !p.batch || !p.rate || !p.mem_gb) return false;
    for (int j = 1; j < p.n_batch; ++j)
        if (p.batch[j] <= p.batch[j - 1]) return false;
    return true;
}

double interp(int n, const int32_t *q, const double *v, int stride, int s)
{
    if (s <= q[0]) return v[0];
    if (s >= q[n - 1]) return v[(size_t)(n - 1) * stride];
    int i = 1;
    while (q[i] < s) ++i;
    const double w = (double)(s - q[i - 1]) / (double)(q[i] - q[i - 1]);
    return v[(size_t)(i - 1) * stride] * (1.0 - w) + v[(size_t)i * stride] * w;
}

struct Cand {
    int s_g, s_t, jg, jt;
    double T_g, T_t, T_r, theta;
    bool feasible;
};

// The batch-size pair with the highest predicted end-to-end rate that fits the memory budget, for one division.
Cand evaluate(const ebrl_alloc_in_t &in, int s_sim, double T_s, int s_g)
{
    Cand best{};
    best.s_g = s_g;
    best.s_t = 100 - s_sim - s_g;
    best.feasible = false;
    for (int jg = 0; jg < in.gen.n_batch; ++jg)
        for (int jt = 0; jt < in.train.n_batch; ++jt) {
            if (in.gen.mem_gb[jg] + in.train.mem_gb[jt] > in.mem_gpu_gb) continue;
            const double T_g = ebrl_profile_rate(&in.gen, s_g, jg), T_t = ebrl_profile_rate(&in.train, best.s_t, jt);
            const double T_r = std::min(T_s, T_g), theta = std::min(T_r, T_t);
            if (!best.feasible || theta > best.theta) {
                best.feasible = true;
                best.jg = jg; best.jt = jt; best.T_g = T_g; best.T_t = T_t; best.T_r = T_r; best.theta = theta;
            }
        }
    return best;
}

// The simulator's knee: the first profiled quota whose rate is within the tolerance of the table's best.
// Rates must be positive finite numbers (a table of zeros, negatives or NaNs has no knee).
bool simulator_knee(const ebrl_alloc_in_t &in, int *knee)
{
    double peak = 0.0;
    for (int i = 0; i < in.n_sim_quota; ++i) {
        const double r = in.sim_rate[i];
        if (!(r > 0.0) || !(r < 1e300)) return false;
        peak = std::max(peak, r);
    }
    for (int i = 0; i < in.n_sim_quota; ++i)
        if (in.sim_rate[i] >= (1.0 - in.knee_tolerance) * peak) { *knee = i; return true; }
    return false;
}

// Integer bisection: shrinks [lo, hi] to adjacent values, keeping pred false towards lo and true towards hi.
template <typename Pred>
void narrow_bracket(int &lo, int &hi, int &probes, Pred pred)
{
    while (hi - lo > 1) {
        const int mid = lo + (hi - lo) / 2;
        if (pred(mid)) hi = mid; else lo = mid;
        ++probes;
    }
}

}  // namespace

struct ebrl_rebalance {
    int window, streak_needed, streak;
    double threshold;
    std::deque<double> ro, tr;
    double sum_ro, sum_tr;
};

extern "C" {

double ebrl_profile_rate(const ebrl_profile_t *p, int32_t quota_pct, int32_t j)
{
    if (!p || !profile_ok(*p) || j < 0 || j >= p->n_batch) return 0.0;
    return interp(p->n_quota, p->quota_pct, p->rate + j, p->n_batch, quota_pct);
}

int32_t ebrl_alloc_elastic(const ebrl_alloc_in_t *in, ebrl_alloc_out_t *out)
{
    if (!in || !out || in->cores < 1 || in->cores_per_env < 1 || !in->sim_rate || !(in->knee_tolerance >= 0.0)) return 1;
    if (!grid_ok(in->n_sim_quota, in->sim_quota_pct, 0) || !profile_ok(in->gen) || !profile_ok(in->train)) return 1;
    if (in->s_g_min < 1 || in->s_t_min < 1) return 1;
    const int E = in->cores / in->cores_per_env;     // environments the host cores can drive
    if (E < 1) return 1;
    int knee = -1;
    if (!simulator_knee(*in, &knee)) return 1;
    const int s_sim = in->sim_quota_pct[knee];
    const double T_s = in->sim_rate[knee];
    int lo = in->s_g_min, hi = 100 - s_sim - in->s_t_min;   // what is left for generation once training has its minimum
    if (hi < lo) return 1;
    int it = 0;
    bool all_feasible = true;
    // rollout_ahead(s_g): with this share, does rollout already outpace training?  False at small shares, true at large ones.
    narrow_bracket(lo, hi, it, [&](int s_g) {
        const Cand c = evaluate(*in, s_sim, T_s, s_g);
        all_feasible = all_feasible && c.feasible;
        return c.feasible && c.T_r > c.T_t;
    });
    if (!all_feasible) return 1;
    const Cand a = evaluate(*in, s_sim, T_s, lo), b = evaluate(*in, s_sim, T_s, hi);
    if (!a.feasible && !b.feasible) return 1;
    const Cand &w = (!b.feasible || (a.feasible && a.theta >= b.theta)) ? a : b;
    out->env_concurrency = E;
    out->s_sim = s_sim; out->s_g = w.s_g; out->s_t = w.s_t;
    out->B_g = in->gen.batch[w.jg]; out->B_t = in->train.batch[w.jt];
    out->T_s = T_s; out->T_g = w.T_g; out->T_t = w.T_t; out->T_r = w.T_r; out->theta = w.theta;
    out->iterations = it;
    return 0;
}

ebrl_rebalance_t ebrl_rebalance_create(int32_t window, int32_t streak, double threshold)
{
    ebrl_rebalance *r = new (std::nothrow) ebrl_rebalance();
    if (!r) return nullptr;
    r->window = window > 0 ? window : 20;
    r->streak_needed = streak > 0 ? streak : 20;
    r->threshold = threshold > 0.0 ? threshold : 0.15;
    r->streak = 0;
    r->sum_ro = r->sum_tr = 0.0;
    return r;
}

int32_t ebrl_rebalance_push(ebrl_rebalance_t r, double ro, double tr)
{
    if (!r) return -1;
    r->ro.push_back(ro); r->sum_ro += ro;
    r->tr.push_back(tr); r->sum_tr += tr;
    if ((int)r->ro.size() > r->window) {
        r->sum_ro -= r->ro.front(); r->ro.pop_front();
        r->sum_tr -= r->tr.front(); r->tr.pop_front();
    }
    const double a = r->sum_ro / (double)r->ro.size(), b = r->sum_tr / (double)r->tr.size();
    const double faster = std::max(a, b), gap = faster - std::min(a, b);
    if (faster > 0.0 && gap > r->threshold * faster) ++r->streak; else r->streak = 0;
    if (r->streak >= r->streak_needed) { r->streak = 0; return 1; }
    return 0;
}

void ebrl_rebalance_get(ebrl_rebalance_t r, double *a, double *b, int32_t *streak)
{
    if (!r) return;
    if (a) *a = r->ro.empty() ? 0.0 : r->sum_ro / (double)r->ro.size();
    if (b) *b = r->tr.empty() ? 0.0 : r->sum_tr / (double)r->tr.size();
    if (streak) *streak = r->streak;
}

void ebrl_rebalance_destroy(ebrl_rebalance_t r) { delete r; }

}  // extern "C"
