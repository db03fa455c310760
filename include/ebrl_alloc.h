/*
 * ebrl_alloc -- the elastic resource allocator of the paper (section 4.3.2, Algorithm 1, Eq. 2)
 * and its runtime re-balance trigger, as host-only C calls.  It consumes stage profiles: the
 * generation profile P_gen(s_g, B_g) is what the bench harness of ebrl_actgen measures
 * (environment action-chunks per second per SM quota and batch size); P_sim and P_train come from
 * the user's own profiling.  All rates are in rollout chunk-steps per second (Eq. 2).
 *
 * Readings where the paper is silent: profiles are tables on a grid of SM-quota percentages and
 * batch sizes; a rate at a quota between grid points is interpolated linearly in the quota and
 * held constant outside the grid; the "simulator knee" is the smallest grid quota whose rate is
 * within knee_tolerance of the table's maximum; a batch size is feasible when the memory the two
 * stages need at their batch sizes fits M_gpu; "best feasible pair" maximises
 * min(T_s, P_gen, P_train) with ties broken toward smaller batches.
 */
#ifndef EBRL_ALLOC_H_
#define EBRL_ALLOC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* A stage profile on a grid: rate[i * n_batch + j] at quota_pct[i] (strictly increasing, 1..100)
 * and batch[j]; mem_gb[j] = device memory the stage needs at batch[j]. */
typedef struct {
    int32_t n_quota, n_batch;
    const int32_t *quota_pct;
    const int32_t *batch;
    const double *rate;
    const double *mem_gb;
} ebrl_profile_t;

typedef struct {
    int32_t cores;              /* N: CPU cores for simulation                                  */
    int32_t cores_per_env;      /* c_env*: profiled per-environment core count                  */
    /* simulator rate at (c_env*, E = floor(N / c_env*)) as a function of its SM quota; a
     * CPU-only simulator passes one grid point with quota 0                                    */
    int32_t n_sim_quota;
    const int32_t *sim_quota_pct;
    const double *sim_rate;
    double knee_tolerance;      /* 0.05: "additional SMs bring little gain" below this relative gap */
    ebrl_profile_t gen, train;
    int32_t s_g_min, s_t_min;   /* minimum generation / training quota, percent                  */
    double mem_gpu_gb;          /* M_gpu                                                         */
} ebrl_alloc_in_t;

typedef struct {
    int32_t env_concurrency;    /* E                                                            */
    int32_t s_sim, s_g, s_t;    /* SM quotas, percent                                           */
    int32_t B_g, B_t;           /* batch sizes                                                  */
    double T_s, T_g, T_t;       /* stage rates at the chosen configuration                      */
    double T_r, theta;          /* Eq. 2: T_r = min(T_s, T_g); theta = min(T_r, T_t)            */
    int32_t iterations;         /* bisection steps taken                                        */
} ebrl_alloc_out_t;

/* Algorithm 1.  Returns 0, or 1 on invalid input (NULL, empty or unsorted grids, no feasible
 * quota interval, no batch pair that fits M_gpu). */
int32_t ebrl_alloc_elastic(const ebrl_alloc_in_t *in, ebrl_alloc_out_t *out);

/* Piecewise-linear lookup of a profile at an integer quota and one of its batch sizes
 * (index j); exported for tests. */
double ebrl_profile_rate(const ebrl_profile_t *p, int32_t quota_pct, int32_t batch_index);

/* Runtime adaptation (section 4.3.2): 20-step moving averages of the observed rollout and
 * training throughputs; the allocator is re-run when their gap exceeds 15 % of the faster stage
 * for 20 consecutive steps.  window, streak and threshold are parameters with those defaults
 * when given as 0. */
typedef struct ebrl_rebalance *ebrl_rebalance_t;
ebrl_rebalance_t ebrl_rebalance_create(int32_t window, int32_t streak, double threshold);
/* Feeds one step's observed rates; returns 1 when the trigger fires (the streak then restarts),
 * else 0; -1 on a NULL handle. */
int32_t ebrl_rebalance_push(ebrl_rebalance_t r, double rollout_rate, double train_rate);
void ebrl_rebalance_get(ebrl_rebalance_t r, double *avg_rollout, double *avg_train, int32_t *current_streak);
void ebrl_rebalance_destroy(ebrl_rebalance_t r);

#ifdef __cplusplus
}
#endif
#endif /* EBRL_ALLOC_H_ */
