/*
 * ebrl_queue -- the bounded producer-consumer queue between simulation and generation (paper section
 * 4.2.2: environments that have finished a simulator step hand their observation to generation
 * through a bounded queue, which limits how many observations wait and lets generation of one
 * group run while other environments still simulate), with the two serving policies of section
 * 4.2.3: whole action chunks per group, or step-level continuous batching, where every Euler step
 * is its own launch and environments that arrive while others are mid-chunk join the next step.
 *
 * Simulator threads push one request per environment; a worker thread owned by the queue forms
 * groups (everything that is waiting, up to max_group, after at most linger_us of waiting for
 * company), runs them through an ebrl_actgen handle and marks the requests complete.  The queue
 * holds at most `capacity` requests that have not been handed to generation; a push beyond that
 * blocks (or fails, for try_push): back-pressure on the simulators.
 *
 * Results do not depend on how requests were grouped: an environment's chunk is the bits the
 * handle delivers for it alone.
 *
 * Everything here is host code; pointers named *_dev are device pointers that are only passed on.
 * All calls return a status and never throw.  Calls on one queue may come from any threads.
 */
#ifndef EBRL_QUEUE_H_
#define EBRL_QUEUE_H_

#include "ebrl_actgen.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ebrl_queue *ebrl_queue_t;

#define EBRL_ERR_QUEUE_FULL 8   /* try_push: `capacity` requests are already waiting            */
#define EBRL_ERR_CLOSED 9       /* the queue is shutting down                                   */

typedef struct {
    int32_t capacity;     /* requests that may wait for generation (>= 1): the bound of the queue */
    int32_t max_group;    /* environments per launched group (>= 1, <= the handle's max_group_envs) */
    int32_t sm_quota;     /* passed to every submit (0 = all SMs)                                  */
    int32_t step_mode;    /* 0: a request is served by one submit that runs it to step K;
                             1: one Euler step per submit; unfinished environments stay in service
                                and environments that arrived meanwhile join the next step        */
    uint32_t linger_us;   /* how long the worker waits for more requests before it launches a group
                             smaller than max_group (0 = launch whatever is there)                */
    uint32_t reserved_;
} ebrl_queue_cfg_t;

/* What the worker calls to run a group.  ebrl_queue_create fills this with the handle's own entry
 * points; tests may supply their own to exercise the queue without a GPU.  Both functions return an
 * ebrl_status_t value (as int32_t).
 *   submit: one group, per-environment device pointers; n_steps = 0 runs every environment to step K. */
typedef int32_t (*ebrl_queue_submit_fn)(void *ctx, int32_t n, const int64_t *env_ids, const void *const *prefix_dev,
                                        const int32_t *prefix_len, const float *const *state_dev, float *const *out_dev,
                                        const int32_t *step_index, int32_t n_steps, int32_t sm_quota, void *stream);
typedef int32_t (*ebrl_queue_sync_fn)(void *ctx);
typedef struct {
    void *ctx;
    int32_t K_steps;
    ebrl_queue_submit_fn submit;
    ebrl_queue_sync_fn sync;
} ebrl_queue_backend_t;

typedef struct {
    uint64_t pushed, completed, failed;   /* requests                                            */
    uint64_t groups;                      /* submits                                             */
    uint64_t group_envs;                  /* environments over all submits (mean size = / groups) */
    uint64_t blocked_pushes;              /* pushes that had to wait for room                    */
    int32_t max_waiting;                  /* most requests ever waiting at once (<= capacity)     */
    int32_t waiting, in_service;          /* now                                                 */
    int32_t reserved_;
} ebrl_queue_stats_t;

/* A queue in front of `gen`, launching on `stream` (cudaStream_t; NULL = default stream).  The
 * queue does not own the handle; destroy the queue first. */
ebrl_status_t ebrl_queue_create(ebrl_actgen_t gen, const ebrl_queue_cfg_t *cfg, void *stream, ebrl_queue_t *out);
/* The same over an arbitrary backend (K_steps >= 1, submit and sync not NULL). */
ebrl_status_t ebrl_queue_create_backend(const ebrl_queue_backend_t *backend, const ebrl_queue_cfg_t *cfg, void *stream,
                                        ebrl_queue_t *out);

/* One environment asks for its next action chunk.
 *   prefix_dev   its prefix (planes or hidden states, as the handle was configured), device memory
 *   prefix_len   P_e
 *   state_dev    device [H][A] fp32: its action state at step_index (the noise when that is 0)
 *   out_dev      device [H][A] fp32: where the final chunk goes; may equal state_dev.  In step mode
 *                it also carries the state between steps.
 *   step_index   k_e in [0, K)
 * Blocks while `capacity` requests are waiting.  *ticket identifies the request for ebrl_queue_wait.
 * The buffers must stay valid until the request has completed.  An env_id may have only one request
 * in the queue at a time (EBRL_ERR_ENV_BUSY otherwise). */
ebrl_status_t ebrl_queue_push(ebrl_queue_t q, int64_t env_id, const void *prefix_dev, int32_t prefix_len,
                              const float *state_dev, float *out_dev, int32_t step_index, uint64_t *ticket);
/* The same, but returns EBRL_ERR_QUEUE_FULL instead of blocking. */
ebrl_status_t ebrl_queue_try_push(ebrl_queue_t q, int64_t env_id, const void *prefix_dev, int32_t prefix_len,
                                  const float *state_dev, float *out_dev, int32_t step_index, uint64_t *ticket);
/* Blocks until the request has completed (its chunk is in out_dev and visible to work enqueued on
 * any stream afterwards: the worker synchronises the handle before it reports completion) or
 * timeout_ms has passed (EBRL_ERR_TIMEOUT; 0 = wait without limit).  Returns the request's own
 * status.  A ticket can be waited for once. */
ebrl_status_t ebrl_queue_wait(ebrl_queue_t q, uint64_t ticket, uint32_t timeout_ms);
ebrl_status_t ebrl_queue_get_stats(ebrl_queue_t q, ebrl_queue_stats_t *out);
/* Serves what is waiting (every accepted request completes), stops the worker, releases pushes
 * that were blocked for room with EBRL_ERR_CLOSED, lets waits that are in progress return, and
 * frees the queue.  No call on the queue may START once destroy has been called. */
ebrl_status_t ebrl_queue_destroy(ebrl_queue_t q);

#ifdef __cplusplus
}
#endif
#endif
