// The bounded request queue in front of a generation handle (host code only): simulator threads
// push per-environment requests, one worker thread forms groups and runs them.  See ebrl_queue.h.
#include "../../include/ebrl_queue.h"

#include <algorithm>
#include <chrono>
#include <condition_variable>
#include <deque>
#include <mutex>
#include <new>
#include <thread>
#include <unordered_map>
#include <unordered_set>
#include <vector>

namespace {

struct Request {
    uint64_t ticket;
    int64_t env_id;
    const void *prefix;
    int32_t prefix_len;
    const float *state;
    float *out;
    int32_t step;      // next Euler step of this environment
};

// The handle's own entry points as a backend.
int32_t gen_submit(void *ctx, int32_t n, const int64_t *env_ids, const void *const *prefix_dev, const int32_t *prefix_len,
                         const float *const *state_dev, float *const *out_dev, const int32_t *step_index, int32_t n_steps,
                         int32_t sm_quota, void *stream)
{
    ebrl_submit_ext_t ext{prefix_len, step_index, n_steps};
    return ebrl_actgen_submit_scattered((ebrl_actgen_t)ctx, n, env_ids, prefix_dev, state_dev, out_dev, sm_quota, stream, &ext);
}
int32_t gen_sync(void *ctx) { return ebrl_actgen_sync((ebrl_actgen_t)ctx); }

}  // namespace

struct ebrl_queue {
    ebrl_queue_backend_t be;
    ebrl_queue_cfg_t cfg;
    void *stream = nullptr;
    std::mutex mu;
    std::condition_variable not_full, not_empty, done_cv;
    std::deque<Request> waiting;                       // pushed, not yet handed to generation
    std::vector<Request> in_service;                   // step mode: mid-chunk environments, in admission order
    std::unordered_set<int64_t> live_envs;             // env ids with a request in the queue
    std::unordered_map<uint64_t, ebrl_status_t> finished;   // completed tickets not yet waited for
    std::unordered_set<uint64_t> consumed;                  // tickets whose result has been handed out: a second wait is an error
    uint64_t next_ticket = 1;
    bool closing = false;
    int callers = 0;                                    // threads inside push or wait (destroy lets them leave first)
    std::condition_variable idle_cv;
    ebrl_queue_stats_t st{};
    std::thread worker;

    void run();
};

// The worker: take what is waiting (after lingering for company), run it, report, repeat.
void ebrl_queue::run()
{
    std::unique_lock<std::mutex> lk(mu);
    for (;;) {
        // wait for work: something waiting, or (step mode) something mid-chunk
        not_empty.wait(lk, [&] { return closing || !waiting.empty() || !in_service.empty(); });
        if (waiting.empty() && in_service.empty()) {
            if (closing) return;
            continue;
        }
        // a group smaller than max_group may wait a little for more arrivals -- but not while
        // environments are mid-chunk (their next step should not be delayed) and not when closing
        if (cfg.linger_us > 0 && in_service.empty() && !closing && (int)waiting.size() < cfg.max_group) {
            const auto until = std::chrono::steady_clock::now() + std::chrono::microseconds(cfg.linger_us);
            not_empty.wait_until(lk, until, [&] { return closing || (int)waiting.size() >= cfg.max_group; });
        }
        // the group: mid-chunk environments first (step mode), then waiting requests in arrival order
        std::vector<Request> group;
        if (cfg.step_mode) {
            group.swap(in_service);
        }
        while (!waiting.empty() && (int)group.size() < cfg.max_group) {
            group.push_back(waiting.front());
            waiting.pop_front();
        }
        st.waiting = (int32_t)waiting.size();
        st.in_service = (int32_t)group.size();
        not_full.notify_all();
        lk.unlock();

        const int n = (int)group.size();
        std::vector<int64_t> ids(n);
        std::vector<const void *> prefix(n);
        std::vector<int32_t> plen(n), sidx(n);
        std::vector<const float *> state(n);
        std::vector<float *> out(n);
        for (int i = 0; i < n; ++i) {
            const Request &r = group[i];
            ids[i] = r.env_id; prefix[i] = r.prefix; plen[i] = r.prefix_len; sidx[i] = r.step;
            state[i] = r.state; out[i] = r.out;
        }
        ebrl_status_t rc = (ebrl_status_t)be.submit(be.ctx, n, ids.data(), prefix.data(), plen.data(), state.data(), out.data(), sidx.data(),
                                     cfg.step_mode ? 1 : 0, cfg.sm_quota, stream);
        const ebrl_status_t rs = (ebrl_status_t)be.sync(be.ctx);   // also after a failed submit: nothing of this group may stay queued in the handle
        if (rc == EBRL_OK) rc = rs;

        lk.lock();
        st.groups += 1;
        st.group_envs += (uint64_t)n;
        for (Request &r : group) {
            bool done = true;
            if (rc == EBRL_OK && cfg.step_mode) {
                r.step += 1;
                r.state = r.out;            // the state continues in the result buffer
                done = r.step >= be.K_steps;
            }
            if (done) {
                finished[r.ticket] = rc;
                live_envs.erase(r.env_id);
                if (rc == EBRL_OK) st.completed += 1; else st.failed += 1;
            } else {
                in_service.push_back(r);
            }
        }
        st.in_service = (int32_t)in_service.size();
        done_cv.notify_all();
    }
}

static ebrl_status_t check_cfg(const ebrl_queue_cfg_t *c)
{
    if (!c || c->capacity < 1 || c->max_group < 1 || c->sm_quota < 0 || (c->step_mode != 0 && c->step_mode != 1))
        return EBRL_ERR_INVALID_ARG;
    return EBRL_OK;
}

extern "C" ebrl_status_t ebrl_queue_create_backend(const ebrl_queue_backend_t *backend, const ebrl_queue_cfg_t *cfg, void *stream,
                                                   ebrl_queue_t *out)
{
    if (out) *out = nullptr;
    if (!out || !backend || !backend->submit || !backend->sync || backend->K_steps < 1 || check_cfg(cfg) != EBRL_OK)
        return EBRL_ERR_INVALID_ARG;
    ebrl_queue *q = new (std::nothrow) ebrl_queue();
    if (!q) return EBRL_ERR_NOMEM;
    q->be = *backend;
    q->cfg = *cfg;
    q->stream = stream;
    try {
        q->worker = std::thread([q] { q->run(); });
    } catch (...) {
        delete q;
        return EBRL_ERR_NOMEM;
    }
    *out = q;
    return EBRL_OK;
}

extern "C" ebrl_status_t ebrl_queue_create(ebrl_actgen_t gen, const ebrl_queue_cfg_t *cfg, void *stream, ebrl_queue_t *out)
{
    if (out) *out = nullptr;
    if (!gen) return EBRL_ERR_INVALID_ARG;
    ebrl_queue_backend_t be{};
    be.ctx = gen;
    be.K_steps = ebrl_actgen_k_steps(gen);
    be.submit = gen_submit;
    be.sync = gen_sync;
    return ebrl_queue_create_backend(&be, cfg, stream, out);
}

static ebrl_status_t push_impl(ebrl_queue *q, bool block, int64_t env_id, const void *prefix_dev, int32_t prefix_len,
                               const float *state_dev, float *out_dev, int32_t step_index, uint64_t *ticket)
{
    if (!q || !ticket || !state_dev || !out_dev || prefix_len < 1 || step_index < 0 || step_index >= q->be.K_steps)
        return EBRL_ERR_INVALID_ARG;
    std::unique_lock<std::mutex> lk(q->mu);
    if (q->closing) return (ebrl_status_t)EBRL_ERR_CLOSED;
    if (q->live_envs.count(env_id)) return EBRL_ERR_ENV_BUSY;
    if ((int)q->waiting.size() >= q->cfg.capacity) {
        if (!block) return (ebrl_status_t)EBRL_ERR_QUEUE_FULL;
        q->st.blocked_pushes += 1;
        q->callers += 1;
        q->not_full.wait(lk, [&] { return q->closing || (int)q->waiting.size() < q->cfg.capacity; });
        q->callers -= 1;
        q->idle_cv.notify_all();
        if (q->closing) return (ebrl_status_t)EBRL_ERR_CLOSED;
        if (q->live_envs.count(env_id)) return EBRL_ERR_ENV_BUSY;
    }
    Request r{q->next_ticket++, env_id, prefix_dev, prefix_len, state_dev, out_dev, step_index};
    q->waiting.push_back(r);
    q->live_envs.insert(env_id);
    q->st.pushed += 1;
    q->st.waiting = (int32_t)q->waiting.size();
    q->st.max_waiting = std::max(q->st.max_waiting, q->st.waiting);
    *ticket = r.ticket;
    q->not_empty.notify_all();
    return EBRL_OK;
}

extern "C" ebrl_status_t ebrl_queue_push(ebrl_queue_t q, int64_t env_id, const void *prefix_dev, int32_t prefix_len,
                                         const float *state_dev, float *out_dev, int32_t step_index, uint64_t *ticket)
{
    return push_impl(q, true, env_id, prefix_dev, prefix_len, state_dev, out_dev, step_index, ticket);
}

extern "C" ebrl_status_t ebrl_queue_try_push(ebrl_queue_t q, int64_t env_id, const void *prefix_dev, int32_t prefix_len,
                                             const float *state_dev, float *out_dev, int32_t step_index, uint64_t *ticket)
{
    return push_impl(q, false, env_id, prefix_dev, prefix_len, state_dev, out_dev, step_index, ticket);
}

extern "C" ebrl_status_t ebrl_queue_wait(ebrl_queue_t q, uint64_t ticket, uint32_t timeout_ms)
{
    if (!q || ticket == 0) return EBRL_ERR_INVALID_ARG;
    std::unique_lock<std::mutex> lk(q->mu);
    if (ticket >= q->next_ticket || q->consumed.count(ticket)) return EBRL_ERR_INVALID_ARG;   // never issued, or already waited for
    auto ready = [&] { return q->finished.count(ticket) != 0 || q->consumed.count(ticket) != 0; };
    q->callers += 1;
    bool got = true;
    if (timeout_ms == 0) q->done_cv.wait(lk, ready);
    else got = q->done_cv.wait_for(lk, std::chrono::milliseconds(timeout_ms), ready);
    q->callers -= 1;
    q->idle_cv.notify_all();
    if (!got) return EBRL_ERR_TIMEOUT;
    auto it = q->finished.find(ticket);
    if (it == q->finished.end()) return EBRL_ERR_INVALID_ARG;      // another waiter on the same ticket took it meanwhile
    const ebrl_status_t rc = it->second;
    q->finished.erase(it);
    q->consumed.insert(ticket);
    q->done_cv.notify_all();      // a second waiter on this ticket must not sleep on
    return rc;
}

extern "C" ebrl_status_t ebrl_queue_get_stats(ebrl_queue_t q, ebrl_queue_stats_t *out)
{
    if (!q || !out) return EBRL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(q->mu);
    *out = q->st;
    out->waiting = (int32_t)q->waiting.size();
    return EBRL_OK;
}

extern "C" ebrl_status_t ebrl_queue_destroy(ebrl_queue_t q)
{
    if (!q) return EBRL_OK;
    {
        std::lock_guard<std::mutex> lk(q->mu);
        q->closing = true;
        q->not_empty.notify_all();
        q->not_full.notify_all();
    }
    if (q->worker.joinable()) q->worker.join();   // serves what was waiting: every accepted request completes
    {
        std::unique_lock<std::mutex> lk(q->mu);
        q->idle_cv.wait(lk, [&] { return q->callers == 0; });   // blocked pushes and waits have left
    }
    delete q;
    return EBRL_OK;
}
