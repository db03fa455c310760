// Driver for the host-only parts of the library (the elastic allocator and the bounded request
// queue) built with AddressSanitizer and UndefinedBehaviorSanitizer: the stand-in, on the host side,
// for a memory checker.  tests/test_host_sanitizers.py compiles this file together with the two
// sources as plain C++ and runs it; any sanitizer report aborts the run with a non-zero status.
// The generation handle's entry points the queue's default backend refers to are stubbed out
// here: the queue is driven through a recording backend, as in the Python queue tests.
#include "../include/ebrl_alloc.h"
#include "../include/ebrl_queue.h"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <thread>
#include <vector>

extern "C" {
ebrl_status_t ebrl_actgen_submit_scattered(ebrl_actgen_t, int32_t, const int64_t *, const void *const *, const float *const *,
                                           float *const *, int32_t, void *, const ebrl_submit_ext_t *) { return EBRL_ERR_UNSUPPORTED; }
ebrl_status_t ebrl_actgen_sync(ebrl_actgen_t) { return EBRL_ERR_UNSUPPORTED; }
int32_t ebrl_actgen_k_steps(ebrl_actgen_t) { return 0; }
}

#define CHECK(cond) do { if (!(cond)) { std::fprintf(stderr, "CHECK failed at line %d: %s\n", __LINE__, #cond); std::exit(2); } } while (0)

namespace {

struct Recorder {
    std::mutex mu;
    std::vector<std::vector<int64_t>> groups;
    std::atomic<int> syncs{0};
};
int32_t rec_submit(void *ctx, int32_t n, const int64_t *env_ids, const void *const *, const int32_t *, const float *const *state,
                   float *const *out, const int32_t *step_index, int32_t, int32_t, void *)
{
    Recorder *r = (Recorder *)ctx;
    std::lock_guard<std::mutex> lk(r->mu);
    r->groups.emplace_back(env_ids, env_ids + n);
    for (int i = 0; i < n; ++i) *out[i] = *state[i] + 1.0f + (float)step_index[i];   // touch every pointer the queue handed over
    return EBRL_OK;
}
int32_t rec_sync(void *ctx) { ((Recorder *)ctx)->syncs++; return EBRL_OK; }

void allocator_cases()
{
    const int32_t q4[4] = {20, 40, 60, 80}, b2[2] = {8, 32}, sq[3] = {10, 20, 30};
    const double gen_rate[8] = {10, 14, 20, 28, 30, 42, 40, 56}, tr_rate[8] = {5, 8, 10, 16, 15, 24, 20, 32};
    const double mem[2] = {10, 30}, sim[3] = {50, 99, 100};
    ebrl_alloc_in_t in{};
    in.cores = 64; in.cores_per_env = 2; in.n_sim_quota = 3; in.sim_quota_pct = sq; in.sim_rate = sim; in.knee_tolerance = 0.05;
    in.gen = ebrl_profile_t{4, 2, q4, b2, gen_rate, mem};
    in.train = ebrl_profile_t{4, 2, q4, b2, tr_rate, mem};
    in.s_g_min = 5; in.s_t_min = 5; in.mem_gpu_gb = 45;
    ebrl_alloc_out_t out{};
    CHECK(ebrl_alloc_elastic(&in, &out) == 0);
    CHECK(out.env_concurrency == 32 && out.s_sim == 20 && out.s_g + out.s_t + out.s_sim == 100 && out.theta > 0);
    CHECK(ebrl_profile_rate(&in.gen, 30, 1) == 21.0 && ebrl_profile_rate(&in.gen, 5, 0) == 10.0 && ebrl_profile_rate(&in.gen, 99, 1) == 56.0);
    CHECK(ebrl_profile_rate(&in.gen, 30, 7) == 0.0);                   // batch index out of range
    // tables without a knee: all rates negative, zero, or not a number
    const double neg[3] = {-1, -2, -3}, zero[3] = {0, 0, 0}, nan3[3] = {NAN, 1, 2};
    in.sim_rate = neg;  CHECK(ebrl_alloc_elastic(&in, &out) == 1);
    in.sim_rate = zero; CHECK(ebrl_alloc_elastic(&in, &out) == 1);
    in.sim_rate = nan3; CHECK(ebrl_alloc_elastic(&in, &out) == 1);
    in.sim_rate = sim;
    in.mem_gpu_gb = 1;  CHECK(ebrl_alloc_elastic(&in, &out) == 1);     // nothing fits
    in.mem_gpu_gb = 45;
    in.s_g_min = 90;    CHECK(ebrl_alloc_elastic(&in, &out) == 1);     // empty interval
    CHECK(ebrl_alloc_elastic(nullptr, &out) == 1 && ebrl_alloc_elastic(&in, nullptr) == 1);
    ebrl_rebalance_t rb = ebrl_rebalance_create(0, 0, 0.0);
    int fired = 0;
    for (int i = 0; i < 100; ++i) fired += ebrl_rebalance_push(rb, 100.0, 50.0);
    CHECK(fired >= 2);
    double a = 0, b = 0; int32_t streak = 0;
    ebrl_rebalance_get(rb, &a, &b, &streak);
    CHECK(a == 100.0 && b == 50.0);
    ebrl_rebalance_destroy(rb);
    CHECK(ebrl_rebalance_push(nullptr, 1, 1) == -1);
}

void queue_cases(int step_mode)
{
    Recorder rec;
    ebrl_queue_backend_t be{&rec, 4, rec_submit, rec_sync};
    ebrl_queue_cfg_t cfg{8, 4, 0, step_mode, 200, 0};
    ebrl_queue_t q = nullptr;
    CHECK(ebrl_queue_create_backend(&be, &cfg, nullptr, &q) == EBRL_OK && q);
    const int threads = 4, per_thread = 25;
    std::vector<float> state(threads * per_thread, 1.0f), out(threads * per_thread, 0.0f);
    std::vector<std::thread> th;
    for (int t = 0; t < threads; ++t)
        th.emplace_back([&, t] {
            for (int i = 0; i < per_thread; ++i) {
                const int k = t * per_thread + i;
                uint64_t ticket = 0;
                CHECK(ebrl_queue_push(q, 1000 + k, &state[k], 1, &state[k], &out[k], 0, &ticket) == EBRL_OK);
                CHECK(ebrl_queue_wait(q, ticket, 0) == EBRL_OK);
                CHECK(ebrl_queue_wait(q, ticket, 10) == EBRL_ERR_INVALID_ARG);   // a ticket is handed out once
            }
        });
    for (auto &t : th) t.join();
    ebrl_queue_stats_t st{};
    CHECK(ebrl_queue_get_stats(q, &st) == EBRL_OK && st.completed == (uint64_t)threads * per_thread && st.failed == 0);
    for (float v : out) CHECK(v >= 2.0f);
    uint64_t t1 = 0, t2 = 0;
    CHECK(ebrl_queue_push(q, 7, &state[0], 1, &state[0], &out[0], 0, &t1) == EBRL_OK);
    const ebrl_status_t dup = ebrl_queue_try_push(q, 7, &state[0], 1, &state[0], &out[0], 0, &t2);
    CHECK(dup == EBRL_OK || dup == EBRL_ERR_ENV_BUSY);                  // busy while the first is queued or in service
    CHECK(ebrl_queue_wait(q, t1, 0) == EBRL_OK);
    if (dup == EBRL_OK) CHECK(ebrl_queue_wait(q, t2, 0) == EBRL_OK);
    CHECK(ebrl_queue_wait(q, 123456, 0) == EBRL_ERR_INVALID_ARG);
    CHECK(ebrl_queue_destroy(q) == EBRL_OK);
    CHECK(ebrl_queue_create_backend(nullptr, &cfg, nullptr, &q) == EBRL_ERR_INVALID_ARG);
}

}  // namespace

int main()
{
    allocator_cases();
    queue_cases(0);
    queue_cases(1);
    std::puts("host sanitizer driver: ok");
    return 0;
}
