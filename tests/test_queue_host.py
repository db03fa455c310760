"""Host-only tests of the bounded request queue (paper section 4.2.2: bounded producer-consumer
queue between simulation and generation; section 4.2.3: step-level continuous batching), run
against a recording backend instead of a GPU handle."""
import ctypes as C
import threading
import time

from paper_2609_27547_b200 import binding as B


class FakeBackend:
    """Records every submit; sync optionally sleeps or blocks on an event; can be told to fail."""

    def __init__(self, K=4, sync_sleep=0.0):
        self.K = K
        self.groups = []           # list of dicts
        self.sync_sleep = sync_sleep
        self.gate = None           # threading.Event the sync waits for
        self.fail_submit_at = None
        self.lock = threading.Lock()

        def submit(ctx, n, ids, prefix, plen, state, out, sidx, n_steps, quota, stream):
            with self.lock:
                g = {"ids": [ids[i] for i in range(n)], "plen": [plen[i] for i in range(n)],
                     "state": [state[i] for i in range(n)], "out": [out[i] for i in range(n)],
                     "step": [sidx[i] for i in range(n)], "n_steps": n_steps, "quota": quota}
                self.groups.append(g)
                if self.fail_submit_at is not None and len(self.groups) - 1 == self.fail_submit_at:
                    return B.ERR_CUDA
            return B.OK

        def sync(ctx):
            if self.gate is not None:
                self.gate.wait(10.0)
            if self.sync_sleep:
                time.sleep(self.sync_sleep)
            return B.OK

        self._submit, self._sync = B.QUEUE_SUBMIT_FN(submit), B.QUEUE_SYNC_FN(sync)
        self.struct = B.QueueBackend(None, K, self._submit, self._sync)


def _addr(env, what):
    return 0x100000 + env * 0x100 + {"prefix": 0, "state": 16, "out": 32}[what]


def _push(q, env, step=0, plen=5):
    return q.push(env, _addr(env, "prefix"), plen, _addr(env, "state"), _addr(env, "out"), step)


def test_groups_respect_arrival_order_group_size_and_the_bound():
    be = FakeBackend(sync_sleep=0.03)
    q = B.Queue(None, capacity=4, max_group=3, sm_quota=37, backend=be.struct)
    tickets = {}

    def producer(lo, hi):
        for e in range(lo, hi):
            tickets[e] = _push(q, e)

    th = [threading.Thread(target=producer, args=(0, 10)), threading.Thread(target=producer, args=(100, 110))]
    for t in th:
        t.start()
    for t in th:
        t.join()
    for e, t in tickets.items():
        assert q.wait(t) == B.OK
    st = q.stats()
    assert st["pushed"] == st["completed"] == 20 and st["failed"] == 0
    assert st["max_waiting"] <= 4 and st["blocked_pushes"] > 0          # the bound held and pushed back
    assert st["groups"] == len(be.groups) and st["group_envs"] == 20
    served = [e for g in be.groups for e in g["ids"]]
    assert sorted(served) == sorted(tickets)
    assert all(1 <= len(g["ids"]) <= 3 and g["n_steps"] == 0 and g["quota"] == 37 for g in be.groups)
    for lo in (0, 100):                                                  # each producer's requests are served in its order
        mine = [e for e in served if lo <= e < lo + 10]
        assert mine == sorted(mine)
    g0 = be.groups[0]
    e = g0["ids"][0]
    assert g0["state"][0] == _addr(e, "state") and g0["out"][0] == _addr(e, "out") and g0["plen"][0] == 5
    q.destroy()


def test_try_push_reports_a_full_queue_and_linger_collects_a_group():
    be = FakeBackend()
    be.gate = threading.Event()
    q = B.Queue(None, capacity=2, max_group=8, backend=be.struct)
    t0 = _push(q, 0)                       # taken by the worker at once, which then blocks in sync
    deadline = time.time() + 5
    while q.stats()["waiting"] != 0 and time.time() < deadline:
        time.sleep(0.001)
    st1, t1 = q.try_push(1, _addr(1, "prefix"), 3, _addr(1, "state"), _addr(1, "out"))
    st2, t2 = q.try_push(2, _addr(2, "prefix"), 3, _addr(2, "state"), _addr(2, "out"))
    st3, _ = q.try_push(3, _addr(3, "prefix"), 3, _addr(3, "state"), _addr(3, "out"))
    assert (st1, st2, st3) == (B.OK, B.OK, B.ERR_QUEUE_FULL)
    assert q.wait(t1, timeout_ms=50) == 7  # EBRL_ERR_TIMEOUT: generation is stuck
    be.gate.set()
    assert q.wait(t0) == B.OK and q.wait(t1) == B.OK and q.wait(t2) == B.OK
    assert [g["ids"] for g in be.groups] == [[0], [1, 2]]                # what piled up behind the busy worker forms one group
    q.destroy()
    # linger: the worker waits for company before launching a small group
    be2 = FakeBackend()
    q2 = B.Queue(None, capacity=8, max_group=4, linger_us=300000, backend=be2.struct)
    ts = [_push(q2, e) for e in range(4)]                                # the fourth arrival fills the group: no need to wait out the linger
    t_start = time.time()
    for t in ts:
        assert q2.wait(t) == B.OK
    assert time.time() - t_start < 0.25
    assert [g["ids"] for g in be2.groups] == [[0, 1, 2, 3]]
    q2.destroy()


def test_step_mode_is_continuous_batching():
    """Every Euler step is its own submit; an environment that arrives while others are mid-chunk
    joins the very next step; the state moves into the result buffer after the first step."""
    be = FakeBackend(K=4)
    be.gate = threading.Event()
    q = B.Queue(None, capacity=8, max_group=4, step_mode=True, backend=be.struct)
    ta = _push(q, 10)                          # step 0 of env 10 is submitted; the worker blocks in sync
    deadline = time.time() + 5
    while not be.groups and time.time() < deadline:
        time.sleep(0.001)
    tb = _push(q, 11, step=2)                  # arrives mid-chunk, already at Euler step 2
    be.gate.set()
    assert q.wait(ta) == B.OK and q.wait(tb) == B.OK
    assert all(g["n_steps"] == 1 for g in be.groups)
    seen = {10: [], 11: []}
    for g in be.groups:
        for e, s in zip(g["ids"], g["step"]):
            seen[e].append(s)
    assert seen[10] == [0, 1, 2, 3] and seen[11] == [2, 3]
    assert be.groups[1]["ids"] == [10, 11] and be.groups[1]["step"] == [1, 2]     # joined at the next step, mid-chunk env first
    first, later = be.groups[0], be.groups[1]
    assert first["state"][0] == _addr(10, "state") and later["state"][0] == _addr(10, "out") == later["out"][0]
    st = q.stats()
    assert st["groups"] == 4 and st["group_envs"] == 6 and st["completed"] == 2
    q.destroy()


def test_errors_busy_ids_invalid_arguments_and_failures():
    be = FakeBackend(K=3)
    be.gate = threading.Event()
    q = B.Queue(None, capacity=4, max_group=2, backend=be.struct)
    t0 = _push(q, 5)
    st, _ = q.try_push(5, 1, 1, 2, 3)
    assert st == B.ERR_ENV_BUSY                                           # one request per environment at a time
    assert q.try_push(6, 1, 0, 2, 3)[0] == B.ERR_INVALID_ARG              # prefix_len < 1
    assert q.try_push(6, 1, 1, 0, 3)[0] == B.ERR_INVALID_ARG              # NULL state
    assert q.try_push(6, 1, 1, 2, 3, step_index=3)[0] == B.ERR_INVALID_ARG   # step index outside [0, K)
    assert q.wait(12345) == B.ERR_INVALID_ARG                             # a ticket never issued
    be.gate.set()
    assert q.wait(t0) == B.OK
    t1 = _push(q, 5)                                                      # the id is free again
    assert q.wait(t1) == B.OK
    be.fail_submit_at = len(be.groups)
    t2 = _push(q, 7)
    assert q.wait(t2) == B.ERR_CUDA and q.stats()["failed"] == 1          # the backend's status reaches the waiter
    t3 = _push(q, 7)
    assert q.wait(t3) == B.OK                                             # and the queue keeps serving
    q.destroy()
    bad = B.QueueBackend(None, 0, be._submit, be._sync)
    h = C.c_void_p()
    assert B.lib().ebrl_queue_create_backend(C.byref(bad), C.byref(B.QueueCfg(1, 1, 0, 0, 0, 0)), None, C.byref(h)) == B.ERR_INVALID_ARG
    assert B.lib().ebrl_queue_create_backend(C.byref(be.struct), C.byref(B.QueueCfg(0, 1, 0, 0, 0, 0)), None, C.byref(h)) == B.ERR_INVALID_ARG
    assert B.lib().ebrl_queue_create(None, C.byref(B.QueueCfg(1, 1, 0, 0, 0, 0)), None, C.byref(h)) == B.ERR_INVALID_ARG


def test_destroy_serves_what_is_waiting():
    be = FakeBackend(sync_sleep=0.02)
    q = B.Queue(None, capacity=2, max_group=1, backend=be.struct)
    for e in range(3):
        _push(q, e)
    blocked = []
    th = threading.Thread(target=lambda: blocked.append(q.try_push(50, 1, 1, 2, 3)[0]))
    th.start()
    th.join()
    assert blocked == [B.ERR_QUEUE_FULL]
    q.destroy()                                                           # returns only after the three requests ran
    assert sorted(e for g in be.groups for e in g["ids"]) == [0, 1, 2]


def test_a_ticket_can_be_waited_for_once():
    """The result of a ticket is handed out once: a second wait on it (with or without a timeout)
    is an argument error instead of a wait that can never end, and destroy still returns."""
    be = FakeBackend()
    q = B.Queue(None, capacity=4, max_group=2, backend=be.struct)
    t = _push(q, 1)
    assert q.wait(t) == B.OK
    assert q.wait(t) == B.ERR_INVALID_ARG
    assert q.wait(t, timeout_ms=50) == B.ERR_INVALID_ARG
    assert q.wait(t + 100) == B.ERR_INVALID_ARG                          # never issued
    q.destroy()
