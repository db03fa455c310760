"""Oracle of the elastic resource allocator (TEST INFRASTRUCTURE ONLY).

Plain Python restatement of the paper's Algorithm 1 and Eq. 2 (section 4.3.2), in the paper's
order and notation: fix the simulator's capacity at its knee quota, then bisect the generation
quota s_g between s_g^min and 100 - s_sim* - s_t^min, at each midpoint giving the rest to
training, choosing the best feasible batch-size pair under M_gpu, and moving toward the slower
of rollout (T_r = min(T_s, P_gen)) and training (T_t); finally take the better endpoint by
Theta = min(T_r, T_t).  `brute_force` evaluates Theta at every integer quota instead.  Shares no
code with the library's implementation.

Readings (the paper leaves them open): table lookups between grid quotas are linear in the quota
and constant outside the grid; the knee is the smallest grid quota within `knee_tolerance` of the
table's maximum; the best pair maximises Theta, first found wins ties (generation batch outer
loop, training batch inner loop, both ascending).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence


@dataclass
class Profile:
    quota_pct: Sequence[int]
    batch: Sequence[int]
    rate: Sequence[Sequence[float]]     # [quota][batch]
    mem_gb: Sequence[float]             # [batch]

    def at(self, s: int, j: int) -> float:
        q = self.quota_pct
        if s <= q[0]:
            return self.rate[0][j]
        if s >= q[-1]:
            return self.rate[-1][j]
        i = 1
        while q[i] < s:
            i += 1
        w = (s - q[i - 1]) / (q[i] - q[i - 1])
        return self.rate[i - 1][j] * (1.0 - w) + self.rate[i][j] * w


def theta(T_s: float, T_g: float, T_t: float):
    """Eq. 2."""
    T_r = min(T_s, T_g)
    return T_r, min(T_r, T_t)


def best_pair(gen: Profile, train: Profile, s_g: int, s_t: int, T_s: float, M_gpu: float):
    best = None
    for jg in range(len(gen.batch)):
        for jt in range(len(train.batch)):
            if gen.mem_gb[jg] + train.mem_gb[jt] > M_gpu:
                continue
            T_g, T_t = gen.at(s_g, jg), train.at(s_t, jt)
            T_r, th = theta(T_s, T_g, T_t)
            if best is None or th > best["theta"]:
                best = dict(s_g=s_g, s_t=s_t, B_g=gen.batch[jg], B_t=train.batch[jt], T_g=T_g, T_t=T_t, T_r=T_r, theta=th)
    return best


def simulator_capacity(sim_quota_pct, sim_rate, knee_tolerance):
    peak = max(sim_rate)
    for q, r in zip(sim_quota_pct, sim_rate):
        if r >= (1.0 - knee_tolerance) * peak:
            return q, r
    raise AssertionError


def elastic_allocation(N, c_env, sim_quota_pct, sim_rate, gen: Profile, train: Profile, s_g_min, s_t_min, M_gpu,
                       knee_tolerance=0.05):
    E = N // c_env
    s_sim, T_s = simulator_capacity(sim_quota_pct, sim_rate, knee_tolerance)
    lo, hi = s_g_min, 100 - s_sim - s_t_min
    assert hi >= lo
    it = 0
    while hi - lo > 1:
        s_g = (lo + hi) // 2
        s_t = 100 - s_sim - s_g
        c = best_pair(gen, train, s_g, s_t, T_s, M_gpu)
        if c["T_r"] > c["T_t"]:
            hi = s_g
        else:
            lo = s_g
        it += 1
    a = best_pair(gen, train, lo, 100 - s_sim - lo, T_s, M_gpu)
    b = best_pair(gen, train, hi, 100 - s_sim - hi, T_s, M_gpu)
    w = a if a["theta"] >= b["theta"] else b
    w.update(E=E, s_sim=s_sim, T_s=T_s, iterations=it)
    return w


def brute_force(sim_quota_pct, sim_rate, gen, train, s_g_min, s_t_min, M_gpu, knee_tolerance=0.05):
    s_sim, T_s = simulator_capacity(sim_quota_pct, sim_rate, knee_tolerance)
    best = None
    for s_g in range(s_g_min, 100 - s_sim - s_t_min + 1):
        c = best_pair(gen, train, s_g, 100 - s_sim - s_g, T_s, M_gpu)
        if c is not None and (best is None or c["theta"] > best["theta"]):
            best = c
    return best


def rebalance_trigger(rollout: List[float], train: List[float], window=20, streak=20, threshold=0.15) -> List[int]:
    """Section 4.3.2, runtime adaptation: per step, 1 when the gap of the `window`-step moving
    averages has exceeded `threshold` of the faster stage for `streak` consecutive steps."""
    out, run = [], 0
    for i in range(len(rollout)):
        lo = max(0, i + 1 - window)
        a = sum(rollout[lo:i + 1]) / (i + 1 - lo)
        b = sum(train[lo:i + 1]) / (i + 1 - lo)
        faster = max(a, b)
        run = run + 1 if faster > 0 and (faster - min(a, b)) > threshold * faster else 0
        if run >= streak:
            out.append(1)
            run = 0
        else:
            out.append(0)
    return out
