"""Rollout-side harness around the generation library: a bounded ready queue fed by environments
whose simulator steps take a seeded, variable time (paper section 4.2.2: simulation and
generation are pipelined across environment groups through a bounded producer-consumer queue;
section 4.2.3: environments advance independently), with two serving policies:

* ``chunk``  -- group-level batching: the ready environments are taken as one group and each is
  run from noise to its final action chunk in one submit;
* ``step``   -- step-level continuous batching: every Euler step is its own submit
  (``n_steps = 1``), so environments that become ready while others are mid-chunk join the very
  next step instead of waiting for the running group to finish.

Simulator time is virtual (drawn from the latency model); generation time is the real device time
of each submit, measured with CUDA events and added to the virtual clock.  The result of every
chunk is checked by the caller against a direct run: batching policy must not change a bit.

The latency model has the shape the paper reports for its simulators (mean 40 ms, P99 60 ms per
step; section 3.1): a log-normal with those two moments, drawn from the counter-based generator.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List

import torch

from . import binding as B
from . import synth

# log-normal with mean 40 ms and 99th percentile 60 ms: sigma solves ln(60/40) = 2.3263 s - s^2 / 2
SIM_SIGMA = 0.18145
SIM_MU = math.log(40.0) - 0.5 * SIM_SIGMA ** 2


def sim_latency_ms(seed: int, env: int, visit: int, steps_per_chunk: int) -> float:
    """Virtual time an environment spends executing one action chunk: ``steps_per_chunk`` simulator steps."""
    z = synth.normal(seed, "sim_latency", env, (visit + 1, steps_per_chunk))[visit].double()
    return float(torch.exp(SIM_MU + SIM_SIGMA * z).sum())


@dataclass
class RolloutResult:
    policy: str
    chunks: int
    makespan_ms: float
    latency_ms: List[float] = field(default_factory=list)     # ready -> chunk delivered
    gen_busy_ms: float = 0.0
    submits: int = 0
    outputs: Dict[tuple, torch.Tensor] = field(default_factory=dict)   # (env, visit) -> chunk

    def summary(self) -> dict:
        lat = sorted(self.latency_ms)
        pick = lambda q: lat[min(len(lat) - 1, int(q * len(lat)))]
        return {"policy": self.policy, "chunks": self.chunks, "chunks_per_s": 1e3 * self.chunks / self.makespan_ms,
                "latency_ms": {"avg": sum(lat) / len(lat), "p50": pick(0.5), "p99": pick(0.99)},
                "generation_busy_frac": self.gen_busy_ms / self.makespan_ms, "submits": self.submits}


def run(w: synth.Workload, weights: dict, n_envs: int, chunks_per_env: int, policy: str, *, seed: int = synth.DEFAULT_SEED,
        quota: int = 0, max_group: int = 64, sim_steps_per_chunk: int = 1, keep_outputs: bool = False) -> RolloutResult:
    """Event-driven rollout of ``n_envs`` environments, ``chunks_per_env`` action chunks each."""
    assert policy in ("chunk", "step")
    dev = torch.device("cuda", torch.cuda.current_device())
    cfg = B.cfg_for(w, max_group_envs=max_group, max_inflight_groups=1, device=dev.index)
    gen = B.ActGen(cfg, weights)
    stream = torch.cuda.Stream(dev)
    envs = [synth.make_env(synth.scaled(w, mixed_steps=False), e, seed, device=dev) for e in range(n_envs)]
    res = RolloutResult(policy, 0, 0.0)
    now = 0.0
    visit = [0] * n_envs
    # every environment starts in its simulator
    arrive = {e: sim_latency_ms(seed, e, 0, sim_steps_per_chunk) for e in range(n_envs)}   # env -> virtual time it becomes ready
    ready_since: Dict[int, float] = {}
    state: Dict[int, torch.Tensor] = {}     # env -> action state (step policy)
    step_of: Dict[int, int] = {}

    def fresh_noise(e):
        return synth.normal(seed, "noise_visit%d" % visit[e], e, (w.H, w.A), device=dev)

    def timed_submit(ids, noise, out, sidx, n_steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        gen.submit([e * 1000003 + visit[e] for e in ids], [envs[e].kv for e in ids], noise, out, sm_quota=quota, stream=stream,
                   step_index=sidx, n_steps=n_steps)
        gen.sync()
        e1.record(stream)
        e1.synchronize()
        res.submits += 1
        return e0.elapsed_time(e1)

    def deliver(e, chunk, t):
        res.latency_ms.append(t - ready_since.pop(e))
        if keep_outputs:
            res.outputs[(e, visit[e])] = chunk.clone()
        res.chunks += 1
        visit[e] += 1
        if visit[e] < chunks_per_env:
            arrive[e] = t + sim_latency_ms(seed, e, visit[e], sim_steps_per_chunk)

    in_service: List[int] = []
    while res.chunks < n_envs * chunks_per_env:
        # environments whose simulator step has finished join the ready set
        for e in [e for e, t in arrive.items() if t <= now]:
            ready_since[e] = arrive.pop(e)
        if policy == "chunk":
            group = sorted(ready_since, key=lambda e: ready_since[e])[:max_group]
            if not group:
                now = min(arrive.values())
                continue
            noise = torch.stack([fresh_noise(e) for e in group])
            out = torch.empty_like(noise)
            ms = timed_submit(group, noise, out, [0] * len(group), 0)
            now += ms
            res.gen_busy_ms += ms
            for i, e in enumerate(group):
                deliver(e, out[i], now)
        else:
            # admit ready environments into the running set (bounded by max_group), then advance everyone one Euler step
            for e in sorted(ready_since, key=lambda e: ready_since[e]):
                if e not in step_of and len(in_service) < max_group:
                    in_service.append(e)
                    step_of[e] = 0
                    state[e] = fresh_noise(e)
            if not in_service:
                now = min(arrive.values())
                continue
            noise = torch.stack([state[e] for e in in_service])
            out = torch.empty_like(noise)
            ms = timed_submit(in_service, noise, out, [step_of[e] for e in in_service], 1)
            now += ms
            res.gen_busy_ms += ms
            still = []
            for i, e in enumerate(in_service):
                step_of[e] += 1
                if step_of[e] == w.K:
                    del step_of[e], state[e]
                    deliver(e, out[i], now)
                else:
                    state[e] = out[i].clone()
                    still.append(e)
            in_service = still
    res.makespan_ms = now
    gen.destroy()
    return res
