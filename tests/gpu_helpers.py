"""Helpers of the GPU tests: run the library through the C-ABI binding on seeded inputs."""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from paper_2609_27547_b200 import binding as B
from paper_2609_27547_b200 import synth

TOL = {"f32": 1e-4, "bf16": 2e-2}   # max chunk-relative error against the fp64 oracle


def to_dev(wt: dict, device="cuda") -> dict:
    out = {k: (v.to(device) if torch.is_tensor(v) else v) for k, v in wt.items() if k != "layers"}
    out["layers"] = [{k: v.to(device) for k, v in l.items()} for l in wt["layers"]]
    return out


class Runner:
    """Holds a handle plus device copies of the environments' inputs."""

    def __init__(self, w: synth.Workload, wt: dict, envs: Sequence[synth.EnvInputs], *, flags: int = 0,
                 max_inflight_groups: int = 2, max_group_envs: Optional[int] = None):
        self.w = w
        self.envs = {e.env_id: e for e in envs}
        self.kv = {e.env_id: e.kv.cuda().contiguous() for e in envs}
        self.noise = {e.env_id: e.noise.cuda().contiguous() for e in envs}
        cfg = B.cfg_for(w, max_group_envs=max_group_envs or len(envs), max_inflight_groups=max_inflight_groups, flags=flags)
        cfg.max_prefix_len = max([w.P[1]] + [e.P for e in envs])
        self.gen = B.ActGen(cfg, wt)

    def run(self, groups: List[List[int]], quota: int = 0, n_steps: int = 0, state=None, steps=None,
            stream=None) -> dict:
        """Submits the groups (lists of env ids) and returns {env_id: float32 [H][A]}."""
        outs = []
        for g in groups:
            noise = torch.stack([(state[e] if state is not None else self.noise[e]) for e in g]) if g else \
                torch.zeros((0, self.w.H, self.w.A), device="cuda")
            out = torch.empty_like(noise)
            sidx = [(steps[e] if steps is not None else self.envs[e].step) for e in g]
            self.gen.submit(g, [self.kv[e] for e in g], noise, out, sm_quota=quota, step_index=sidx,
                            n_steps=n_steps, stream=stream)
            outs.append((g, noise, out))
        self.gen.sync()
        res = {}
        for g, _, out in outs:
            o = out.cpu().numpy()
            for i, e in enumerate(g):
                res[e] = o[i]
        return res

    def close(self):
        self.gen.destroy()


def stack(res: dict, ids: Sequence[int]) -> np.ndarray:
    return np.stack([res[e] for e in ids])
