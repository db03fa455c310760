"""Seeded synthetic inputs for batched action generation.

This module only *draws numbers and shapes*: it contains none of the method's arithmetic and is
the one module that both the CUDA path's tests/bench and the CPU oracle's tests may use.

The paper evaluates on simulator suites with pretrained policies; none of that is available or
needed here.  These inputs stand in for it and take only the workload's shapes: action chunks
of 8 or 16 actions of 7 (single-arm) or 14 (bimanual) dimensions (section 2.1), hundreds to
thousands of concurrent environments arriving in groups (section 4.2.2), SM quotas from an
allocator's grid (section 4.3).

Every value is a pure function of (seed, tensor tag, environment id, element index) through a
counter-based generator (splitmix64 -> Box-Muller in fp64 -> one rounding to the stored dtype),
so an environment's inputs do not depend on which group it arrives in.  The generator is
written with torch integer ops and runs on CPU or CUDA tensors alike; the two devices may
differ in the last bit of a transcendental, so a test that needs identical bits on both sides
draws once and copies.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Tuple

import torch

DEFAULT_SEED = 20260927

_M64 = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _s64(x: int) -> int:
    """Unsigned 64-bit value -> the int64 with the same bits."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _splitmix_scalar(x: int) -> int:
    x = (x + _GOLD) & _M64
    z = x
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, tag: str, env: int = 0) -> int:
    """64-bit key of one tensor's random stream."""
    k = _splitmix_scalar(seed & _M64)
    for ch in tag.encode():
        k = _splitmix_scalar(k ^ ch)
    return _splitmix_scalar(k ^ ((env * 0xD1342543DE82EF95) & _M64))


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def _splitmix_tensor(ctr: torch.Tensor, key: int) -> torch.Tensor:
    """splitmix64 finaliser of (key + (ctr+1)*GOLD) on int64 tensors (wrapping arithmetic)."""
    z = ctr * _s64(_GOLD) + _s64((key + _GOLD) & _M64)
    z = (z ^ _lsr(z, 30)) * _s64(_C1)
    z = (z ^ _lsr(z, 27)) * _s64(_C2)
    return z ^ _lsr(z, 31)


def uniform_int(seed: int, tag: str, env: int, lo: int, hi: int, index: int = 0) -> int:
    """One integer uniform on lo..hi inclusive (scalar, exact on any device)."""
    z = _splitmix_scalar((stream_key(seed, tag, env) + index * _GOLD) & _M64)
    return lo + (z % (hi - lo + 1))


def normal(seed: int, tag: str, env: int, shape, *, std: float = 1.0, mean: float = 0.0,
           dtype=torch.float32, device="cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """N(mean, std^2) samples of the given shape, rounded once (RNE) to ``dtype``."""
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=dtype, device=device)
    key = stream_key(seed, tag, env)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        i = torch.arange(lo, hi, dtype=torch.int64, device=device)
        z1 = _splitmix_tensor(2 * i, key)
        z2 = _splitmix_tensor(2 * i + 1, key)
        u1 = (_lsr(z1, 11).to(torch.float64) + 1.0) * (1.0 / 9007199254740992.0)   # (0, 1]
        u2 = _lsr(z2, 11).to(torch.float64) * (1.0 / 9007199254740992.0)           # [0, 1)
        g = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        out[lo:hi] = (g * std + mean).to(torch.float32).to(dtype)
    return out.reshape(*shape)


# --------------------------------------------------------------------------------------------
# Workload shapes (the benchmark's five configurations)
# --------------------------------------------------------------------------------------------

@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str                  # "f32" or "bf16": matrices and prefix planes
    B: int                      # environments
    H: int
    A: int
    d: int
    L: int
    n_heads: int
    K: int
    P: Tuple[int, int]          # prefix length range (lo, hi), inclusive
    group: Optional[Tuple[int, int]]   # arrival group size range; None = one group
    quota: int                  # SM quota the configuration names (0 = all)
    mixed_steps: bool = False   # environments start at independent Euler steps
    mlp_mult: int = 4
    d_ctx: int = 0              # > 0: prefixes are hidden states [P][d_ctx], projected to K/V per layer

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def head_dim(self) -> int:
        return self.d // self.n_heads

    def flops_per_env_step(self, P: float) -> float:
        """2*m*n*k FLOPs of one Euler step of one environment with prefix length P."""
        H, A, d, L = self.H, self.A, self.d, self.L
        proj = (3 + 1 + 1 + 1 + 2 * self.mlp_mult) * 2 * H * d * d
        return L * (proj + 4 * H * P * d + 4 * H * H * d) + 4 * H * A * d


WORKLOADS: Dict[int, Workload] = {
    0: Workload("cfg0_tiny_f32", "f32", 16, 8, 7, 256, 2, 4, 4, (32, 32), None, 0),
    1: Workload("cfg1_mid_bf16", "bf16", 256, 8, 7, 1024, 4, 16, 10, (256, 256), None, 0),
    2: Workload("cfg2_ragged_f32", "f32", 512, 8, 7, 256, 2, 4, 4, (64, 512), (1, 64), 0,
                mixed_steps=True),
    3: Workload("cfg3_quota_sweep_f32", "f32", 1024, 8, 7, 256, 2, 4, 4, (256, 256), None, 0),
    4: Workload("cfg4_large_bf16", "bf16", 2048, 16, 14, 2048, 8, 16, 10, (768, 768), (32, 256), 74),
    # The other reading of "the config-1 model" in configurations 2 and 3 (counting from zero: the
    # bf16 mid-size head of WORKLOADS[1] instead of the tiny fp32 one); same arrivals and quotas.
    12: Workload("cfg2_ragged_mid_bf16", "bf16", 512, 8, 7, 1024, 4, 16, 10, (64, 512), (1, 64), 0,
                 mixed_steps=True),
    13: Workload("cfg3_quota_sweep_mid_bf16", "bf16", 1024, 8, 7, 1024, 4, 16, 10, (256, 256), None, 0),
}


def workload_label(i: int) -> str:
    """The name a result line carries: ``configs[i] <name>`` (12 and 13 are configurations 2 and 3 on
    the WORKLOADS[1] model)."""
    w = WORKLOADS[i]
    return "configs[%d] %s" % (i - 10, w.name) if i >= 10 else "configs[%d] %s" % (i, w.name)


def scaled(w: Workload, **kw) -> Workload:
    """A smaller or altered copy of a workload (parity-test sizes)."""
    return replace(w, **kw)


def make_weights(w: Workload, seed: int = DEFAULT_SEED, device="cpu", random_gains: bool = False
                 ) -> dict:
    """Matrices ~ N(0, 1/fan_in) in the workload's dtype; gains 1 (or 1 + 0.1 N(0,1));
    b_out ~ 0.1 N(0,1).  Gains and b_out are fp32.  Matrices are [out][in]."""
    dt, d, A, md = w.torch_dtype, w.d, w.A, w.mlp_mult * w.d

    def mat(tag, n_out, n_in, env=0):
        return normal(seed, tag, env, (n_out, n_in), std=n_in ** -0.5, dtype=dt, device=device)

    def gain(tag, env=0):
        if random_gains:
            return normal(seed, tag, env, (d,), std=0.1, mean=1.0, device=device)
        return torch.ones(d, dtype=torch.float32, device=device)

    out = {
        "w_in": mat("w_in", d, A), "w_out": mat("w_out", A, d),
        "b_out": normal(seed, "b_out", 0, (A,), std=0.1, device=device),
        "g_final": gain("g_final"), "layers": [],
    }
    for l in range(w.L):
        out["layers"].append({
            "g1": gain("g1", l), "g2": gain("g2", l), "g3": gain("g3", l),
            "w_qkv": mat("w_qkv", 3 * d, d, l), "w_o": mat("w_o", d, d, l),
            "w_qc": mat("w_qc", d, d, l), "w_oc": mat("w_oc", d, d, l),
            "w_1": mat("w_1", md, d, l), "w_2": mat("w_2", d, md, l),
        })
        if w.d_ctx > 0:
            out["layers"][-1]["w_kc"] = mat("w_kc", d, w.d_ctx, l)
            out["layers"][-1]["w_vc"] = mat("w_vc", d, w.d_ctx, l)
    return out


@dataclass
class EnvInputs:
    env_id: int
    noise: torch.Tensor        # [H][A] fp32: the action state at step ``step``
    kv: torch.Tensor           # [1][2][P][d] in the workload's dtype (plane 0 = K, 1 = V); with
                               # d_ctx > 0 the hidden states [P][d_ctx] instead
    P: int
    step: int                  # Euler step index the environment sits at


def make_env(w: Workload, env_id: int, seed: int = DEFAULT_SEED, device="cpu") -> EnvInputs:
    P = uniform_int(seed, "prefix_len", env_id, w.P[0], w.P[1])
    step = uniform_int(seed, "step_index", env_id, 0, w.K - 1) if w.mixed_steps else 0
    noise = normal(seed, "noise", env_id, (w.H, w.A), device=device)
    if w.d_ctx > 0:
        kv = normal(seed, "prefix_hidden", env_id, (P, w.d_ctx), dtype=w.torch_dtype, device=device)
    else:
        kv = normal(seed, "prefix_kv", env_id, (1, 2, P, w.d), dtype=w.torch_dtype, device=device)
    return EnvInputs(env_id, noise, kv, P, step)


def arrival_groups(w: Workload, seed: int = DEFAULT_SEED, env_ids: Optional[List[int]] = None
                   ) -> List[List[int]]:
    """Seeded ragged arrivals: a Fisher-Yates shuffle of the environment ids cut into groups of
    uniformly drawn size (the last group takes what is left).  One group if the workload has
    no group range."""
    ids = list(range(w.B)) if env_ids is None else list(env_ids)
    if w.group is None:
        return [ids]
    for i in range(len(ids) - 1, 0, -1):
        j = uniform_int(seed, "shuffle", 0, 0, i, index=i)
        ids[i], ids[j] = ids[j], ids[i]
    groups, pos, g = [], 0, 0
    while pos < len(ids):
        size = uniform_int(seed, "group_size", 0, w.group[0], w.group[1], index=g)
        groups.append(ids[pos:pos + size])
        pos += size
        g += 1
    return groups


def shard_env_ids(n_envs: int, rank: int, world: int) -> List[int]:
    """Environment ids owned by one rank when a job is spread over ``world`` replicas
    (environments are independent, section 4.2.2: no exchange between replicas)."""
    return [e for e in range(n_envs) if e % world == rank]
