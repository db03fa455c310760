"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: every
environment of the workload submitted in its seeded arrival groups at the workload's SM quota
with the bench's queue depth.  The oracle cannot run thousands of environments in seconds, so a
seeded sample of environments is compared element-wise (environments are independent), and the
rest is covered by a property that holds at any size: the batch result of an environment equals
the result of running it alone, bit for bit.
"""
import numpy as np
import pytest
import torch

from paper_2609_27547_b200 import binding as B
from paper_2609_27547_b200 import synth
from helpers import chunk_rel_err, oracle_cfg, oracle_weights, np32
from gpu_helpers import TOL

import oracle

pytestmark = pytest.mark.gpu
SEED = synth.DEFAULT_SEED


def _run_full(w, wt, envs, groups, quota, n_steps=0, inflight=8):
    gen = B.ActGen(B.cfg_for(w, max_group_envs=max(len(g) for g in groups), max_inflight_groups=inflight), wt)
    order = [e for g in groups for e in g]
    pos = {e: i for i, e in enumerate(order)}
    noise = torch.stack([envs[e].noise for e in order]).contiguous()
    out = torch.empty_like(noise)
    for g in groups:
        lo = pos[g[0]]
        gen.submit(g, [envs[e].kv for e in g], noise[lo:lo + len(g)], out[lo:lo + len(g)], sm_quota=quota,
                   step_index=[envs[e].step for e in g], n_steps=n_steps)
    gen.sync()
    return gen, out, pos


def _oracle(w, wt_cpu, envs, ids, n_steps=0):
    return oracle.actgen(oracle_cfg(w), oracle_weights(wt_cpu), [np32(envs[e].kv) for e in ids],
                         np.stack([np32(envs[e].noise) for e in ids]), step_index=[envs[e].step for e in ids], n_steps=n_steps)


def _alone(gen, w, envs, e, quota, n_steps=0):
    noise = envs[e].noise[None].contiguous()
    out = torch.empty_like(noise)
    gen.submit([e], [envs[e].kv], noise, out, sm_quota=quota, step_index=[envs[e].step], n_steps=n_steps)
    gen.sync()
    return out[0]


def test_configs1_full_size_sampled():
    """configs[1]: 256 envs, one group, full quota; 8 sampled envs against the oracle."""
    w = synth.WORKLOADS[1]
    wt = synth.make_weights(w, SEED, device="cuda")
    envs = {e: synth.make_env(w, e, SEED, device="cuda") for e in range(w.B)}
    groups = synth.arrival_groups(w, SEED)
    gen, out, pos = _run_full(w, wt, envs, groups, 0)
    sample = [0, 1, 77, 128, 200, 254, 255, 31]
    ref = _oracle(w, wt, envs, sample)
    got = np.stack([out[pos[e]].cpu().numpy() for e in sample])
    assert chunk_rel_err(got, ref) <= TOL["bf16"]
    for e in sample[:3]:
        assert torch.equal(_alone(gen, w, envs, e, 37), out[pos[e]])
    gen.destroy()


def test_configs2_full_size_ragged_sampled():
    """configs[2]: 512 envs in seeded groups of 1..64, prefix lengths 64..512, mixed step indices."""
    w = synth.WORKLOADS[2]
    wt = synth.make_weights(w, SEED, device="cuda")
    envs = {e: synth.make_env(w, e, SEED, device="cuda") for e in range(w.B)}
    groups = synth.arrival_groups(w, SEED)
    assert len(groups) > 8 and len({envs[e].step for e in range(w.B)}) == w.K
    gen, out, pos = _run_full(w, wt, envs, groups, 0, inflight=4)
    sample = [groups[0][0], groups[0][-1], groups[3][0], groups[-1][-1]] + list(range(100, 112))
    ref = _oracle(w, wt, envs, sample)
    got = np.stack([out[pos[e]].cpu().numpy() for e in sample])
    assert chunk_rel_err(got, ref) <= TOL["f32"]
    for e in sample[:4]:
        assert torch.equal(_alone(gen, w, envs, e, 16), out[pos[e]])   # "identical to processing every env alone"
    gen.destroy()


def test_configs3_quota_sweep_bit_identity():
    """configs[3]: 1024 envs, P=256, quotas 16/37/74/148 bit-identical, also as 8 groups of 128."""
    w = synth.WORKLOADS[3]
    wt = synth.make_weights(w, SEED, device="cuda")
    envs = {e: synth.make_env(w, e, SEED, device="cuda") for e in range(w.B)}
    ids = list(range(w.B))
    base = None
    for q in (148, 74, 37, 16):
        gen, out, pos = _run_full(w, wt, envs, [ids], q)
        gen.destroy()
        if base is None:
            base = out.clone()
        else:
            assert torch.equal(out, base), "quota %d" % q
    gen, out, pos = _run_full(w, wt, envs, [ids[i:i + 128] for i in range(0, w.B, 128)], 74)
    gen.destroy()
    assert torch.equal(out, base)
    sample = [0, 500, 1023, 77]
    ref = _oracle(w, wt, envs, sample)
    assert chunk_rel_err(np.stack([base[e].cpu().numpy() for e in sample]), ref) <= TOL["f32"]


def test_configs2_and_3_on_the_mid_size_bf16_model():
    """The other reading of "the config-1 model" (the bf16 mid-size head of configs[1]): the ragged
    arrivals of configs[2] against the oracle and alone, the quota sweep of configs[3] bit-identical."""
    w = synth.WORKLOADS[12]
    wt = synth.make_weights(w, SEED, device="cuda")
    envs = {e: synth.make_env(w, e, SEED, device="cuda") for e in range(w.B)}
    groups = synth.arrival_groups(w, SEED)
    gen, out, pos = _run_full(w, wt, envs, groups, 0, inflight=4)
    sample = [groups[0][0], groups[3][0], groups[-1][-1], 100, 101, 102]
    ref = _oracle(w, wt, envs, sample)
    got = np.stack([out[pos[e]].cpu().numpy() for e in sample])
    assert chunk_rel_err(got, ref) <= TOL["bf16"]
    for e in sample[:3]:
        assert torch.equal(_alone(gen, w, envs, e, 16), out[pos[e]])
    gen.destroy()
    del envs
    w = synth.WORKLOADS[13]
    envs = {e: synth.make_env(w, e, SEED, device="cuda") for e in range(w.B)}
    ids = list(range(w.B))
    base = None
    for q in (148, 74, 37, 16):
        gen, out, pos = _run_full(w, wt, envs, [ids], q)
        gen.destroy()
        if base is None:
            base = out.clone()
        else:
            assert torch.equal(out, base), "quota %d" % q
    gen, out, pos = _run_full(w, wt, envs, [ids[i:i + 128] for i in range(0, w.B, 128)], 74)
    gen.destroy()
    assert torch.equal(out, base)
    sample = [0, 1023]
    ref = _oracle(w, wt, envs, sample)
    assert chunk_rel_err(np.stack([base[e].cpu().numpy() for e in sample]), ref) <= TOL["bf16"]


def test_configs4_full_size_sampled():
    """configs[4]: 2048 envs, ragged groups of 32..256 at the 74-SM quota, queue depth 16 (the bench's
    launch configuration: the whole step is one packed batch of 32768 rows); also at depth 8 (two batches).
    One Euler step of four sampled envs against the oracle, then the whole chunk (K = 10 steps) of six
    envs against the oracle (about a minute of host time per environment, one thread each), plus the
    whole-chunk result of sampled envs against running them alone."""
    w = synth.WORKLOADS[4]
    wt = synth.make_weights(w, SEED, device="cuda")
    envs = {e: synth.make_env(w, e, SEED, device="cuda") for e in range(w.B)}
    groups = synth.arrival_groups(w, SEED)
    gen, out1, pos = _run_full(w, wt, envs, groups, w.quota, n_steps=1, inflight=16)
    sample = [groups[0][0], groups[5][-1], groups[-1][-1], 1234]
    ref = _oracle(w, wt, envs, sample, n_steps=1)
    got = np.stack([out1[pos[e]].cpu().numpy() for e in sample])
    assert chunk_rel_err(got, ref) <= TOL["bf16"]
    gen.destroy()
    gen, out, pos = _run_full(w, wt, envs, groups, w.quota, inflight=16)
    assert torch.isfinite(out).all()
    # the FINAL action chunk (all K = 10 Euler steps) of six environments against the oracle.  Packed
    # rows follow the arrival order (all environments run the same number of steps), 16 environments
    # per 256-row pair tile: positions 0 and 15 are the first and last rows of the first pair tile,
    # 7 and 8 the last rows of its leader CTA and the first of its peer CTA, 1000 sits mid-batch
    # and 2047 holds the last 16 rows of the batch.
    order = [e for g in groups for e in g]
    chunk_sample = [order[p] for p in (0, 7, 8, 15, 1000, w.B - 1)]
    ref_k = _oracle(w, wt, envs, chunk_sample)
    got_k = np.stack([out[pos[e]].cpu().numpy() for e in chunk_sample])
    assert chunk_rel_err(got_k, ref_k) <= TOL["bf16"]
    for e in sample[:2]:
        assert torch.equal(_alone(gen, w, envs, e, 148), out[pos[e]])
    gen.destroy()
    gen, out8, _ = _run_full(w, wt, envs, groups, w.quota, inflight=8)     # two batches instead of one: same bits
    assert torch.equal(out8, out)                                          # (the first batch ends in a ragged row tile)
    assert sum(len(g) for g in groups[:8]) * w.H % 256 != 0
    gen.destroy()
