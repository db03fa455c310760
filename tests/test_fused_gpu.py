"""The persistent step kernel (one resident grid walking every Euler step of a small batch) against
the fp64 oracle and against the per-operation kernels: the two paths must deliver the same bits,
at any SM quota, for ragged groups, mixed step indices and per-layer planes."""
import numpy as np
import pytest
import torch

from paper_2609_27547_b200 import binding as B
from paper_2609_27547_b200 import synth
from helpers import chunk_rel_err, oracle_run, np32
from gpu_helpers import Runner, TOL, stack

pytestmark = pytest.mark.gpu
SEED = synth.DEFAULT_SEED


def _setup(w, seed=SEED):
    wt = synth.make_weights(w, seed, random_gains=True)
    envs = [synth.make_env(w, e, seed) for e in range(w.B)]
    return wt, envs


def _launches(r):
    return r.gen.stats()["kernel_launches"]


@pytest.mark.parametrize("shape", ["hd64_H8", "hd128_H16"])
def test_fused_matches_oracle_and_per_op_path_bitwise(shape):
    """Several row blocks plus a ragged one, ragged prefixes (one key, lengths that are no multiple of
    the key block), mixed step indices.  Every row against the oracle; fused == per-operation bit for bit."""
    if shape == "hd64_H8":
        w = synth.scaled(synth.WORKLOADS[0], B=45, dtype="bf16", d=256, n_heads=4, L=2, K=4, P=(1, 97), mixed_steps=True)
    else:
        w = synth.scaled(synth.WORKLOADS[0], B=21, dtype="bf16", H=16, A=14, d=512, n_heads=4, L=2, K=3, P=(3, 70),
                         mixed_steps=True)
    wt, envs = _setup(w)
    ref = oracle_run(w, wt, envs)
    ids = list(range(w.B))
    rf = Runner(w, wt, envs, flags=B.FLAG_FORCE_FUSED)
    got = stack(rf.run([ids]), ids)
    n_fused = _launches(rf)
    assert n_fused == 1                                   # ONE launch for the whole batch, all Euler steps
    assert rf.gen.stats()["classes"]["fused"]["launches"] == 0   # (timing off: classes are not filled)
    assert chunk_rel_err(got, ref) <= TOL["bf16"]
    rp = Runner(w, wt, envs, flags=B.FLAG_NO_FUSED)
    base = stack(rp.run([ids]), ids)
    assert _launches(rp) > 10 * n_fused
    rp.close()
    assert np.array_equal(got, base)
    for q in (1, 7, 37, 74):                              # any quota: same bits (one CTA walks the whole list alone)
        assert np.array_equal(stack(rf.run([ids], quota=q), ids), base), "quota %d" % q
    # group partitions and order: two batches, reversed
    assert np.array_equal(stack(rf.run([ids[:13], ids[13:]]), ids), base)
    assert np.array_equal(stack(rf.run([ids[::-1]]), ids), base)
    rf.close()


def test_fused_step_at_a_time_and_row_limit_selection(monkeypatch):
    """Step-level batching (n_steps = 1 submits) through the persistent kernel gives the bits of whole
    chunks; with a row limit set at create, batches up to that size take the persistent kernel
    without the flag, larger ones do not; without a limit none does."""
    w = synth.scaled(synth.WORKLOADS[0], B=20, dtype="bf16", d=256, n_heads=4, L=2, K=4, P=(16, 48))
    wt, envs = _setup(w)
    ids = list(range(w.B))
    r0 = Runner(w, wt, envs)                               # no limit: the per-operation kernels
    r0.run([ids])
    assert _launches(r0) > 10
    r0.close()
    monkeypatch.setenv("EBRL_FUSED_MAX_ROWS", "160")       # read when the handle is created
    r = Runner(w, wt, envs)
    monkeypatch.delenv("EBRL_FUSED_MAX_ROWS")
    r.run([ids[:19]])                                      # 152 rows: under the limit
    assert _launches(r) == 1
    r.gen.reset_stats()
    whole = r.run([ids])                                   # 160 rows: at the limit
    assert _launches(r) == 1
    state = {e: r.noise[e] for e in ids}
    for k in range(w.K):
        res = r.run([ids], n_steps=1, state=state, steps={e: k for e in ids})
        state = {e: torch.from_numpy(res[e]).cuda() for e in ids}
    assert np.array_equal(stack(whole, ids), np.stack([state[e].cpu().numpy() for e in ids]))
    assert chunk_rel_err(stack(whole, ids), oracle_run(w, wt, envs)) <= TOL["bf16"]
    r.close()


def test_fused_per_layer_planes_and_timing_class():
    """kv_layers = n_layers through the persistent kernel, with the per-class timing on."""
    import oracle
    from helpers import oracle_cfg, oracle_weights
    w = synth.scaled(synth.WORKLOADS[0], B=9, dtype="bf16", d=256, n_heads=4, L=3, K=3, P=(9, 70), mixed_steps=True)
    wt, envs = _setup(w)
    kvs = [synth.normal(SEED, "kv_per_layer", e.env_id, (w.L, 2, e.P, w.d), dtype=w.torch_dtype) for e in envs]
    oc = oracle_cfg(w)
    oc.kv_layers = w.L
    ref = oracle.actgen(oc, oracle_weights(wt), [np32(k) for k in kvs], np.stack([np32(e.noise) for e in envs]),
                        step_index=[e.step for e in envs])
    outs = {}
    for name, flags in (("fused", B.FLAG_FORCE_FUSED | B.FLAG_TIMING), ("per_op", B.FLAG_NO_FUSED)):
        cfg = B.cfg_for(w, max_group_envs=w.B, max_inflight_groups=1, flags=flags)
        cfg.kv_layers = w.L
        cfg.max_prefix_len = 70
        gen = B.ActGen(cfg, wt)
        noise = torch.stack([e.noise for e in envs]).cuda()
        out = torch.empty_like(noise)
        gen.submit(list(range(w.B)), [k.cuda() for k in kvs], noise, out, step_index=[e.step for e in envs])
        gen.sync()
        if name == "fused":
            cl = gen.stats()["classes"]["fused"]
            assert cl["launches"] == 1 and cl["ms"] > 0 and cl["flops"] > 0
        gen.destroy()
        outs[name] = out.cpu().numpy()
    assert chunk_rel_err(outs["fused"], ref) <= TOL["bf16"]
    assert np.array_equal(outs["fused"], outs["per_op"])


def test_fused_configs1_model_sampled():
    """The configs[1] model (d = 1024, 16 heads of 64, L = 4, K = 10) at 64 environments through the
    persistent kernel: sampled environments against the oracle, all of them against the per-operation path."""
    w = synth.scaled(synth.WORKLOADS[1], B=64)
    wt = synth.make_weights(w, SEED)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    ids = list(range(w.B))
    rf = Runner(w, wt, envs, flags=B.FLAG_FORCE_FUSED)
    got = stack(rf.run([ids]), ids)
    assert _launches(rf) == 1
    rf.close()
    rp = Runner(w, wt, envs, flags=B.FLAG_NO_FUSED)
    base = stack(rp.run([ids]), ids)
    rp.close()
    assert np.array_equal(got, base)
    sample = [0, 15, 16, 63]
    ref = oracle_run(w, wt, [envs[e] for e in sample])
    assert chunk_rel_err(got[sample], ref) <= TOL["bf16"]
