"""The allocation-free entry point (collected last on purpose: a failure here cannot hide the
other tests of a run that stops at the first failure).

Some callers of this library cannot allocate device memory when they need an action step -- a
control loop that must not take the allocator's lock, a worker whose memory budget was fixed at
start-up.  ``ebrl_actgen_l0_step_noalloc`` serves them with scratch that is part of the library
image.  The test calls it through the C ABI twice in a row (the scratch keeps the first call's
contents) and checks each result against the ordinary entry point run on the same inputs, within
the fp32 tolerance of the parity tests; both are also checked against the fp64 oracle's single
Euler step of the same layer-less model.
"""
import math

import numpy as np
import pytest
import torch

from paper_2609_27547_b200 import binding as B
from paper_2609_27547_b200 import synth
from helpers import chunk_rel_err, oracle_cfg, oracle_weights
from gpu_helpers import TOL

pytestmark = pytest.mark.gpu


def _temb_row(w, k):
    half = w.d // 2
    ang = (1000.0 * k / w.K) * np.power(10000.0, -np.arange(half, dtype=np.float64) / half)
    return torch.from_numpy(np.concatenate([np.sin(ang), np.cos(ang)]).astype(np.float32)).cuda()


def test_no_alloc_step_matches_submit_on_two_calls_in_a_row():
    w = synth.scaled(synth.WORKLOADS[0], B=23, L=0, d=384, n_heads=6, K=5, P=(4, 4))
    wt = synth.make_weights(w, 77, random_gains=True)
    dev = {k: v.cuda() for k, v in wt.items() if k != "layers"}
    gen = B.ActGen(B.cfg_for(w, max_group_envs=w.B), wt)
    kv = [torch.zeros((1, 2, 4, w.d), device="cuda") for _ in range(w.B)]
    ids = list(range(w.B))
    import oracle
    for call, (seed, k) in enumerate([(5, 0), (6, 3)]):
        a = synth.normal(seed, "state", 0, (w.B, w.H, w.A)).cuda()
        want = torch.empty_like(a)
        gen.submit(ids, kv, a, want, step_index=[k] * w.B, n_steps=1)
        gen.sync()
        got = torch.full_like(a, float("nan"))
        st = B.l0_step_noalloc(a, got, dev["w_in"], dev["w_out"], dev["b_out"], dev["g_final"], _temb_row(w, k), w.K,
                               sm_quota=37 if call else 0)
        assert st == B.OK
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        assert chunk_rel_err(got.cpu().numpy(), want.cpu().numpy().astype(np.float64)) <= TOL["f32"], "call %d" % call
        ref = oracle.actgen(oracle_cfg(w), oracle_weights(wt), [np.zeros((1, 2, 4, w.d), np.float32)] * w.B, a.cpu().numpy(),
                            step_index=[k] * w.B, n_steps=1)
        assert chunk_rel_err(got.cpu().numpy(), ref) <= TOL["f32"], "call %d against the oracle" % call
        assert chunk_rel_err(want.cpu().numpy(), ref) <= TOL["f32"], "call %d, ordinary entry point against the oracle" % call
    gen.destroy()


def test_no_alloc_step_rejects_sizes_beyond_its_scratch():
    A, K = 7, 4
    for rows, d, expect in ((513, 256, B.ERR_UNSUPPORTED), (8, 2048, B.ERR_UNSUPPORTED), (8, 200, B.ERR_UNSUPPORTED)):
        a = torch.zeros((rows, A), device="cuda")
        st = B.l0_step_noalloc(a, a.clone(), torch.zeros((d, A), device="cuda"), torch.zeros((A, d), device="cuda"),
                               torch.zeros(A, device="cuda"), torch.ones(d, device="cuda"), torch.zeros(d, device="cuda"), K)
        assert st == expect
