"""Failure detection without a fault: the give-up path of the real kernels, and the guard words
around the workspaces.

Every device-side wait of the library is bounded.  Here the copy-issuing thread of a kernel family
is told (test flag) to issue nothing on a one-tile batch with a 50 ms limit, so the waits of the
other roles run out: the MMA thread's wait for operands, the epilogue warps' wait for the
accumulator (in the CTA-pair kernel the peer CTA's warps wait out their own limit before the final
cluster barrier), the attention heads' wait for their key block.  The kernels must return normally
with EBRL_ERR_TIMEOUT in the status word, tensor memory freed, and the context must stay usable:
a fresh handle then reproduces the oracle.  No trap, no bad address, no endless loop is involved.
"""
import time

import numpy as np
import pytest
import torch

from paper_2609_27547_b200 import binding as B
from paper_2609_27547_b200 import synth
from helpers import chunk_rel_err, oracle_run
from gpu_helpers import Runner, TOL, stack

pytestmark = pytest.mark.gpu
SEED = synth.DEFAULT_SEED
LIMIT_NS = 50_000_000


def _tiny(dtype="bf16"):
    w = synth.scaled(synth.WORKLOADS[0], B=4, dtype=dtype, d=256, n_heads=4, L=1, K=1, P=(16, 40))
    wt = synth.make_weights(w, SEED, random_gains=True)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    return w, wt, envs


def _expect_timeout_then_recover(flags, monkeypatch=None, shape=None, dtype="bf16"):
    w, wt, envs = _tiny(dtype)
    ids = list(range(w.B))
    if shape is not None:
        monkeypatch.setenv("EBRL_GEMM_SHAPE", shape)
    cfg = B.cfg_for(w, max_group_envs=w.B, max_inflight_groups=1, flags=flags)
    cfg.max_prefix_len = 40
    cfg.wait_limit_ns = LIMIT_NS
    gen = B.ActGen(cfg, wt)
    if shape is not None:
        monkeypatch.delenv("EBRL_GEMM_SHAPE")
    noise = torch.stack([e.noise for e in envs]).cuda()
    out = torch.empty_like(noise)
    t0 = time.perf_counter()
    gen.submit(ids, [e.kv.cuda() for e in envs], noise, out)
    with pytest.raises(B.EbrlError) as ei:
        gen.sync()
    dt = time.perf_counter() - t0
    assert ei.value.status == B.ERR_TIMEOUT
    assert dt < 10.0                                   # a handful of kernels, each giving up after about 2 x 50 ms
    with pytest.raises(B.EbrlError) as ei2:            # the failure is sticky on this handle
        gen.submit([100 + e for e in ids], [e.kv.cuda() for e in envs], noise, out)
    assert ei2.value.status == B.ERR_TIMEOUT
    gen.destroy()
    # the context survived: a fresh handle computes the oracle's chunks
    r = Runner(w, wt, envs)
    got = stack(r.run([ids]), ids)
    r.close()
    assert chunk_rel_err(got, oracle_run(w, wt, envs)) <= TOL[dtype]


@pytest.mark.parametrize("shape", ["128", "2"])
def test_fp32_tensor_core_projection_kernels_give_up_cleanly(monkeypatch, shape):
    """The split-operand kernels of the fp32 models (six operand tiles per stage): single CTAs and CTA pairs."""
    _expect_timeout_then_recover(B.FLAG_TEST_DROP_GEMM_COPIES, monkeypatch, shape, dtype="f32")


@pytest.mark.parametrize("shape", ["128", "256", "2"])
def test_projection_kernels_give_up_cleanly(monkeypatch, shape):
    """One-CTA kernels on 128 x 128 and 128 x 256 tiles, and the CTA-pair kernel."""
    _expect_timeout_then_recover(B.FLAG_TEST_DROP_GEMM_COPIES | B.FLAG_NO_FUSED, monkeypatch, shape)


def test_attention_kernel_gives_up_cleanly():
    _expect_timeout_then_recover(B.FLAG_TEST_DROP_ATTN_COPIES | B.FLAG_NO_FUSED)


@pytest.mark.parametrize("what", ["gemm", "attn"])
def test_persistent_step_kernel_gives_up_cleanly(what):
    drop = B.FLAG_TEST_DROP_GEMM_COPIES if what == "gemm" else B.FLAG_TEST_DROP_ATTN_COPIES
    _expect_timeout_then_recover(drop | B.FLAG_FORCE_FUSED)


@pytest.mark.parametrize("path", ["per_op_bf16", "fused_bf16", "plain_alu_f32"])
def test_guard_words_behind_every_workspace_stay_intact(path):
    """EBRL_FLAG_DEBUG_CANARY: 256 pattern bytes behind every buffer the handle allocates, checked at
    every sync.  A ragged batch whose last row tile is partial (the tiles' loads and the epilogues'
    stores reach up to the buffers' ends) must leave all of them untouched, and still match the oracle."""
    dtype = "f32" if path == "plain_alu_f32" else "bf16"
    w = synth.scaled(synth.WORKLOADS[0], B=37, dtype=dtype, P=(1, 97), mixed_steps=True, K=3)
    wt = synth.make_weights(w, SEED, random_gains=True)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    flags = B.FLAG_DEBUG_CANARY | (B.FLAG_FORCE_FUSED if path == "fused_bf16" else B.FLAG_NO_FUSED)
    r = Runner(w, wt, envs, flags=flags, max_group_envs=w.B, max_inflight_groups=1)   # workspace = exactly the batch's rows
    ids = list(range(w.B))
    got = stack(r.run([ids]), ids)                     # sync raises if a guard changed
    got2 = stack(r.run([ids[:20], ids[20:]]), ids)     # one group per batch now: two smaller batches
    r.close()
    assert np.array_equal(got, got2)
    assert chunk_rel_err(got, oracle_run(w, wt, envs)) <= TOL[dtype]
