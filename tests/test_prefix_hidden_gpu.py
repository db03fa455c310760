"""GPU tests of the hidden-state prefix variant (cfg.d_ctx > 0): the prefix of an environment is
the backbone's hidden states [P][d_ctx]; every layer's cross-attention keys and values are
projected from them once per batch (section 2.1: the head is conditioned on what the backbone
has cached; here that cache holds features, not ready-made keys and values).

All calls go through the C ABI; expected values come from the fp64 oracle only.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2609_27547_b200 import binding as B
from paper_2609_27547_b200 import synth
from gpu_helpers import Runner, TOL, stack
from helpers import chunk_rel_err, oracle_run

pytestmark = pytest.mark.gpu
SEED = 4321


def _case(dtype, d_ctx, **kw):
    base = dict(B=9, dtype=dtype, L=2, P=(9, 150), mixed_steps=True, d_ctx=d_ctx)
    base.update(kw)
    w = synth.scaled(synth.WORKLOADS[0], **base)
    wt = synth.make_weights(w, SEED, random_gains=True)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    return w, wt, envs


@pytest.mark.parametrize("dtype,d_ctx", [("f32", 128), ("f32", 64), ("bf16", 128), ("bf16", 192), ("bf16", 512)])
def test_parity_with_the_oracle(dtype, d_ctx):
    w, wt, envs = _case(dtype, d_ctx)
    ref = oracle_run(w, wt, envs)
    r = Runner(w, wt, envs, max_inflight_groups=2, flags=B.FLAG_TIMING)
    ids = list(range(w.B))
    got = stack(r.run([ids[:5], ids[5:]], quota=37), ids)
    st = r.gen.stats()
    r.close()
    assert chunk_rel_err(got, ref) <= TOL[dtype]
    # one gather plus a key and a value projection per layer, once for the whole batch
    assert st["classes"]["prefix"]["launches"] == 1 + 2 * w.L


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_result_does_not_depend_on_batching_or_quota(dtype):
    """The projected planes of an environment are a function of its own hidden rows only: alone, in
    any group, in any order and under any quota the chunk is the same bits."""
    w, wt, envs = _case(dtype, 128)
    ids = list(range(w.B))
    r = Runner(w, wt, envs, max_inflight_groups=4)
    base = stack(r.run([ids], quota=0), ids)
    alone = stack(r.run([[e] for e in ids], quota=0), ids)
    parts = stack(r.run([ids[6:], ids[:2], ids[2:6][::-1]], quota=74), ids)
    small = stack(r.run([ids[::-1]], quota=16), ids)
    r.close()
    r1 = Runner(w, wt, envs, max_inflight_groups=1)     # every group its own batch
    solo = stack(r1.run([[e] for e in ids], quota=37), ids)
    r1.close()
    for other in (alone, parts, small, solo):
        assert np.array_equal(base, other)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_identity_projections_reduce_to_the_plane_form(dtype):
    """d_ctx = d and W_kc = W_vc = I: the projected planes equal the hidden states exactly (the
    products add only zeros), so the run must match, bit for bit, a handle that is given
    K = V = h as ready-made planes."""
    w, wt, envs = _case(dtype, 256)
    for l in wt["layers"]:
        l["w_kc"] = torch.eye(w.d, dtype=w.torch_dtype)
        l["w_vc"] = torch.eye(w.d, dtype=w.torch_dtype)
    ids = list(range(w.B))
    r = Runner(w, wt, envs)
    got = stack(r.run([ids], quota=74), ids)
    r.close()
    wp = synth.scaled(w, d_ctx=0)
    plane_envs = [synth.EnvInputs(e.env_id, e.noise, torch.stack([e.kv, e.kv])[None].contiguous(), e.P, e.step) for e in envs]
    rp = Runner(wp, wt, plane_envs)
    want = stack(rp.run([ids], quota=74), ids)
    rp.close()
    assert np.array_equal(got, want)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_host_buffers_and_step_by_step(dtype):
    """The host-buffer entry point stages hidden states instead of planes; advancing one Euler
    step per submit (re-projecting each time) gives the same chunk as one submit."""
    w, wt, envs = _case(dtype, 128, mixed_steps=False)
    ids = list(range(w.B))
    r = Runner(w, wt, envs, max_inflight_groups=2)
    base = r.run([ids], quota=37)
    h_noise = torch.stack([e.noise for e in envs]).pin_memory()
    h_out = torch.empty_like(h_noise).pin_memory()
    h_kv = [e.kv.contiguous().pin_memory() for e in envs]
    r.gen.submit_host(ids[:4], h_kv[:4], h_noise[:4], h_out[:4], sm_quota=37)
    r.gen.submit_host(ids[4:], h_kv[4:], h_noise[4:], h_out[4:], sm_quota=37)
    r.gen.sync()
    assert np.array_equal(h_out.numpy(), stack(base, ids))
    state = {e: r.noise[e] for e in ids}
    for k in range(w.K):
        res = r.run([ids[:3], ids[3:]], quota=37, n_steps=1, state=state, steps={e: k for e in ids})
        state = {e: torch.from_numpy(res[e]).cuda() for e in ids}
    r.close()
    assert np.array_equal(np.stack([state[e].cpu().numpy() for e in ids]), stack(base, ids))


def test_scratch_grows_with_the_batch():
    """A later, larger batch than any seen before makes the projected-plane scratch grow; results
    of the small and the large batch agree with the oracle."""
    w, wt, envs = _case("bf16", 128, B=24, P=(40, 300))
    ref = oracle_run(w, wt, envs)
    ids = list(range(w.B))
    r = Runner(w, wt, envs, max_inflight_groups=1)
    first = r.run([ids[:2]], quota=74)
    second = r.run([ids], quota=74)
    third = r.run([ids[:2]], quota=74)
    r.close()
    assert chunk_rel_err(stack(second, ids), ref) <= TOL["bf16"]
    assert np.array_equal(stack(first, ids[:2]), stack(second, ids[:2]))
    assert np.array_equal(stack(first, ids[:2]), stack(third, ids[:2]))


def test_configuration_errors():
    w, wt, envs = _case("f32", 128, B=2)
    cfg = B.cfg_for(w, max_group_envs=2)
    assert cfg.d_ctx == 128 and cfg.kv_layers == w.L
    cfg.kv_layers = 1
    assert B.lib().ebrl_actgen_check_cfg(C.byref(cfg)) == B.ERR_INVALID_ARG
    cfg.kv_layers = w.L
    missing = {**wt, "layers": [{k: v for k, v in l.items()} for l in wt["layers"]]}
    gen = B.ActGen(cfg, missing)     # complete weights: fine
    gen.destroy()
    # a NULL projection although d_ctx > 0 is refused at create
    lw = (B.LayerWeights * w.L)()
    keep = []
    for i, l in enumerate(wt["layers"]):
        t = {k: v.cuda().contiguous() for k, v in l.items()}
        keep.append(t)
        lw[i] = B.LayerWeights(t["g1"].data_ptr(), t["g2"].data_ptr(), t["g3"].data_ptr(), t["w_qkv"].data_ptr(),
                               t["w_o"].data_ptr(), t["w_qc"].data_ptr(), t["w_oc"].data_ptr(), t["w_1"].data_ptr(),
                               t["w_2"].data_ptr(), t["w_kc"].data_ptr(), None)
    top = {k: wt[k].cuda().contiguous() for k in ("w_in", "w_out", "b_out", "g_final")}
    ws = B.Weights(top["w_in"].data_ptr(), top["w_out"].data_ptr(), top["b_out"].data_ptr(), top["g_final"].data_ptr(),
                   C.cast(lw, C.POINTER(B.LayerWeights)))
    h = C.c_void_p()
    assert B.lib().ebrl_actgen_create(C.byref(cfg), C.byref(ws), C.byref(h)) == B.ERR_INVALID_ARG
    assert not h.value


def test_weight_publication_replaces_the_projections_too():
    """A published policy version carries its own W_kc / W_vc: batches launched after the update
    project the prefixes with the new matrices, batches queued before it with the old ones."""
    w, wA, envs = _case("bf16", 128)
    wB = synth.make_weights(w, SEED + 7, random_gains=True)
    ids = list(range(w.B))
    refs = {}
    for name, wt in (("A", wA), ("B", wB)):
        r = Runner(w, wt, envs)
        refs[name] = stack(r.run([ids]), ids)
        r.close()
    only_proj = {**wA, "layers": [{**la, "w_kc": lb["w_kc"], "w_vc": lb["w_vc"]} for la, lb in zip(wA["layers"], wB["layers"])]}
    r = Runner(w, only_proj, envs)
    ref_proj = stack(r.run([ids]), ids)
    r.close()
    assert not np.array_equal(refs["A"], ref_proj)      # the projections matter on their own
    r = Runner(w, wA, envs, max_inflight_groups=4)
    noise = torch.stack([r.noise[e] for e in ids])
    out1, out2 = torch.empty_like(noise), torch.empty_like(noise)
    kv = [r.kv[e] for e in ids]
    sidx = [envs[e].step for e in ids]
    r.gen.submit(ids[:4], kv[:4], noise[:4], out1[:4], step_index=sidx[:4])      # queued under version 1
    assert r.gen.update_weights(wB) == 2
    r.gen.submit([100 + e for e in ids], kv, noise, out2, step_index=sidx)         # runs with version 2
    r.gen.sync()
    assert np.array_equal(out1[:4].cpu().numpy(), refs["A"][:4])
    assert np.array_equal(out2.cpu().numpy(), refs["B"])
    assert r.gen.update_weights(only_proj) == 3
    assert np.array_equal(stack(r.run([ids]), ids), ref_proj)
    r.close()
