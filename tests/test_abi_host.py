"""CPU-only tests of the boundary: the shared library loads without a GPU and exports every
symbol the header declares; the argument rules and the batcher's plan behave as documented;
without a CUDA device the product path fails loudly (no CPU fallback)."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2609_27547_b200 import binding as B
from paper_2609_27547_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names.update(re.findall(r"\b(ebrl_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert "ebrl_actgen_create" in names and "ebrl_actgen_submit" in names and "ebrl_actgen_sync" in names
    assert len(names) >= 24 and "ebrl_alloc_elastic" in names and "ebrl_actgen_update_weights" in names
    lib = B.lib()
    for n in names:
        assert hasattr(lib, n), n
    assert lib.ebrl_actgen_abi_version() == B.ABI_VERSION


def test_struct_sizes_match_the_header_layout():
    assert C.sizeof(B.Cfg) == 96
    assert C.sizeof(B.LayerWeights) == 88 and C.sizeof(B.Weights) == 40 and C.sizeof(B.SubmitExt) == 24
    assert C.sizeof(B.Stats) == 8 * 4 + 16 + 7 * 8 * 4 + 8     # seven kernel classes
    # and the library, as compiled from the header, agrees with the hand-written mirrors
    for which, mirror in enumerate((B.Cfg, B.LayerWeights, B.Weights, B.SubmitExt, B.Stats)):
        assert B.lib().ebrl_actgen_struct_size(which) == C.sizeof(mirror), mirror.__name__
    assert B.lib().ebrl_actgen_struct_size(5) == 0


def _cfg(**kw):
    base = dict(H=8, A=7, d=256, n_layers=2, n_heads=4, K_steps=4, max_prefix_len=64, max_group_envs=16)
    base.update(kw)
    return B.make_cfg(**base)


@pytest.mark.parametrize("kw,status", [
    ({}, B.OK),
    ({"d": 255}, B.ERR_INVALID_ARG),          # odd d
    ({"n_heads": 3}, B.ERR_INVALID_ARG),      # d % heads
    ({"K_steps": 0}, B.ERR_INVALID_ARG),
    ({"max_group_envs": 0}, B.ERR_INVALID_ARG),
    ({"kv_layers": 3}, B.ERR_INVALID_ARG),
    ({"H": 33}, B.ERR_UNSUPPORTED),
    ({"d": 192, "n_heads": 3}, B.ERR_UNSUPPORTED),   # d not a multiple of 128
    ({"n_heads": 1}, B.ERR_UNSUPPORTED),             # head_dim 256
    ({"n_layers": 0}, B.OK),
    ({"d_ctx": 128}, B.OK),                          # hidden-state prefixes (make_cfg sets kv_layers = n_layers)
    ({"d_ctx": 100}, B.ERR_UNSUPPORTED),             # not a multiple of 64
    ({"d_ctx": -64}, B.ERR_INVALID_ARG),
])
def test_check_cfg(kw, status):
    assert B.lib().ebrl_actgen_check_cfg(C.byref(_cfg(**kw))) == status
    if status != B.OK:
        assert len(B.lib().ebrl_actgen_last_error(None)) > 0


def test_check_cfg_abi_version_and_null():
    c = _cfg()
    c.abi_version = 99
    assert B.lib().ebrl_actgen_check_cfg(C.byref(c)) == B.ERR_INVALID_ARG
    assert B.lib().ebrl_actgen_check_cfg(None) == B.ERR_INVALID_ARG


def _check_submit(cfg, ids, kv, quota=0, prefix_len=None, step_index=None, n_steps=0, n_sms=148, noise=0x1000, out=0x2000):
    n = len(ids)
    a_ids = (C.c_int64 * max(1, n))(*ids)
    a_kv = (C.c_void_p * max(1, n))(*kv) if kv is not None else None
    ext, keep = B._ext(prefix_len, step_index, n_steps)
    return B.lib().ebrl_actgen_check_submit(C.byref(cfg), n_sms, n, a_ids, a_kv, noise, out, quota, C.byref(ext))


def test_check_submit_rules():
    cfg = _cfg()
    kv = [0x10000 + 256 * i for i in range(4)]
    assert _check_submit(cfg, [1, 2, 3, 4], kv) == B.OK
    assert _check_submit(cfg, [], None) == B.OK                                   # empty group: no-op
    assert _check_submit(cfg, [1, 2, 2, 4], kv) == B.ERR_INVALID_ARG              # duplicate id
    assert b"duplicate" in B.lib().ebrl_actgen_last_error(None)
    assert _check_submit(cfg, [1, 2, 3, 4], kv, quota=149) == B.ERR_QUOTA
    assert _check_submit(cfg, [1, 2, 3, 4], kv, quota=-1) == B.ERR_QUOTA
    assert _check_submit(cfg, [1, 2, 3, 4], kv, quota=37) == B.OK
    assert _check_submit(cfg, [1, 2, 3, 4], kv, prefix_len=[1, 64, 3, 4]) == B.OK
    assert _check_submit(cfg, [1, 2, 3, 4], kv, prefix_len=[0, 64, 3, 4]) == B.ERR_INVALID_ARG
    assert _check_submit(cfg, [1, 2, 3, 4], kv, prefix_len=[1, 65, 3, 4]) == B.ERR_INVALID_ARG
    assert _check_submit(cfg, [1, 2, 3, 4], kv, step_index=[0, 3, 1, 2]) == B.OK
    assert _check_submit(cfg, [1, 2, 3, 4], kv, step_index=[0, 4, 1, 2]) == B.ERR_INVALID_ARG
    assert _check_submit(cfg, [1, 2, 3, 4], kv, n_steps=-1) == B.ERR_INVALID_ARG
    assert _check_submit(cfg, [1, 2, 3, 4], [kv[0], 0, kv[2], kv[3]]) == B.ERR_INVALID_ARG   # NULL plane
    assert _check_submit(cfg, [1, 2, 3, 4], [kv[0], kv[1] + 8, kv[2], kv[3]]) == B.ERR_INVALID_ARG   # misaligned
    assert _check_submit(cfg, list(range(17)), [0x10000] * 17) == B.ERR_INVALID_ARG   # > max_group_envs
    assert _check_submit(cfg, [1, 2, 3, 4], kv, noise=None) == B.ERR_INVALID_ARG


def test_plan_group_orders_longest_first_and_is_stable():
    cfg = _cfg(K_steps=4)
    S, order, ns, na = B.plan_group(cfg, 6, step_index=[3, 0, 2, 0, 1, 3])
    assert S == 4
    assert order == [1, 3, 4, 2, 0, 5]          # steps 4,4,3,2,1,1: ties keep arrival order
    assert ns == [4, 4, 3, 2, 1, 1]
    assert na == [6, 4, 3, 2]                   # environments still active at inner step s
    S, order, ns, na = B.plan_group(cfg, 3, step_index=[0, 3, 1], n_steps=2)
    assert S == 2 and ns == [2, 2, 1] and order == [0, 2, 1] and na == [3, 2, 0, 0]
    assert B.plan_group(cfg, 0)[0] == 0
    assert B.plan_group(cfg, 2, step_index=[0, 9])[0] == -1


@pytest.mark.skipif(torch.cuda.is_available(), reason="this check is for a box without a GPU")
def test_create_fails_loudly_without_a_device():
    w = synth.scaled(synth.WORKLOADS[0], B=2)
    wt = synth.make_weights(w)
    with pytest.raises(B.EbrlError) as ei:
        B.ActGen(B.cfg_for(w), wt)
    assert ei.value.status == B.ERR_CUDA


def test_corunner_argument_checks_need_no_device():
    L = B.lib()
    assert L.ebrl_sim_corunner_launch(None, 1024, 1, 1, None) == B.ERR_INVALID_ARG
    assert L.ebrl_sim_corunner_launch(0x1000, 1023, 1, 1, None) == B.ERR_INVALID_ARG
    assert L.ebrl_sim_corunner_launch(0x1000, 1024, 1, 0, None) == B.ERR_INVALID_ARG
    assert L.ebrl_sim_corunner_launch(0x1000, 0, 1, 4, None) == B.OK
