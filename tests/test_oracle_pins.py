"""Pins for the fp64 oracle: closed forms, invariants, special cases, brute force, and an
independent library composition.  None of these needs a GPU.

The paper prints no worked example of the action head, so the pins are what the mathematics
fixes.  Each is chosen so that a plausible mistake (dropped term, wrong sign or index,
transposed operand, wrong head slice) fails at least one of them.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2609_27547_b200 import synth
from helpers import oracle_cfg, oracle_weights, oracle_run, np32

SEED = 1234


def small(**kw):
    base = dict(name="t", dtype="f32", B=4, H=4, A=3, d=16, L=2, n_heads=2, K=4, P=(5, 5),
                group=None, quota=0)
    base.update(kw)
    return synth.Workload(**base)


def zero_matrices(wt):
    for k in ("w_in", "w_out"):
        wt[k].zero_()
    for l in wt["layers"]:
        for k in ("w_qkv", "w_o", "w_qc", "w_oc", "w_1", "w_2"):
            l[k].zero_()
    return wt


# ---------------------------------------------------------------- Euler loop + output bias

def test_zero_weights_gives_a0_plus_b():
    """All matrices zero: v = b every step, so a_K = a_0 + b."""
    w = small()
    wt = zero_matrices(synth.make_weights(w, SEED))
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    out = oracle_run(w, wt, envs)
    for i, e in enumerate(envs):
        want = np32(e.noise).astype(np.float64) + np32(wt["b_out"]).astype(np.float64)[None, :]
        assert np.abs(out[i] - want).max() < 1e-14


@pytest.mark.parametrize("k0,s", [(0, 1), (1, 2), (2, 0), (3, 5)])
def test_zero_weights_partial_steps(k0, s):
    """From step k0, advancing s steps (0 = to the end, never beyond K): a = a_k0 + n*b/K."""
    w = small()
    wt = zero_matrices(synth.make_weights(w, SEED))
    e = synth.make_env(w, 0, SEED)
    e.step = k0
    out = oracle_run(w, wt, [e], n_steps=s)[0]
    n = (w.K - k0) if s == 0 else min(s, w.K - k0)
    want = np32(e.noise).astype(np.float64) + n * np32(wt["b_out"]).astype(np.float64)[None, :] / w.K
    assert np.abs(out - want).max() < 1e-14


@pytest.mark.parametrize("K", [1, 2, 4, 10])
def test_pull_field_closed_form(K):
    """v = c - a under explicit Euler with step 1/K: a_K = c + (a_0 - c)(1 - 1/K)^K."""
    w = small(K=K)
    wt = synth.make_weights(w, SEED)
    cfg, ow = oracle_cfg(w), oracle_weights(wt)
    a0 = np32(synth.normal(SEED, "noise", 0, (3, w.H, w.A)))
    c = np32(wt["b_out"]).astype(np.float64)
    out = oracle.actgen(cfg, ow, [], a0, pull=True)
    want = c[None, None, :] + (a0.astype(np.float64) - c[None, None, :]) * (1.0 - 1.0 / K) ** K
    assert np.abs(out - want).max() < 1e-14
    if K >= 4:   # starting at step k0 leaves K - k0 contractions
        out = oracle.actgen(cfg, ow, [], a0, step_index=[1, 2, 3], pull=True)
        for i, k0 in enumerate([1, 2, 3]):
            want = c[None, :] + (a0[i].astype(np.float64) - c[None, :]) * (1.0 - 1.0 / K) ** (K - k0)
            assert np.abs(out[i] - want).max() < 1e-14


# ---------------------------------------------------------------- timestep embedding

def test_temb_special_values():
    cfg = oracle.OracleConfig(H=1, A=1, d=64, n_layers=0, n_heads=1, K_steps=10)
    t0 = oracle.timestep_embedding(cfg, 0)
    assert np.all(t0[:32] == 0.0) and np.all(t0[32:] == 1.0)
    for k in (1, 3, 9):
        t = oracle.timestep_embedding(cfg, k)
        tau = 1000.0 * k / 10
        assert abs(t[0] - math.sin(tau)) < 1e-15 and abs(t[32] - math.cos(tau)) < 1e-15
        # j = 16 is halfway: w = 10000^(-1/2) = 0.01
        assert abs(t[16] - math.sin(tau * 0.01)) < 1e-13
        assert abs(t[48] - math.cos(tau * 0.01)) < 1e-13
        # last frequency: 10000^(-31/32)
        assert abs(t[31] - math.sin(tau * 10000.0 ** (-31.0 / 32.0))) < 1e-13
        assert abs(np.sum(t * t) - 32.0) < 1e-12          # sin^2 + cos^2 per frequency


def test_no_layers_no_embedding_is_hand_computable():
    """L = 0 and W_in = 0: x = temb, sum(temb^2) = d/2, so
    v = W_out (g * temb / sqrt(1/2 + eps)) + b."""
    w = small(L=0, d=8, K=5, H=2, A=3)
    wt = synth.make_weights(w, SEED, random_gains=True)
    wt["w_in"].zero_()
    cfg, ow = oracle_cfg(w), oracle_weights(wt)
    a = np.zeros((w.H, w.A))
    k = 3
    tau = 1000.0 * k / 5
    temb = np.array([math.sin(tau * 10000.0 ** (-j / 4.0)) for j in range(4)] +
                    [math.cos(tau * 10000.0 ** (-j / 4.0)) for j in range(4)])
    y = np32(wt["g_final"]).astype(np.float64) * temb / math.sqrt(0.5 + 1e-6)
    want = np32(wt["w_out"]).astype(np.float64) @ y + np32(wt["b_out"]).astype(np.float64)
    v = oracle.velocity(cfg, ow, np.zeros((1, 2, 1, w.d), np.float32), a, k)
    assert np.abs(v - want[None, :]).max() < 1e-13


# ---------------------------------------------------------------- RMSNorm, GELU, softmax

def test_rmsnorm_properties():
    rng = np.random.default_rng(0)
    x = rng.standard_normal(32)
    g = (1.0 + 0.1 * rng.standard_normal(32)).astype(np.float32)
    y = oracle.rmsnorm(x, g, eps=0.0)
    assert np.abs(oracle.rmsnorm(7.5 * x, g, eps=0.0) - y).max() < 1e-14      # scale invariance
    assert abs(np.mean((y / g) ** 2) - 1.0) < 1e-14                            # unit mean square
    c = oracle.rmsnorm(np.full(32, -3.0), g, eps=0.0)
    assert np.abs(c + g).max() < 1e-15                                         # constant -> g*sign
    # eps sits inside the square root, added to the mean square
    z = oracle.rmsnorm(np.zeros(4) + 1e-3, np.ones(4, np.float32), eps=1e-6)
    assert np.abs(z - 1e-3 / math.sqrt(1e-6 + 1e-6)).max() < 1e-15


def test_gelu_values():
    assert oracle.gelu(0.0) == 0.0
    for z in (-3.0, -1.0, -0.1, 0.5, 2.0, 6.0):
        assert abs(oracle.gelu(z) - 0.5 * z * (1.0 + math.erf(z / math.sqrt(2.0)))) < 1e-15
        assert abs(oracle.gelu(z) - oracle.gelu(-z) - z) < 1e-15
    assert abs(oracle.gelu(1.0) - 0.8413447460685429) < 1e-15     # Phi(1)
    # the tanh approximation differs visibly; make sure the exact form is what is computed
    z = 2.0
    tanh_form = 0.5 * z * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)))
    assert abs(oracle.gelu(z) - tanh_form) > 5e-5


def test_softmax_row():
    s = oracle.softmax_row([1.0, 2.0, 3.0])
    e = np.exp([1.0, 2.0, 3.0])
    assert np.abs(s - e / e.sum()).max() < 1e-15
    big = oracle.softmax_row([1000.0, 1000.0, -1000.0])          # needs the max subtraction
    assert np.abs(big - np.array([0.5, 0.5, 0.0])).max() < 1e-15
    assert oracle.softmax_row([42.0])[0] == 1.0


def test_attention_head_special_cases():
    rng = np.random.default_rng(1)
    q = rng.standard_normal((3, 4))
    k = rng.standard_normal((6, 4)).astype(np.float32)
    v = rng.standard_normal((6, 4)).astype(np.float32)
    # one key: softmax of a single score is 1, output = that value row whatever q is
    o = oracle.attention_head(q, k[:1], v[:1])
    assert np.abs(o - v[:1].astype(np.float64)).max() == 0.0
    # zero queries: uniform weights, output = column means of v
    o = oracle.attention_head(np.zeros((3, 4)), k, v)
    assert np.abs(o - v.astype(np.float64).mean(axis=0)[None, :]).max() < 1e-15
    # definition, written with numpy; scale 1/sqrt(hd)
    s = q @ k.astype(np.float64).T / 2.0
    p = np.exp(s - s.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    assert np.abs(oracle.attention_head(q, k, v) - p @ v.astype(np.float64)).max() < 1e-14
    # a query aligned with one key and scaled up picks that key's value
    qq = np.zeros((1, 4)); qq[0] = 200.0 * k[2]
    kk = k.copy(); kk[2] *= 3.0
    assert np.abs(oracle.attention_head(qq, kk, v)[0] - v[2]).max() < 1e-9


# ---------------------------------------------------------------- whole-network special cases

def _only_cross(w, wt):
    """Keep only the cross-attention branch alive: W_o = 0 and W_2 = 0."""
    for l in wt["layers"]:
        l["w_o"].zero_()
        l["w_2"].zero_()
    return wt


def _embed(w, wt, a, k):
    cfg = oracle_cfg(w)
    temb = np.array([math.sin(cfg.temb_scale * k / w.K * cfg.temb_max_period ** (-j / (w.d / 2)))
                     for j in range(w.d // 2)] +
                    [math.cos(cfg.temb_scale * k / w.K * cfg.temb_max_period ** (-j / (w.d / 2)))
                     for j in range(w.d // 2)])
    return a @ np32(wt["w_in"]).astype(np.float64).T + temb[None, :]


def _head(w, wt, x):
    g = np32(wt["g_final"]).astype(np.float64)
    y = g[None, :] * x / np.sqrt((x * x).mean(axis=1, keepdims=True) + 1e-6)
    return y @ np32(wt["w_out"]).astype(np.float64).T + np32(wt["b_out"]).astype(np.float64)[None, :]


def test_single_prefix_token_cross_attention():
    """P = 1: every head's softmax is 1, so each layer adds W_oc V[0] to every token."""
    w = small(P=(1, 1), L=2)
    wt = _only_cross(w, synth.make_weights(w, SEED, random_gains=True))
    e = synth.make_env(w, 0, SEED)
    a = np32(e.noise).astype(np.float64)
    x = _embed(w, wt, a, 2)
    v0 = np32(e.kv)[0, 1, 0].astype(np.float64)
    for l in wt["layers"]:
        x = x + (np32(l["w_oc"]).astype(np.float64) @ v0)[None, :]
    want = _head(w, wt, x)
    got = oracle.velocity(oracle_cfg(w), oracle_weights(wt), np32(e.kv), a, 2)
    assert np.abs(got - want).max() < 1e-12


def test_zero_query_projection_gives_prefix_mean():
    """W_qc = 0: uniform attention, each layer adds W_oc mean_p V[p]."""
    w = small(P=(7, 7), L=1)
    wt = _only_cross(w, synth.make_weights(w, SEED))
    wt["layers"][0]["w_qc"].zero_()
    e = synth.make_env(w, 1, SEED)
    a = np32(e.noise).astype(np.float64)
    x = _embed(w, wt, a, 1)
    vbar = np32(e.kv)[0, 1].astype(np.float64).mean(axis=0)
    x = x + (np32(wt["layers"][0]["w_oc"]).astype(np.float64) @ vbar)[None, :]
    got = oracle.velocity(oracle_cfg(w), oracle_weights(wt), np32(e.kv), a, 1)
    assert np.abs(got - _head(w, wt, x)).max() < 1e-12


def test_head_slices_of_values():
    """Values constant within a head's columns: softmax weights sum to 1, so the attention
    output is that constant in that head's columns whatever the scores are."""
    w = small(P=(6, 6), L=1, n_heads=4, d=16)
    wt = _only_cross(w, synth.make_weights(w, SEED))
    e = synth.make_env(w, 2, SEED)
    kv = np32(e.kv).copy()
    consts = np.array([0.5, -1.25, 2.0, 3.5])
    for h in range(4):
        kv[0, 1, :, 4 * h:4 * h + 4] = consts[h]
    a = np32(e.noise).astype(np.float64)
    x = _embed(w, wt, a, 0)
    att = np.repeat(consts, 4)
    x = x + (np32(wt["layers"][0]["w_oc"]).astype(np.float64) @ att)[None, :]
    got = oracle.velocity(oracle_cfg(w), oracle_weights(wt), kv, a, 0)
    assert np.abs(got - _head(w, wt, x)).max() < 1e-12


def test_head_slices_of_keys():
    """Keys zero in head 1's columns: head 1 attends uniformly (mean of its value columns);
    with W_oc reading only head 1's columns the result is known exactly."""
    w = small(P=(5, 5), L=1, n_heads=2, d=16)
    wt = _only_cross(w, synth.make_weights(w, SEED))
    wt["layers"][0]["w_oc"][:, :8] = 0.0
    e = synth.make_env(w, 3, SEED)
    kv = np32(e.kv).copy()
    kv[0, 0, :, 8:] = 0.0
    a = np32(e.noise).astype(np.float64)
    x = _embed(w, wt, a, 3)
    att = np.zeros(16)
    att[8:] = kv[0, 1, :, 8:].astype(np.float64).mean(axis=0)
    x = x + (np32(wt["layers"][0]["w_oc"]).astype(np.float64) @ att)[None, :]
    got = oracle.velocity(oracle_cfg(w), oracle_weights(wt), kv, a, 3)
    assert np.abs(got - _head(w, wt, x)).max() < 1e-12


def test_self_attention_single_token_and_uniform():
    """H = 1: self-attention output = v of that token, so the layer adds W_o W_v RMSNorm(x).
    W_q = 0 with H > 1: uniform weights, every token receives W_o mean_h(v_h)."""
    for H, zero_q in ((1, False), (3, True)):
        w = small(H=H, L=1, P=(2, 2))
        wt = synth.make_weights(w, SEED, random_gains=True)
        l = wt["layers"][0]
        l["w_oc"].zero_(); l["w_2"].zero_()
        if zero_q:
            l["w_qkv"][:w.d].zero_()
        e = synth.make_env(w, 0, SEED)
        a = np32(e.noise).astype(np.float64)
        x = _embed(w, wt, a, 1)
        g1 = np32(l["g1"]).astype(np.float64)
        y = g1[None, :] * x / np.sqrt((x * x).mean(axis=1, keepdims=True) + 1e-6)
        vv = y @ np32(l["w_qkv"]).astype(np.float64)[2 * w.d:].T
        mix = vv.mean(axis=0, keepdims=True) if zero_q else vv
        x = x + mix @ np32(l["w_o"]).astype(np.float64).T
        got = oracle.velocity(oracle_cfg(w), oracle_weights(wt), np32(e.kv), a, 1)
        assert np.abs(got - _head(w, wt, x)).max() < 1e-12


def test_prefix_duplication_and_permutation_invariance():
    w = small(P=(9, 9))
    wt = synth.make_weights(w, SEED, random_gains=True)
    e = synth.make_env(w, 0, SEED)
    base = oracle_run(w, wt, [e])[0]
    kv = np32(e.kv)
    dup = np.concatenate([kv, kv], axis=2)                     # every token twice
    perm = kv[:, :, np.random.default_rng(3).permutation(9), :]   # K and V rows moved together
    cfg, ow = oracle_cfg(w), oracle_weights(wt)
    for alt in (dup, perm):
        out = oracle.actgen(cfg, ow, [alt], np32(e.noise)[None])[0]
        assert np.abs(out - base).max() < 1e-12
    # moving K rows without V rows must change the result (the test above is not vacuous)
    bad = kv.copy(); bad[0, 0] = bad[0, 0, ::-1]
    assert np.abs(oracle.actgen(cfg, ow, [bad], np32(e.noise)[None])[0] - base).max() > 1e-6


def test_action_token_permutation_equivariance():
    """No positional term over the H tokens: permuting the noise rows permutes the output."""
    w = small(H=5)
    wt = synth.make_weights(w, SEED, random_gains=True)
    e = synth.make_env(w, 0, SEED)
    base = oracle_run(w, wt, [e])[0]
    perm = np.array([3, 0, 4, 1, 2])
    out = oracle.actgen(oracle_cfg(w), oracle_weights(wt), [np32(e.kv)], np32(e.noise)[perm][None])[0]
    assert np.abs(out - base[perm]).max() < 1e-12


def test_group_composition_order_and_threads_do_not_matter():
    w = small(B=6, P=(3, 9), mixed_steps=True)
    wt = synth.make_weights(w, SEED)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    assert len({e.P for e in envs}) > 1 and len({e.step for e in envs}) > 1
    together = oracle_run(w, wt, envs, n_threads=3)
    for i, e in enumerate(envs):
        alone = oracle_run(w, wt, [e], n_threads=1)[0]
        assert np.array_equal(alone, together[i])
    rev = oracle_run(w, wt, envs[::-1], n_threads=8)
    assert np.array_equal(rev[::-1], together)


# ---------------------------------------------------------------- brute force, tiny

def test_tiny_case_by_scalar_arithmetic():
    """H = A = 1, d = 2, one head, one layer, two prefix tokens, K = 2, written out scalar by
    scalar with python floats (every quantity is a 2-vector)."""
    w = small(H=1, A=1, d=2, L=1, n_heads=1, K=2, P=(2, 2), mlp_mult=1)
    win = [0.7, -0.4]; wout = [0.3, 0.9]; b = 0.05; gf = [1.1, 0.8]
    g1 = [0.9, 1.2]; g2 = [1.0, 0.7]; g3 = [1.3, 1.0]
    wqkv = [[0.2, -0.1], [0.4, 0.3], [0.5, 0.6], [-0.7, 0.8], [0.15, -0.25], [0.35, 0.45]]
    wo = [[0.6, -0.2], [0.1, 0.5]]; wqc = [[0.3, 0.7], [-0.5, 0.2]]; woc = [[0.25, 0.4], [-0.6, 0.1]]
    w1 = [[0.8, -0.3], [0.2, 0.9]]; w2 = [[-0.4, 0.5], [0.7, 0.3]]
    Kc = [[0.5, -1.0], [1.5, 0.25]]; Vc = [[2.0, -0.5], [-1.0, 0.75]]
    a0 = 0.6

    def rms(x, g):
        r = math.sqrt((x[0] * x[0] + x[1] * x[1]) / 2.0 + 1e-6)
        return [g[0] * x[0] / r, g[1] * x[1] / r]

    def mv(W, x):
        return [sum(W[o][i] * x[i] for i in range(len(x))) for o in range(len(W))]

    def gelu(z):
        return 0.5 * z * (1.0 + math.erf(z / math.sqrt(2.0)))

    a = a0
    for k in range(2):
        tau = 1000.0 * k / 2
        x = [win[0] * a + math.sin(tau), win[1] * a + math.cos(tau)]      # d/2 = 1: w_0 = 1
        qkv = mv(wqkv, rms(x, g1))
        s = qkv[4:6]                                   # one token: self-attention returns v
        x = [x[i] + mv(wo, s)[i] for i in range(2)]
        qc = mv(wqc, rms(x, g2))
        sc = [(qc[0] * Kc[j][0] + qc[1] * Kc[j][1]) / math.sqrt(2.0) for j in range(2)]
        m = max(sc); ex = [math.exp(t - m) for t in sc]; z = ex[0] + ex[1]
        c = [(ex[0] * Vc[0][i] + ex[1] * Vc[1][i]) / z for i in range(2)]
        x = [x[i] + mv(woc, c)[i] for i in range(2)]
        u = [gelu(t) for t in mv(w1, rms(x, g3))]
        x = [x[i] + mv(w2, u)[i] for i in range(2)]
        y = rms(x, gf)
        v = wout[0] * y[0] + wout[1] * y[1] + b
        a = a + v / 2.0

    f32 = lambda z: np.array(z, dtype=np.float32)
    ow = oracle.OracleWeights(
        w_in=f32(win).reshape(2, 1), w_out=f32(wout).reshape(1, 2), b_out=f32([b]), g_final=f32(gf),
        layers=[dict(g1=f32(g1), g2=f32(g2), g3=f32(g3), w_qkv=f32(wqkv), w_o=f32(wo),
                     w_qc=f32(wqc), w_oc=f32(woc), w_1=f32(w1), w_2=f32(w2))])
    kv = f32([Kc, Vc]).reshape(1, 2, 2, 2)
    out = oracle.actgen(oracle_cfg(w), ow, [kv], f32([[[a0]]]))
    # the python-float reference uses the decimal constants; the oracle sees them rounded to
    # fp32, hence the 1e-6 tolerance instead of 1e-15
    assert abs(out[0, 0, 0] - a) < 2e-6
    # and exactly, with the same fp32-rounded constants fed to the scalar code
    r = lambda z: [float(np.float32(t)) for t in z]
    win, wout, gf, g1, g2, g3 = map(r, (win, wout, gf, g1, g2, g3))
    b = float(np.float32(b)); a0 = float(np.float32(a0))
    wqkv, wo, wqc, woc, w1, w2, Kc, Vc = [[r(row) for row in M] for M in (wqkv, wo, wqc, woc, w1, w2, Kc, Vc)]
    a = a0
    for k in range(2):
        tau = 1000.0 * k / 2
        x = [win[0] * a + math.sin(tau), win[1] * a + math.cos(tau)]
        qkv = mv(wqkv, rms(x, g1)); s = qkv[4:6]
        x = [x[i] + mv(wo, s)[i] for i in range(2)]
        qc = mv(wqc, rms(x, g2))
        sc = [(qc[0] * Kc[j][0] + qc[1] * Kc[j][1]) / math.sqrt(2.0) for j in range(2)]
        m = max(sc); ex = [math.exp(t - m) for t in sc]; z = ex[0] + ex[1]
        c = [(ex[0] * Vc[0][i] + ex[1] * Vc[1][i]) / z for i in range(2)]
        x = [x[i] + mv(woc, c)[i] for i in range(2)]
        u = [gelu(t) for t in mv(w1, rms(x, g3))]
        x = [x[i] + mv(w2, u)[i] for i in range(2)]
        y = rms(x, gf)
        a = a + (wout[0] * y[0] + wout[1] * y[1] + b) / 2.0
    assert abs(out[0, 0, 0] - a) < 1e-13


# ---------------------------------------------------------------- library composition

def _torch_reference(w, wt, env, n_steps=0, planes=None):
    """The same network composed from torch's own fp64 routines (rms_norm, softmax, erf-GELU,
    matmul), vectorised over tokens and heads: independent of the C loops.  ``planes`` [L][2][P][d]
    gives every layer its own K/V pair (kv_layers = n_layers) instead of the environment's shared one."""
    F = torch.nn.functional
    D = torch.float64
    H, d, nh, hd = w.H, w.d, w.n_heads, w.head_dim
    a = env.noise.to(D)
    if w.d_ctx == 0:
        Kc, Vc = env.kv[0, 0].to(D), env.kv[0, 1].to(D)
    k1 = w.K if n_steps == 0 else min(w.K, env.step + n_steps)
    for k in range(env.step, k1):
        j = torch.arange(d // 2, dtype=D)
        ang = (1000.0 * k / w.K) * torch.pow(torch.tensor(10000.0, dtype=D), -j / (d // 2))
        x = a @ wt["w_in"].to(D).T + torch.cat([torch.sin(ang), torch.cos(ang)])[None, :]
        for li, l in enumerate(wt["layers"]):
            y = F.rms_norm(x, (d,), l["g1"].to(D), 1e-6)
            q, kk, v = (y @ l["w_qkv"].to(D).T).split(d, dim=1)
            sh = lambda t, n: t.reshape(n, nh, hd).transpose(0, 1)
            p = torch.softmax(sh(q, H) @ sh(kk, H).transpose(1, 2) / math.sqrt(hd), dim=-1)
            x = x + (p @ sh(v, H)).transpose(0, 1).reshape(H, d) @ l["w_o"].to(D).T
            y = F.rms_norm(x, (d,), l["g2"].to(D), 1e-6)
            qc = y @ l["w_qc"].to(D).T
            if w.d_ctx > 0:   # this layer's keys and values from the prefix's hidden states
                Kc, Vc = env.kv.to(D) @ l["w_kc"].to(D).T, env.kv.to(D) @ l["w_vc"].to(D).T
            elif planes is not None:   # this layer's own cached pair
                Kc, Vc = planes[li, 0].to(D), planes[li, 1].to(D)
            P = Kc.shape[0]
            p = torch.softmax(sh(qc, H) @ sh(Kc, P).transpose(1, 2) / math.sqrt(hd), dim=-1)
            x = x + (p @ sh(Vc, P)).transpose(0, 1).reshape(H, d) @ l["w_oc"].to(D).T
            y = F.rms_norm(x, (d,), l["g3"].to(D), 1e-6)
            x = x + F.gelu(y @ l["w_1"].to(D).T, approximate="none") @ l["w_2"].to(D).T
        y = F.rms_norm(x, (d,), wt["g_final"].to(D), 1e-6)
        a = a + (y @ wt["w_out"].to(D).T + wt["b_out"].to(D)[None, :]) / w.K
    return a.numpy()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_against_torch_fp64_composition(dtype):
    w = synth.scaled(synth.WORKLOADS[0], B=3, dtype=dtype, P=(17, 40), mixed_steps=True)
    wt = synth.make_weights(w, SEED, random_gains=True)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    got = oracle_run(w, wt, envs)
    for i, e in enumerate(envs):
        assert np.abs(got[i] - _torch_reference(w, wt, e)).max() < 1e-11
    got1 = oracle_run(w, wt, envs, n_steps=1)
    for i, e in enumerate(envs):
        assert np.abs(got1[i] - _torch_reference(w, wt, e, n_steps=1)).max() < 1e-11


# ---------------------------------------------------------------- per-layer prefix planes (kv_layers = n_layers)

def _layer_planes(w, env_id, P):
    return synth.normal(SEED, "kv_per_layer", env_id, (w.L, 2, P, w.d), dtype=w.torch_dtype)


def _per_layer_cfg(w):
    oc = oracle_cfg(w)
    oc.kv_layers = w.L
    return oc


def test_per_layer_planes_uniform_attention_closed_form():
    """kv_layers = n_layers with W_qc = 0 and only the cross-attention branch alive: the softmax is
    uniform, so layer l adds W_oc_l mean_p V_l[p] -- its OWN value plane -- to every token.  A wrong
    plane stride, a K/V swap or a layer mix-up all change the sum."""
    w = small(P=(6, 6), L=3)
    wt = _only_cross(w, synth.make_weights(w, SEED, random_gains=True))
    for l in wt["layers"]:
        l["w_qc"].zero_()
    e = synth.make_env(w, 2, SEED)
    planes = _layer_planes(w, 2, e.P)
    a = np32(e.noise).astype(np.float64)
    x = _embed(w, wt, a, 3)
    for li, l in enumerate(wt["layers"]):
        vbar = np32(planes)[li, 1].astype(np.float64).mean(axis=0)
        x = x + (np32(l["w_oc"]).astype(np.float64) @ vbar)[None, :]
    got = oracle.velocity(_per_layer_cfg(w), oracle_weights(wt), np32(planes), a, 3)
    assert np.abs(got - _head(w, wt, x)).max() < 1e-12
    # the key planes play no part here, the value planes all do
    other = np32(planes).copy()
    other[:, 0] = 7.0
    assert np.abs(oracle.velocity(_per_layer_cfg(w), oracle_weights(wt), other, a, 3) - got).max() < 1e-12
    for li in range(w.L):
        other = np32(planes).copy()
        other[li, 1] += 1.0
        assert np.abs(oracle.velocity(_per_layer_cfg(w), oracle_weights(wt), other, a, 3) - got).max() > 1e-3


def test_per_layer_planes_single_token_closed_form():
    """P = 1 and per-layer planes: layer l adds W_oc_l V_l[0] whatever the queries and keys are."""
    w = small(P=(1, 1), L=2)
    wt = _only_cross(w, synth.make_weights(w, SEED, random_gains=True))
    e = synth.make_env(w, 0, SEED)
    planes = _layer_planes(w, 0, 1)
    a = np32(e.noise).astype(np.float64)
    x = _embed(w, wt, a, 1)
    for li, l in enumerate(wt["layers"]):
        x = x + (np32(l["w_oc"]).astype(np.float64) @ np32(planes)[li, 1, 0].astype(np.float64))[None, :]
    got = oracle.velocity(_per_layer_cfg(w), oracle_weights(wt), np32(planes), a, 1)
    assert np.abs(got - _head(w, wt, x)).max() < 1e-12


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_per_layer_planes_against_torch_fp64_composition(dtype):
    """The whole network with a K/V pair per layer against the torch composition, and the checks
    that make the layout matter: swapping two layers' pairs, or K and V inside one layer, changes
    the result; repeating one pair for every layer reproduces the shared-plane form exactly."""
    w = synth.scaled(synth.WORKLOADS[0], B=3, dtype=dtype, L=3, P=(9, 33), mixed_steps=True)
    wt = synth.make_weights(w, SEED, random_gains=True)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    planes = [_layer_planes(w, e.env_id, e.P) for e in envs]

    def run(pl, n_steps=0):
        return oracle.actgen(_per_layer_cfg(w), oracle_weights(wt), [np32(p) for p in pl],
                             np.stack([np32(e.noise) for e in envs]), step_index=[e.step for e in envs], n_steps=n_steps)

    got = run(planes)
    for i, e in enumerate(envs):
        assert np.abs(got[i] - _torch_reference(w, wt, e, planes=planes[i])).max() < 1e-11
    got1 = run(planes, n_steps=1)
    for i, e in enumerate(envs):
        assert np.abs(got1[i] - _torch_reference(w, wt, e, n_steps=1, planes=planes[i])).max() < 1e-11
    assert np.abs(run([p[[1, 0, 2]] for p in planes]) - got).max() > 1e-4          # layers 0 and 1 exchanged
    assert np.abs(run([p[[0, 2, 1]] for p in planes]) - got).max() > 1e-4          # layers 1 and 2 exchanged
    kvswap = [p.clone() for p in planes]
    for p in kvswap:
        p[2] = p[2].flip(0)                                                        # K <-> V in the last layer only
    assert np.abs(run(kvswap) - got).max() > 1e-4
    shared = oracle_run(w, wt, envs)                                               # kv_layers = 1 on each env's own pair
    rep = run([e.kv.expand(w.L, -1, -1, -1).contiguous() for e in envs])
    assert np.array_equal(rep, shared)


# ---------------------------------------------------------------- hidden-state prefixes

def test_hidden_prefix_with_identity_projections_is_the_plane_form():
    """d_ctx = d and W_kc = W_vc = I in every layer: keys and values are the hidden states
    themselves, i.e. the cached-plane form with K = V = h (exact: the products add only zeros)."""
    w = small(d_ctx=16)
    wt = synth.make_weights(w, SEED, random_gains=True)
    for l in wt["layers"]:
        l["w_kc"] = torch.eye(w.d)
        l["w_vc"] = torch.eye(w.d)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    got = oracle_run(w, wt, envs)
    wp = small()
    plane_envs = [synth.EnvInputs(e.env_id, e.noise, torch.stack([e.kv, e.kv])[None], e.P, e.step) for e in envs]
    want = oracle_run(wp, wt, plane_envs)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_hidden_prefix_against_torch_fp64_composition(dtype):
    """Per-layer K = h W_kc^T, V = h W_vc^T composed from torch matmuls: pins the orientation of the
    projections, which of the two feeds keys and which values, and the layer each pair belongs to."""
    w = synth.scaled(synth.WORKLOADS[0], B=3, dtype=dtype, P=(9, 33), mixed_steps=True, d_ctx=64)
    wt = synth.make_weights(w, SEED, random_gains=True)
    envs = [synth.make_env(w, e, SEED) for e in range(w.B)]
    assert envs[0].kv.shape == (envs[0].P, 64) and wt["layers"][1]["w_kc"].shape == (w.d, 64)
    got = oracle_run(w, wt, envs)
    for i, e in enumerate(envs):
        assert np.abs(got[i] - _torch_reference(w, wt, e)).max() < 1e-11
    # swapping the two projections, or the two layers' projections, must change the result
    sw = {**wt, "layers": [{**l, "w_kc": l["w_vc"], "w_vc": l["w_kc"]} for l in wt["layers"]]}
    assert np.abs(oracle_run(w, sw, envs) - got).max() > 1e-4
    l0, l1 = wt["layers"]
    sl = {**wt, "layers": [{**l0, "w_kc": l1["w_kc"], "w_vc": l1["w_vc"]}, {**l1, "w_kc": l0["w_kc"], "w_vc": l0["w_vc"]}]}
    assert np.abs(oracle_run(w, sl, envs) - got).max() > 1e-4


def test_hidden_prefix_single_token_closed_form():
    """P = 1: the softmax over one key is 1, so the cross-attention block adds W_oc W_vc h_0 to
    every token whatever the queries and W_kc are; with the other blocks silenced,
    v = W_out RMSNorm(x0 + W_oc W_vc h_0) + b."""
    w = small(L=1, K=1, P=(1, 1), d_ctx=64)
    wt = _only_cross(w, synth.make_weights(w, SEED, random_gains=True))
    e = synth.make_env(w, 0, SEED)
    l = wt["layers"][0]
    x = _embed(w, wt, np32(e.noise), 0)
    add = np32(l["w_oc"]).astype(np.float64) @ (np32(l["w_vc"]).astype(np.float64) @ np32(e.kv).astype(np.float64)[0])
    want = np32(e.noise) + _head(w, wt, x + add[None, :])
    got = oracle_run(w, wt, [e])[0]
    assert np.abs(got - want).max() < 1e-12
    l["w_kc"] = torch.zeros_like(l["w_kc"])
    assert np.abs(oracle_run(w, wt, [e])[0] - want).max() < 1e-12


def test_golden_regression():
    """Stored outputs written by tests/golden/make_golden.py (which calls only the oracle):
    guards the oracle against silent changes."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "oracle_cfg0_first4.txt")
    want = np.loadtxt(path).reshape(4, 8, 7)
    w = synth.WORKLOADS[0]
    wt = synth.make_weights(w, synth.DEFAULT_SEED)
    envs = [synth.make_env(w, e, synth.DEFAULT_SEED) for e in range(4)]
    assert np.abs(oracle_run(w, wt, envs) - want).max() < 1e-12
