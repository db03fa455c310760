"""fp64 CPU oracle for batched action generation -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the bench's CPU-baseline leg may import this package.  It
wraps ``actgen_oracle.c`` (plain C, fp64, threads across environments only) with ctypes and
numpy.  It shares nothing with the CUDA path and never imports it.

The functions follow the paper's outline of action generation (section 2.1: an action head
denoises a random tensor into an action chunk over several steps, conditioned on the backbone's
cached K/V; section 4.2.2: environments are independent) with the concrete head the benchmark
configurations state.  That this architecture is the one used by the paper's policies is
"parity unpinned" by the paper; every arithmetic piece is pinned in ``tests/test_oracle_pins.py``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "actgen_oracle.c")
_LIB = os.path.join(_HERE, "libebrl_oracle.so")


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no contraction) and return the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm", "-lpthread"])
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [("H", C.c_int32), ("A", C.c_int32), ("d", C.c_int32), ("n_layers", C.c_int32),
                ("n_heads", C.c_int32), ("mlp_mult", C.c_int32), ("K_steps", C.c_int32),
                ("kv_layers", C.c_int32), ("rms_eps", C.c_double), ("temb_scale", C.c_double),
                ("temb_max_period", C.c_double), ("d_ctx", C.c_int32)]


_FP = C.POINTER(C.c_float)
_FPP = C.POINTER(_FP)


class _Weights(C.Structure):
    _fields_ = [("w_in", _FP), ("w_out", _FP), ("b_out", _FP), ("g_final", _FP),
                ("g1", _FPP), ("g2", _FPP), ("g3", _FPP), ("w_qkv", _FPP), ("w_o", _FPP),
                ("w_qc", _FPP), ("w_oc", _FPP), ("w_1", _FPP), ("w_2", _FPP), ("w_kc", _FPP), ("w_vc", _FPP)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.ebrl_oracle_gelu.restype = C.c_double
        lib.ebrl_oracle_gelu.argtypes = [C.c_double]
        lib.ebrl_oracle_actgen.restype = C.c_int
        lib.ebrl_oracle_velocity.restype = C.c_int
        _lib = lib
    return _lib


@dataclass
class OracleConfig:
    H: int
    A: int
    d: int
    n_layers: int
    n_heads: int
    K_steps: int
    mlp_mult: int = 4
    kv_layers: int = 1
    rms_eps: float = 1e-6
    temb_scale: float = 1000.0
    temb_max_period: float = 10000.0
    d_ctx: int = 0     # > 0: prefixes are hidden states [P][d_ctx]; layers carry w_kc, w_vc [d][d_ctx]

    def _c(self) -> _Cfg:
        return _Cfg(self.H, self.A, self.d, self.n_layers, self.n_heads, self.mlp_mult,
                    self.K_steps, self.kv_layers, self.rms_eps, self.temb_scale,
                    self.temb_max_period, self.d_ctx)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _fp(a: np.ndarray):
    return a.ctypes.data_as(_FP)


@dataclass
class OracleWeights:
    """Weights as float32 numpy arrays (bf16 models pass values already rounded to bf16).

    ``layers`` is a list of dicts with keys g1, g2, g3, w_qkv, w_o, w_qc, w_oc, w_1, w_2 (and
    w_kc, w_vc [d][d_ctx] when the prefix is given as hidden states).
    All matrices are [out][in] row-major: y = W x.
    """
    w_in: np.ndarray
    w_out: np.ndarray
    b_out: np.ndarray
    g_final: np.ndarray
    layers: List[dict] = field(default_factory=list)

    def _c(self):
        keep = []
        w = _Weights()
        for name in ("w_in", "w_out", "b_out", "g_final"):
            arr = _f32(getattr(self, name))
            keep.append(arr)
            setattr(w, name, _fp(arr))
        for name in ("g1", "g2", "g3", "w_qkv", "w_o", "w_qc", "w_oc", "w_1", "w_2", "w_kc", "w_vc"):
            if name in ("w_kc", "w_vc") and not all(name in l for l in self.layers):
                continue   # only models with hidden-state prefixes carry them
            arrs = [_f32(l[name]) for l in self.layers]
            keep.extend(arrs)
            ptrs = (_FP * max(1, len(arrs)))(*[_fp(a) for a in arrs])
            keep.append(ptrs)
            setattr(w, name, C.cast(ptrs, _FPP))
        return w, keep


def timestep_embedding(cfg: OracleConfig, k: int) -> np.ndarray:
    out = np.zeros(cfg.d, dtype=np.float64)
    c = cfg._c()
    _load().ebrl_oracle_timestep_embedding(C.byref(c), C.c_int(k), out.ctypes.data_as(C.c_void_p))
    return out


def rmsnorm(x, g, eps: float = 1e-6) -> np.ndarray:
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    g = _f32(g)
    y = np.zeros_like(x)
    _load().ebrl_oracle_rmsnorm(x.ctypes.data_as(C.c_void_p), _fp(g), C.c_int(x.shape[0]),
                                C.c_double(eps), y.ctypes.data_as(C.c_void_p))
    return y


def gelu(z: float) -> float:
    return float(_load().ebrl_oracle_gelu(float(z)))


def softmax_row(s) -> np.ndarray:
    s = np.array(s, dtype=np.float64, copy=True)
    _load().ebrl_oracle_softmax_row(s.ctypes.data_as(C.c_void_p), C.c_int(s.shape[0]))
    return s


def attention_head(q, k, v) -> np.ndarray:
    """softmax(q k^T / sqrt(hd)) v for one head; q [nq][hd] float64, k/v [nk][hd] float32."""
    q = np.ascontiguousarray(np.asarray(q, dtype=np.float64))
    k = _f32(k)
    v = _f32(v)
    out = np.zeros_like(q)
    _load().ebrl_oracle_attention_head(q.ctypes.data_as(C.c_void_p), C.c_int(q.shape[0]), _fp(k),
                                       _fp(v), C.c_int(k.shape[0]), C.c_int(q.shape[1]),
                                       out.ctypes.data_as(C.c_void_p))
    return out


def velocity(cfg: OracleConfig, w: OracleWeights, kv, a, k: int) -> np.ndarray:
    """Network velocity of one environment at Euler step k.  kv: [kv_layers][2][P][d], or the
    hidden states [P][d_ctx] when ``cfg.d_ctx > 0``."""
    kv = _f32(kv)
    P = kv.shape[-2]
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64)).reshape(cfg.H, cfg.A)
    v = np.zeros_like(a)
    cw, keep = w._c()
    c = cfg._c()
    rc = _load().ebrl_oracle_velocity(C.byref(c), C.byref(cw), _fp(kv), C.c_int(P),
                                      a.ctypes.data_as(C.c_void_p), C.c_int(k),
                                      v.ctypes.data_as(C.c_void_p))
    if rc:
        raise RuntimeError("oracle velocity failed: %d" % rc)
    del keep
    return v


def actgen(cfg: OracleConfig, w: OracleWeights, prefix_kv: Sequence, noise,
           step_index: Optional[Sequence[int]] = None, n_steps: int = 0,
           n_threads: Optional[int] = None, pull: bool = False) -> np.ndarray:
    """Advance every environment of a group; returns float64 [n][H][A].

    prefix_kv[i]: array [kv_layers][2][P_i][d] (values already rounded to the stored dtype), or the
    hidden states [P_i][d_ctx] when ``cfg.d_ctx > 0``.
    noise: [n][H][A] float32, environment i's action state at step ``step_index[i]``.
    ``pull`` replaces the network by the linear field v = b_out - a (integrator pin).
    """
    noise = _f32(noise)
    n = noise.shape[0]
    kvs = [_f32(p) for p in prefix_kv]
    assert len(kvs) == n or pull
    plen = np.array([p.shape[-2] for p in kvs] if kvs else [0] * n, dtype=np.int32)
    if kvs:
        for p in kvs:
            if cfg.d_ctx > 0:
                assert p.ndim == 2 and p.shape[-1] == cfg.d_ctx     # hidden states [P][d_ctx]
            else:
                assert p.shape[-1] == cfg.d and p.shape[-3] == 2
        ptrs = (_FP * max(1, n))(*[_fp(p) for p in kvs])
        ptrs_arg = C.cast(ptrs, _FPP)
    else:
        ptrs_arg = C.cast(None, _FPP)
    sidx = None
    if step_index is not None:
        sidx = np.ascontiguousarray(np.asarray(step_index, dtype=np.int32))
        assert sidx.shape[0] == n
    out = np.zeros((n, cfg.H, cfg.A), dtype=np.float64)
    cw, keep = w._c()
    c = cfg._c()
    if n_threads is None:
        n_threads = os.cpu_count() or 1
    rc = _load().ebrl_oracle_actgen(
        C.byref(c), C.byref(cw), C.c_int(n), ptrs_arg, plen.ctypes.data_as(C.c_void_p),
        sidx.ctypes.data_as(C.c_void_p) if sidx is not None else None, C.c_int(n_steps),
        _fp(noise), out.ctypes.data_as(C.c_void_p), C.c_int(n_threads), C.c_int(1 if pull else 0))
    if rc:
        raise RuntimeError("oracle actgen failed: %d" % rc)
    del keep
    return out
