"""ctypes binding of the elastic allocator calls (``include/ebrl_alloc.h``): marshalling only."""
from __future__ import annotations

import ctypes as C
from typing import Sequence

from .binding import lib


class Profile(C.Structure):
    _fields_ = [("n_quota", C.c_int32), ("n_batch", C.c_int32), ("quota_pct", C.POINTER(C.c_int32)),
                ("batch", C.POINTER(C.c_int32)), ("rate", C.POINTER(C.c_double)), ("mem_gb", C.POINTER(C.c_double))]


class AllocIn(C.Structure):
    _fields_ = [("cores", C.c_int32), ("cores_per_env", C.c_int32), ("n_sim_quota", C.c_int32),
                ("sim_quota_pct", C.POINTER(C.c_int32)), ("sim_rate", C.POINTER(C.c_double)),
                ("knee_tolerance", C.c_double), ("gen", Profile), ("train", Profile), ("s_g_min", C.c_int32),
                ("s_t_min", C.c_int32), ("mem_gpu_gb", C.c_double)]


class AllocOut(C.Structure):
    _fields_ = [("env_concurrency", C.c_int32), ("s_sim", C.c_int32), ("s_g", C.c_int32), ("s_t", C.c_int32),
                ("B_g", C.c_int32), ("B_t", C.c_int32), ("T_s", C.c_double), ("T_g", C.c_double), ("T_t", C.c_double),
                ("T_r", C.c_double), ("theta", C.c_double), ("iterations", C.c_int32)]


def _ints(v):
    return (C.c_int32 * len(v))(*[int(x) for x in v])


def _dbls(v):
    return (C.c_double * len(v))(*[float(x) for x in v])


def make_profile(quota_pct: Sequence[int], batch: Sequence[int], rate, mem_gb):
    keep = [_ints(quota_pct), _ints(batch), _dbls([x for row in rate for x in row]), _dbls(mem_gb)]
    p = Profile(len(quota_pct), len(batch), C.cast(keep[0], C.POINTER(C.c_int32)), C.cast(keep[1], C.POINTER(C.c_int32)),
                C.cast(keep[2], C.POINTER(C.c_double)), C.cast(keep[3], C.POINTER(C.c_double)))
    return p, keep


def profile_rate(p: Profile, quota_pct: int, batch_index: int) -> float:
    L = lib()
    L.ebrl_profile_rate.restype = C.c_double
    L.ebrl_profile_rate.argtypes = [C.POINTER(Profile), C.c_int32, C.c_int32]
    return float(L.ebrl_profile_rate(C.byref(p), quota_pct, batch_index))


def elastic_allocation(N, c_env, sim_quota_pct, sim_rate, gen, train, s_g_min, s_t_min, M_gpu, knee_tolerance=0.05):
    """``ebrl_alloc_elastic``; gen/train are (quota_pct, batch, rate[quota][batch], mem_gb) tuples.
    Returns a dict, or None when the input is rejected."""
    L = lib()
    L.ebrl_alloc_elastic.argtypes = [C.POINTER(AllocIn), C.POINTER(AllocOut)]
    pg, k1 = make_profile(*gen)
    pt, k2 = make_profile(*train)
    sq, sr = _ints(sim_quota_pct), _dbls(sim_rate)
    a = AllocIn(N, c_env, len(sim_quota_pct), C.cast(sq, C.POINTER(C.c_int32)), C.cast(sr, C.POINTER(C.c_double)),
                knee_tolerance, pg, pt, s_g_min, s_t_min, M_gpu)
    o = AllocOut()
    if L.ebrl_alloc_elastic(C.byref(a), C.byref(o)) != 0:
        return None
    return dict(E=o.env_concurrency, s_sim=o.s_sim, s_g=o.s_g, s_t=o.s_t, B_g=o.B_g, B_t=o.B_t, T_s=o.T_s, T_g=o.T_g,
                T_t=o.T_t, T_r=o.T_r, theta=o.theta, iterations=o.iterations)


class Rebalance:
    def __init__(self, window=0, streak=0, threshold=0.0):
        L = lib()
        L.ebrl_rebalance_create.restype = C.c_void_p
        L.ebrl_rebalance_create.argtypes = [C.c_int32, C.c_int32, C.c_double]
        L.ebrl_rebalance_push.argtypes = [C.c_void_p, C.c_double, C.c_double]
        L.ebrl_rebalance_get.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int32)]
        L.ebrl_rebalance_destroy.argtypes = [C.c_void_p]
        self._L, self._h = L, L.ebrl_rebalance_create(window, streak, threshold)

    def push(self, rollout_rate: float, train_rate: float) -> int:
        return int(self._L.ebrl_rebalance_push(self._h, rollout_rate, train_rate))

    def averages(self):
        a, b, s = C.c_double(), C.c_double(), C.c_int32()
        self._L.ebrl_rebalance_get(self._h, C.byref(a), C.byref(b), C.byref(s))
        return a.value, b.value, s.value

    def __del__(self):
        if getattr(self, "_h", None):
            self._L.ebrl_rebalance_destroy(self._h)
            self._h = None
