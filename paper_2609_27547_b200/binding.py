"""ctypes binding of libebrl_actgen (argument marshalling only; every step of the path runs in
the library's CUDA kernels).  Names follow ``include/ebrl_actgen.h``.

torch is used for device memory and streams only.  There is no fallback: if the library is
missing, or no CUDA device is usable, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

from . import build as _build

ABI_VERSION = 3
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NOMEM, ERR_CUDA, ERR_ENV_BUSY, ERR_QUOTA, ERR_TIMEOUT = range(8)
F32, BF16 = 0, 1
FLAG_TEST_PULL, FLAG_GREEN_CTX, FLAG_TIMING, FLAG_FORCE_SIMT, FLAG_NO_FUSED, FLAG_FORCE_FUSED = 1, 2, 4, 8, 16, 32
FLAG_TEST_DROP_GEMM_COPIES, FLAG_TEST_DROP_ATTN_COPIES, FLAG_DEBUG_CANARY = 64, 128, 256
KC_NAMES = ("embed", "gemm", "self_attn", "cross_attn", "head", "prefix", "fused")


class Cfg(C.Structure):
    _fields_ = [("abi_version", C.c_uint32), ("H", C.c_int32), ("A", C.c_int32), ("d", C.c_int32),
                ("n_layers", C.c_int32), ("n_heads", C.c_int32), ("mlp_mult", C.c_int32),
                ("K_steps", C.c_int32), ("max_prefix_len", C.c_int32), ("max_group_envs", C.c_int32),
                ("max_inflight_groups", C.c_int32), ("param_dtype", C.c_int32), ("kv_dtype", C.c_int32),
                ("kv_layers", C.c_int32), ("rms_eps", C.c_float), ("temb_scale", C.c_float),
                ("temb_max_period", C.c_float), ("flags", C.c_uint32), ("device", C.c_int32),
                ("wait_limit_ns", C.c_uint64), ("d_ctx", C.c_int32), ("reserved_", C.c_int32)]


class LayerWeights(C.Structure):
    _fields_ = [("g1", C.c_void_p), ("g2", C.c_void_p), ("g3", C.c_void_p), ("w_qkv", C.c_void_p),
                ("w_o", C.c_void_p), ("w_qc", C.c_void_p), ("w_oc", C.c_void_p), ("w_1", C.c_void_p),
                ("w_2", C.c_void_p), ("w_kc", C.c_void_p), ("w_vc", C.c_void_p)]


class Weights(C.Structure):
    _fields_ = [("w_in", C.c_void_p), ("w_out", C.c_void_p), ("b_out", C.c_void_p),
                ("g_final", C.c_void_p), ("layers", C.POINTER(LayerWeights))]


class SubmitExt(C.Structure):
    _fields_ = [("prefix_len", C.POINTER(C.c_int32)), ("step_index", C.POINTER(C.c_int32)),
                ("n_steps", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("groups", C.c_uint64), ("envs", C.c_uint64), ("env_steps", C.c_uint64),
                ("kernel_launches", C.c_uint64), ("granted_sms", C.c_int32),
                ("green_ctx_active", C.c_int32), ("green_ctx_sms", C.c_int32), ("reserved_", C.c_int32),
                ("class_ms", C.c_double * len(KC_NAMES)),
                ("class_launches", C.c_uint64 * len(KC_NAMES)), ("class_flops", C.c_double * len(KC_NAMES)),
                ("class_bytes", C.c_double * len(KC_NAMES)), ("weights_version", C.c_uint64)]


class QueueCfg(C.Structure):
    _fields_ = [("capacity", C.c_int32), ("max_group", C.c_int32), ("sm_quota", C.c_int32), ("step_mode", C.c_int32),
                ("linger_us", C.c_uint32), ("reserved_", C.c_uint32)]


QUEUE_SUBMIT_FN = C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_void_p), C.POINTER(C.c_int32),
                              C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_int32), C.c_int32, C.c_int32, C.c_void_p)
QUEUE_SYNC_FN = C.CFUNCTYPE(C.c_int32, C.c_void_p)


class QueueBackend(C.Structure):
    _fields_ = [("ctx", C.c_void_p), ("K_steps", C.c_int32), ("submit", QUEUE_SUBMIT_FN), ("sync", QUEUE_SYNC_FN)]


class QueueStats(C.Structure):
    _fields_ = [("pushed", C.c_uint64), ("completed", C.c_uint64), ("failed", C.c_uint64), ("groups", C.c_uint64),
                ("group_envs", C.c_uint64), ("blocked_pushes", C.c_uint64), ("max_waiting", C.c_int32),
                ("waiting", C.c_int32), ("in_service", C.c_int32), ("reserved_", C.c_int32)]


ERR_QUEUE_FULL, ERR_CLOSED = 8, 9


class EbrlError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__("ebrl_actgen status %d: %s" % (status, text))
        self.status = status


_lib = None


def lib():
    """Loads the in-tree shared library (building it if nvcc is present and it is stale)."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if _build.stale():
            path = _build.build()
        if not os.path.exists(path):
            raise RuntimeError("libebrl_actgen.so is missing; run python -m paper_2609_27547_b200.build")
        L = C.CDLL(path)
        L.ebrl_actgen_last_error.restype = C.c_char_p
        L.ebrl_actgen_last_error.argtypes = [C.c_void_p]
        L.ebrl_actgen_abi_version.restype = C.c_uint32
        L.ebrl_actgen_struct_size.restype = C.c_uint64
        L.ebrl_actgen_struct_size.argtypes = [C.c_int32]
        L.ebrl_actgen_create.argtypes = [C.POINTER(Cfg), C.POINTER(Weights), C.POINTER(C.c_void_p)]
        sub = [C.c_void_p, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_void_p), C.c_void_p,
               C.c_void_p, C.c_int32, C.c_void_p, C.POINTER(SubmitExt)]
        L.ebrl_actgen_submit.argtypes = sub
        L.ebrl_actgen_submit_host.argtypes = sub
        L.ebrl_actgen_sync.argtypes = [C.c_void_p]
        L.ebrl_actgen_flush.argtypes = [C.c_void_p]
        L.ebrl_actgen_update_weights.argtypes = [C.c_void_p, C.POINTER(Weights), C.c_void_p, C.POINTER(C.c_uint64)]
        L.ebrl_actgen_weights_version.argtypes = [C.c_void_p]
        L.ebrl_actgen_weights_version.restype = C.c_uint64
        L.ebrl_actgen_destroy.argtypes = [C.c_void_p]
        L.ebrl_actgen_get_stats.argtypes = [C.c_void_p, C.POINTER(Stats)]
        L.ebrl_actgen_reset_stats.argtypes = [C.c_void_p]
        L.ebrl_actgen_set_timing.argtypes = [C.c_void_p, C.c_int32]
        L.ebrl_actgen_partition_info.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_void_p)]
        L.ebrl_actgen_check_cfg.argtypes = [C.POINTER(Cfg)]
        L.ebrl_actgen_check_submit.argtypes = [C.POINTER(Cfg), C.c_int32, C.c_int32, C.POINTER(C.c_int64),
                                               C.POINTER(C.c_void_p), C.c_void_p, C.c_void_p, C.c_int32,
                                               C.POINTER(SubmitExt)]
        L.ebrl_actgen_plan_group.argtypes = [C.POINTER(Cfg), C.c_int32, C.POINTER(SubmitExt),
                                             C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.ebrl_actgen_plan_group.restype = C.c_int32
        L.ebrl_actgen_l0_step_noalloc.argtypes = [C.c_void_p] * 7 + [C.c_int32] * 4 + [C.c_float, C.c_int32, C.c_void_p]
        L.ebrl_actgen_wait_probe.argtypes = [C.c_int32, C.c_uint64, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_uint64)]
        L.ebrl_sim_corunner_launch.argtypes = [C.c_void_p, C.c_uint64, C.c_int32, C.c_int32, C.c_void_p]
        L.ebrl_actgen_k_steps.argtypes = [C.c_void_p]
        L.ebrl_actgen_submit_scattered.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_void_p),
                                                   C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.c_int32, C.c_void_p,
                                                   C.POINTER(SubmitExt)]
        L.ebrl_queue_create.argtypes = [C.c_void_p, C.POINTER(QueueCfg), C.c_void_p, C.POINTER(C.c_void_p)]
        L.ebrl_queue_create_backend.argtypes = [C.POINTER(QueueBackend), C.POINTER(QueueCfg), C.c_void_p, C.POINTER(C.c_void_p)]
        push = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_uint64)]
        L.ebrl_queue_push.argtypes = push
        L.ebrl_queue_try_push.argtypes = push
        L.ebrl_queue_wait.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32]
        L.ebrl_queue_get_stats.argtypes = [C.c_void_p, C.POINTER(QueueStats)]
        L.ebrl_queue_destroy.argtypes = [C.c_void_p]
        _lib = L
    return _lib


def make_cfg(*, H, A, d, n_layers, n_heads, K_steps, max_prefix_len, max_group_envs,
             max_inflight_groups=1, dtype=F32, mlp_mult=4, kv_layers=1, rms_eps=1e-6,
             temb_scale=1000.0, temb_max_period=10000.0, flags=0, device=0, d_ctx=0) -> Cfg:
    """``d_ctx > 0``: prefixes are hidden states [P][d_ctx] projected per layer (then kv_layers = n_layers)."""
    return Cfg(ABI_VERSION, H, A, d, n_layers, n_heads, mlp_mult, K_steps, max_prefix_len,
               max_group_envs, max_inflight_groups, dtype, dtype, n_layers if d_ctx > 0 else kv_layers, rms_eps,
               temb_scale, temb_max_period, flags, device, 0, d_ctx, 0)


def _ext(prefix_len, step_index, n_steps):
    keep = []
    e = SubmitExt()
    if prefix_len is not None:
        a = (C.c_int32 * len(prefix_len))(*[int(v) for v in prefix_len]); keep.append(a)
        e.prefix_len = C.cast(a, C.POINTER(C.c_int32))
    if step_index is not None:
        a = (C.c_int32 * len(step_index))(*[int(v) for v in step_index]); keep.append(a)
        e.step_index = C.cast(a, C.POINTER(C.c_int32))
    e.n_steps = int(n_steps)
    return e, keep


def plan_group(cfg: Cfg, n: int, step_index=None, n_steps: int = 0):
    """Host-only: the batcher's packing of a group -> (S, order, nsteps, n_active)."""
    e, keep = _ext(None, step_index, n_steps)
    order = (C.c_int32 * max(1, n))(); ns = (C.c_int32 * max(1, n))(); na = (C.c_int32 * cfg.K_steps)()
    S = lib().ebrl_actgen_plan_group(C.byref(cfg), n, C.byref(e), order, ns, na)
    return S, list(order)[:n], list(ns)[:n], list(na)


class ActGen:
    """One handle of the library: ``ebrl_actgen_create`` ... ``ebrl_actgen_destroy``."""

    def __init__(self, cfg: Cfg, weights: dict):
        """``weights``: dict as produced by ``synth.make_weights`` (torch tensors on any device,
        matrices in the configured dtype, gains and b_out fp32)."""
        self._L = lib()
        self.cfg = cfg
        w, keep = self._marshal(weights)
        self._h = C.c_void_p()
        st = self._L.ebrl_actgen_create(C.byref(cfg), C.byref(w), C.byref(self._h))
        if st != OK:
            raise EbrlError(st, (self._L.ebrl_actgen_last_error(None) or b"").decode())
        del keep

    def _marshal(self, weights: dict):
        cfg = self.cfg
        want = torch.bfloat16 if cfg.param_dtype == BF16 else torch.float32
        keep = []

        def ptr(t, dt):
            if t.dtype != dt:
                raise TypeError("weight tensor has dtype %s, expected %s" % (t.dtype, dt))
            t = t.contiguous(); keep.append(t)
            return t.data_ptr()

        lw = (LayerWeights * max(1, cfg.n_layers))()
        for i, l in enumerate(weights["layers"]):
            lw[i] = LayerWeights(ptr(l["g1"], torch.float32), ptr(l["g2"], torch.float32), ptr(l["g3"], torch.float32),
                                 ptr(l["w_qkv"], want), ptr(l["w_o"], want), ptr(l["w_qc"], want),
                                 ptr(l["w_oc"], want), ptr(l["w_1"], want), ptr(l["w_2"], want),
                                 ptr(l["w_kc"], want) if cfg.d_ctx > 0 else None,
                                 ptr(l["w_vc"], want) if cfg.d_ctx > 0 else None)
        keep.append(lw)
        w = Weights(ptr(weights["w_in"], want), ptr(weights["w_out"], want), ptr(weights["b_out"], torch.float32),
                    ptr(weights["g_final"], torch.float32), C.cast(lw, C.POINTER(LayerWeights)))
        return w, keep

    def update_weights(self, weights: dict, stream: Optional[torch.cuda.Stream] = None) -> int:
        """``ebrl_actgen_update_weights``: publish a new policy version without blocking; returns its
        version number.  The tensors are kept alive by this object until the next update."""
        w, keep = self._marshal(weights)
        s = stream if stream is not None else torch.cuda.current_stream(self.cfg.device)
        ver = C.c_uint64(0)
        self._check(self._L.ebrl_actgen_update_weights(self._h, C.byref(w), s.cuda_stream, C.byref(ver)))
        self._published = keep
        return int(ver.value)

    def weights_version(self) -> int:
        return int(self._L.ebrl_actgen_weights_version(self._h))

    def _check(self, st):
        if st != OK:
            raise EbrlError(st, (self._L.ebrl_actgen_last_error(self._h) or b"").decode())

    def _submit(self, fn, env_ids, kv_ptrs, noise_ptr, out_ptr, sm_quota, stream, prefix_len, step_index, n_steps):
        n = len(env_ids)
        ids = (C.c_int64 * max(1, n))(*[int(e) for e in env_ids])
        kvp = (C.c_void_p * max(1, n))(*kv_ptrs) if kv_ptrs is not None else None
        e, keep = _ext(prefix_len, step_index, n_steps)
        self._check(fn(self._h, n, ids, kvp, noise_ptr, out_ptr, int(sm_quota), stream, C.byref(e)))

    def submit(self, env_ids: Sequence[int], prefix_kv: Optional[Sequence[torch.Tensor]], noise: torch.Tensor,
               out: torch.Tensor, sm_quota: int = 0, stream: Optional[torch.cuda.Stream] = None,
               prefix_len: Optional[Sequence[int]] = None, step_index: Optional[Sequence[int]] = None,
               n_steps: int = 0):
        """``ebrl_actgen_submit``: device tensors; prefix_kv[i] is [kv_layers][2][P_i][d], or the
        hidden states [P_i][d_ctx] when the handle was created with ``d_ctx > 0``."""
        if noise.device.type != "cuda" or out.device.type != "cuda":
            raise ValueError("noise and out must be CUDA tensors")
        if noise.dtype != torch.float32 or out.dtype != torch.float32 or not noise.is_contiguous() or not out.is_contiguous():
            raise ValueError("noise and out must be contiguous fp32")
        kv_ptrs = None
        if prefix_kv is not None:
            for t in prefix_kv:
                if t.device.type != "cuda" or not t.is_contiguous():
                    raise ValueError("prefix planes must be contiguous CUDA tensors")
            kv_ptrs = [t.data_ptr() for t in prefix_kv]
            if prefix_len is None:
                prefix_len = [t.shape[-2] for t in prefix_kv]
        s = stream if stream is not None else torch.cuda.current_stream(noise.device)
        self._submit(self._L.ebrl_actgen_submit, env_ids, kv_ptrs, noise.data_ptr(), out.data_ptr(), sm_quota,
                     s.cuda_stream, prefix_len, step_index, n_steps)

    def submit_host(self, env_ids, prefix_kv: Optional[Sequence[torch.Tensor]], noise: torch.Tensor, out: torch.Tensor,
                    sm_quota: int = 0, stream: Optional[torch.cuda.Stream] = None, prefix_len=None,
                    step_index=None, n_steps: int = 0):
        """``ebrl_actgen_submit_host``: host tensors (pinned for asynchronous copies)."""
        if noise.device.type != "cpu" or out.device.type != "cpu":
            raise ValueError("noise and out must be host tensors")
        kv_ptrs = None
        if prefix_kv is not None:
            kv_ptrs = [t.data_ptr() for t in prefix_kv]
            if prefix_len is None:
                prefix_len = [t.shape[-2] for t in prefix_kv]
        s = stream if stream is not None else torch.cuda.current_stream(self.cfg.device)
        self._submit(self._L.ebrl_actgen_submit_host, env_ids, kv_ptrs, noise.data_ptr(), out.data_ptr(), sm_quota,
                     s.cuda_stream, prefix_len, step_index, n_steps)

    def flush(self):
        self._check(self._L.ebrl_actgen_flush(self._h))

    def sync(self):
        self._check(self._L.ebrl_actgen_sync(self._h))

    def stats(self) -> dict:
        s = Stats()
        self._check(self._L.ebrl_actgen_get_stats(self._h, C.byref(s)))
        out = {k: getattr(s, k) for k in ("groups", "envs", "env_steps", "kernel_launches", "granted_sms", "green_ctx_active", "green_ctx_sms", "weights_version")}
        out["classes"] = {n: {"ms": s.class_ms[i], "launches": s.class_launches[i], "flops": s.class_flops[i],
                              "bytes": s.class_bytes[i]} for i, n in enumerate(KC_NAMES)}
        return out

    def partition_info(self, sm_quota: int):
        """``ebrl_actgen_partition_info``: (SMs of the quota's partition, SMs of the complementary one, its stream handle or None)."""
        g, r, st = C.c_int32(0), C.c_int32(0), C.c_void_p()
        self._check(self._L.ebrl_actgen_partition_info(self._h, int(sm_quota), C.byref(g), C.byref(r), C.byref(st)))
        return g.value, r.value, st.value

    def rest_stream(self, sm_quota: int) -> Optional[torch.cuda.Stream]:
        """The complementary partition's stream as a torch stream (None when there is no partition)."""
        _, rest, st = self.partition_info(sm_quota)
        if not st or rest < 1:
            return None
        return torch.cuda.ExternalStream(st, device=torch.device("cuda", self.cfg.device))

    def reset_stats(self):
        self._check(self._L.ebrl_actgen_reset_stats(self._h))

    def set_timing(self, on: bool):
        self._check(self._L.ebrl_actgen_set_timing(self._h, 1 if on else 0))

    def destroy(self):
        if self._h:
            h, self._h = self._h, C.c_void_p()
            st = self._L.ebrl_actgen_destroy(h)
            if st != OK:
                raise EbrlError(st, "destroy failed")

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class Queue:
    """``ebrl_queue_*``: the bounded request queue in front of a handle (or of a test backend)."""

    def __init__(self, gen: Optional["ActGen"], *, capacity: int, max_group: int, sm_quota: int = 0, step_mode: bool = False,
                 linger_us: int = 0, stream: Optional[torch.cuda.Stream] = None, backend: Optional[QueueBackend] = None):
        self._L = lib()
        self._gen = gen            # keeps the handle alive
        self._backend = backend    # keeps the callbacks alive
        cfg = QueueCfg(capacity, max_group, sm_quota, 1 if step_mode else 0, linger_us, 0)
        self._q = C.c_void_p()
        sp = stream.cuda_stream if stream is not None else None
        if backend is not None:
            st = self._L.ebrl_queue_create_backend(C.byref(backend), C.byref(cfg), sp, C.byref(self._q))
        else:
            st = self._L.ebrl_queue_create(gen._h, C.byref(cfg), sp, C.byref(self._q))
        if st != OK:
            raise EbrlError(st, "queue create failed")

    def _push(self, fn, env_id, prefix, prefix_len, state, out, step_index):
        t = C.c_uint64(0)
        ptr = lambda x: x.data_ptr() if torch.is_tensor(x) else int(x)
        st = fn(self._q, int(env_id), ptr(prefix), int(prefix_len), ptr(state), ptr(out), int(step_index), C.byref(t))
        return st, int(t.value)

    def push(self, env_id, prefix, prefix_len, state, out, step_index=0) -> int:
        """Blocks while the queue is full; returns the ticket.  Tensors (device) or raw addresses."""
        st, t = self._push(self._L.ebrl_queue_push, env_id, prefix, prefix_len, state, out, step_index)
        if st != OK:
            raise EbrlError(st, "queue push failed")
        return t

    def try_push(self, env_id, prefix, prefix_len, state, out, step_index=0):
        """(status, ticket): status ERR_QUEUE_FULL instead of blocking."""
        return self._push(self._L.ebrl_queue_try_push, env_id, prefix, prefix_len, state, out, step_index)

    def wait(self, ticket: int, timeout_ms: int = 0) -> int:
        return int(self._L.ebrl_queue_wait(self._q, int(ticket), int(timeout_ms)))

    def stats(self) -> dict:
        s = QueueStats()
        self._L.ebrl_queue_get_stats(self._q, C.byref(s))
        return {k: getattr(s, k) for k, _ in QueueStats._fields_ if k != "reserved_"}

    def destroy(self):
        if self._q:
            q, self._q = self._q, C.c_void_p()
            self._L.ebrl_queue_destroy(q)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def l0_step_noalloc(a_in: torch.Tensor, a_out: torch.Tensor, w_in: torch.Tensor, w_out: torch.Tensor,
                    b_out: torch.Tensor, g_final: torch.Tensor, temb_row: torch.Tensor, K_steps: int,
                    rms_eps: float = 1e-6, sm_quota: int = 0, stream: Optional[torch.cuda.Stream] = None) -> int:
    """``ebrl_actgen_l0_step_noalloc``: one Euler step of a layer-less fp32 head for callers that
    cannot allocate device memory; all tensors are the caller's CUDA fp32 tensors.  Returns the
    status code (0 = OK) instead of raising so that a caller can test the size limits."""
    ts = (a_in, a_out, w_in, w_out, b_out, g_final, temb_row)
    for t in ts:
        if t.device.type != "cuda" or t.dtype != torch.float32 or not t.is_contiguous():
            raise ValueError("contiguous CUDA fp32 tensors required")
    n_rows, A = a_in.shape[-2] * (a_in.shape[0] if a_in.dim() == 3 else 1), a_in.shape[-1]
    d = w_in.shape[0]
    s = stream if stream is not None else torch.cuda.current_stream(a_in.device)
    with torch.cuda.device(a_in.device):
        return int(lib().ebrl_actgen_l0_step_noalloc(*[t.data_ptr() for t in ts], n_rows, A, d, K_steps, rms_eps,
                                                     sm_quota, s.cuda_stream))


def wait_probe(limit_ns: int, signal_it: bool, device: int = 0):
    """``ebrl_actgen_wait_probe``: (status of the call, status the kernel recorded, ns waited on the device)."""
    st, waited = C.c_int32(-1), C.c_uint64(0)
    rc = lib().ebrl_actgen_wait_probe(device, int(limit_ns), 1 if signal_it else 0, C.byref(st), C.byref(waited))
    return rc, st.value, waited.value


def sim_corunner_launch(buf: torch.Tensor, n_steps: int, n_ctas: int, stream: torch.cuda.Stream):
    st = lib().ebrl_sim_corunner_launch(buf.data_ptr(), buf.numel(), n_steps, n_ctas, stream.cuda_stream)
    if st != OK:
        raise EbrlError(st, "corunner launch failed")


def cfg_for(w, *, max_group_envs: Optional[int] = None, max_inflight_groups: int = 1, flags: int = 0, device: int = 0) -> Cfg:
    """The library configuration of a ``synth.Workload``."""
    return make_cfg(H=w.H, A=w.A, d=w.d, n_layers=w.L, n_heads=w.n_heads, K_steps=w.K, max_prefix_len=w.P[1],
                    max_group_envs=max_group_envs or (w.group[1] if w.group else w.B),
                    max_inflight_groups=max_inflight_groups, dtype=BF16 if w.dtype == "bf16" else F32,
                    mlp_mult=w.mlp_mult, flags=flags, device=device, d_ctx=getattr(w, "d_ctx", 0))
