"""Glue shared by the tests: synthetic inputs -> oracle arguments, and the error metric."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2609_27547_b200 import synth


def oracle_cfg(w: synth.Workload) -> oracle.OracleConfig:
    return oracle.OracleConfig(H=w.H, A=w.A, d=w.d, n_layers=w.L, n_heads=w.n_heads, K_steps=w.K,
                               mlp_mult=w.mlp_mult, d_ctx=w.d_ctx, kv_layers=w.L if w.d_ctx > 0 else 1)


def np32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy()


def oracle_weights(wt: dict) -> oracle.OracleWeights:
    return oracle.OracleWeights(
        w_in=np32(wt["w_in"]), w_out=np32(wt["w_out"]), b_out=np32(wt["b_out"]),
        g_final=np32(wt["g_final"]),
        layers=[{k: np32(v) for k, v in l.items()} for l in wt["layers"]])


def oracle_run(w: synth.Workload, wt: dict, envs, n_steps: int = 0, n_threads=None) -> np.ndarray:
    return oracle.actgen(oracle_cfg(w), oracle_weights(wt), [np32(e.kv) for e in envs],
                         np.stack([np32(e.noise) for e in envs]),
                         step_index=[e.step for e in envs], n_steps=n_steps, n_threads=n_threads)


def chunk_rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """Per environment max|got - ref| / max(1, max|ref|), maximised over environments."""
    got = np.asarray(got, dtype=np.float64).reshape(ref.shape[0], -1)
    ref = np.asarray(ref, dtype=np.float64).reshape(ref.shape[0], -1)
    if ref.shape[0] == 0:
        return 0.0
    num = np.abs(got - ref).max(axis=1)
    den = np.maximum(1.0, np.abs(ref).max(axis=1))
    return float((num / den).max())
