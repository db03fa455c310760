"""Event timeline of the persistent step kernel (a tuning aid, needs a tuning build).

    EBRL_NVCC_EXTRA=-DEBRL_FUSED_PROF python -m paper_2609_27547_b200.build --force
    python -m paper_2609_27547_b200.fused_timeline <config> <envs> [sm_quota]
    python -m paper_2609_27547_b200.build --force          # back to the normal library

In a tuning build the kernel logs {event, task, CTA, globaltimer} for every task of row block 0 in
the first Euler step; this script runs one batch of `envs` environments of a benchmark
configuration through the kernel and prints, per operation of the first layer, when the first
and the last CTA reached each event (microseconds from the first event):

    P dep       the producer thread saw the task's dependency satisfied
    M kb0       the first operand k-block of a projection tile landed
    M issued    the last tcgen05.mma of the tile was issued
    W dep       an epilogue warp saw the dependency announced
    W epi       the tile's epilogue finished          W sig   its completion counter was raised
    A start / A done / A sig   the same for an attention item
"""
from __future__ import annotations

import ctypes as C
import os
import sys

import numpy as np
import torch

from . import binding as B
from . import synth

NAMES = {1: "P dep", 3: "M kb0", 4: "M issued", 5: "W dep", 6: "W epi", 7: "W sig", 8: "A start", 9: "A done", 10: "A sig"}


def main(argv):
    cfgi, nb = int(argv[0]), int(argv[1])
    quota = int(argv[2]) if len(argv) > 2 else 0
    if not hasattr(B.lib(), "ebrl_actgen_debug_events"):
        raise SystemExit("this library was not built with -DEBRL_FUSED_PROF (see the module docstring)")
    os.environ["EBRL_TRACE"] = "1"
    w = synth.WORKLOADS[cfgi]
    wt = synth.make_weights(w, device="cuda")
    envs = [synth.make_env(w, e, device="cuda") for e in range(nb)]
    gen = B.ActGen(B.cfg_for(w, max_group_envs=nb, max_inflight_groups=1, flags=B.FLAG_FORCE_FUSED), wt)
    noise = torch.stack([e.noise for e in envs]).contiguous()
    out = torch.empty_like(noise)
    st = torch.cuda.Stream()

    def step():
        gen.submit(list(range(nb)), [e.kv for e in envs], noise, out, sm_quota=quota, stream=st)
        gen.sync()

    for _ in range(3):
        step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(st)
    step()
    e1.record(st)
    torch.cuda.synchronize()
    print("ms per batch of %d chunks: %.3f" % (nb, e0.elapsed_time(e1)))
    cap = 4000
    ev = (C.c_longlong * (2 * cap))()
    cnt = C.c_int32(0)
    B.lib().ebrl_actgen_debug_events(gen._h, ev, cap, C.byref(cnt))
    n = min(cnt.value, cap)
    e = np.frombuffer(ev, dtype=np.int64).reshape(cap, 2)[:n]
    rows = sorted((int(x[1]), int(x[0]) >> 48, int(x[0]) & 0xffffffff) for x in e)
    if not rows:
        raise SystemExit("no events were logged")
    t0 = rows[0][0]
    nt_d, nt_qkv, nt_md = w.d // 128, 3 * w.d // 128, w.mlp_mult * w.d // 128
    mt = (nb * w.H + 127) // 128
    nslab = max(1, w.n_heads // 8)
    base, ranges = mt, []
    for name, ntasks in (("QKV", mt * nt_qkv), ("self-attn", nb * nslab), ("W_o", mt * nt_d), ("W_qc", mt * nt_d),
                         ("cross-attn", nb * nslab), ("W_oc", mt * nt_d), ("W_1", mt * nt_md), ("W_2", mt * nt_d)):
        ranges.append((base, base + ntasks - 1, name))
        base += ntasks
    seen = {}
    for t, ty, task in rows:
        for lo, hi, name in ranges:
            if lo <= task <= hi:
                seen.setdefault((name, NAMES.get(ty, str(ty))), []).append((t - t0) / 1e3)
    for lo, hi, name in ranges:
        parts = ["%s %.1f..%.1f" % (k[1], min(v), max(v)) for k, v in seen.items() if k[0] == name]
        print("%-10s %s" % (name, "   ".join(parts)))
    gen.destroy()


if __name__ == "__main__":
    main(sys.argv[1:])
