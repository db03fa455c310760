#!/usr/bin/env python
"""Bench harness of the action-generation library (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--quota Q] [--impl ours|reference]

A "step" is one pass of the whole hot path over one batch of synthetic input: every environment
of the workload, submitted in its seeded arrival groups at the workload's SM quota, taken from
its noise to its final action chunk, then a sync.  The metric is environment action-chunks per
second (a chunk = one environment's K Euler steps).

* ``value``: inputs resident in HBM before the timed region; device time by CUDA events on the
  launching stream; max over ranks.
* ``e2e``: the same through ``ebrl_actgen_submit_host`` with pinned HOST buffers (host->device
  copies of planes and noise and the device->host copy of the chunks inside the timed region).
* ``roofline``: the dominant kernel class (the GEMMs) timed with CUDA events around each launch
  in a second pass of the same steps; peak from MEASURED_PEAKS.json scaled by quota/SMs.
* ``cpu_baseline``: the fp64 oracle as it stands on this machine's host cores, on a bounded sample.
* ``--impl reference`` times that oracle alone (there is no other reference implementation).

Under torchrun each rank runs the same workload shape on its own shard of environment ids
(environments are independent: no data-path collective); ``value`` sums over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "env_action_chunks_per_sec"
UNIT = "chunks/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
N_SMS = 148
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12   # 148 SMs x 128 FFMA lanes x 2 flop x 1965 MHz


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["source"] = "fallback"
    return d


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=int(os.environ.get("EBRL_BENCH_CONFIG", "4")))
    ap.add_argument("--quota", type=int, default=-1, help="SM quota; -1 = the workload's own")
    ap.add_argument("--envs", type=int, default=0, help="override the number of environments")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--corunner", action="store_true", help="run the streaming co-runner on the other SMs")
    ap.add_argument("--simt", action="store_true", help="force the plain-ALU kernels")
    ap.add_argument("--green-ctx", action="store_true", help="run inside an SM partition (green context) of the quota")
    ap.add_argument("--pgen-sweep", action="store_true",
                    help="emit the generation profile P_gen(s_g, B_g): chunks/s on a grid of SM quotas and group sizes")
    ap.add_argument("--rollout-sim", action="store_true",
                    help="event-driven rollout with a synthetic simulator-latency model: chunk latency avg/P50/P99 under "
                         "group-level batching and under step-level continuous batching")
    ap.add_argument("--min-warmup", type=int, default=3, help="lower bound on warm-up steps (profiling captures use 1)")
    ap.add_argument("--d-ctx", type=int, default=0, help="variant: prefixes are hidden states [P][d_ctx], projected to K/V per layer")
    ap.add_argument("--inflight", type=int, default=16, help="groups queued before a batch is launched")
    return ap.parse_args()


def workload_flops(w, envs) -> float:
    """Algorithmic 2mnk FLOPs of one step (every environment from its step index to K)."""
    proj = 4.0 * w.L * w.d * w.d_ctx   # hidden-state prefixes: K and V projections of one prefix row, once per chunk
    return sum(w.flops_per_env_step(e.P) * (w.K - e.step) + proj * e.P for e in envs)


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------

def oracle_sample_rate(w, seed, cores, budget_s=20.0):
    """Times the oracle on a bounded sample of the workload and returns (chunks/s, description).

    Sample: `cores` environments (one per thread).  When a whole chunk would take too long the
    sample runs a single Euler step of each environment and the rate is scaled by the steps a
    chunk has; the description says so."""
    import numpy as np
    import torch
    import oracle
    from paper_2609_27547_b200 import synth

    def np32(t):
        return t.detach().to("cpu", torch.float32).numpy()

    wt = synth.make_weights(w, seed)
    n = max(1, min(cores, w.B))
    envs = [synth.make_env(w, e, seed) for e in range(n)]
    oc = oracle.OracleConfig(H=w.H, A=w.A, d=w.d, n_layers=w.L, n_heads=w.n_heads, K_steps=w.K, mlp_mult=w.mlp_mult)
    ow = oracle.OracleWeights(w_in=np32(wt["w_in"]), w_out=np32(wt["w_out"]), b_out=np32(wt["b_out"]),
                              g_final=np32(wt["g_final"]),
                              layers=[{k: np32(v) for k, v in l.items()} for l in wt["layers"]])
    kvs = [np32(e.kv) for e in envs]
    noise = np.stack([np32(e.noise) for e in envs])
    est_chunk_s = w.flops_per_env_step(sum(e.P for e in envs) / n) * w.K / 2.0e9   # ~2 GFLOP/s/core
    one_step = est_chunk_s > budget_s
    t0 = time.perf_counter()
    oracle.actgen(oc, ow, kvs, noise, step_index=[0] * n, n_steps=1 if one_step else 0, n_threads=cores)
    dt = time.perf_counter() - t0
    if one_step:
        rate = n / (dt * w.K)
        desc = "%d envs (ids 0..%d) x 1 Euler step of %d, rate scaled by 1/%d" % (n, n - 1, w.K, w.K)
    else:
        rate = n / dt
        desc = "%d envs (ids 0..%d), whole chunks" % (n, n - 1)
    return rate, desc, dt


def run_reference(args):
    from paper_2609_27547_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.WORKLOADS[args.config]
    if args.envs:
        w = synth.scaled(w, B=args.envs)
    seed = args.seed or synth.DEFAULT_SEED
    cores = os.cpu_count() or 1
    rates, times, desc = [], [], ""
    steps = max(1, min(args.steps, 3))
    for i in range(min(args.warmup, 1) + steps):
        r, desc, dt = oracle_sample_rate(w, seed, cores, budget_s=10.0)
        if i >= min(args.warmup, 1):
            rates.append(r)
            times.append(dt)
    value = len(rates) / sum(1.0 / r for r in rates)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * sum(times) / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "configs[%d] %s" % (args.config, w.name), "note": "fp64 CPU oracle on host cores; each step is a bounded sample"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        self.idx = device_index
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                                          "-i", str(device_index), "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons, power = [], [], set(), []
        for ln in out.splitlines():
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "power_w_max": max(power), "samples": len(sm)}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2609_27547_b200 import binding as B
    from paper_2609_27547_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = synth.WORKLOADS[args.config]
    if args.envs:
        w = synth.scaled(w, B=args.envs)
    if args.d_ctx:
        w = synth.scaled(w, d_ctx=args.d_ctx, name=w.name + "_hidden%d" % args.d_ctx)
    seed = args.seed or synth.DEFAULT_SEED
    quota = w.quota if args.quota < 0 else args.quota
    q_eff = quota if quota > 0 else N_SMS
    peaks = load_peaks()

    # this rank's shard: the same workload shape on its own environment ids (weak scaling)
    ids = [rank * w.B + e for e in range(w.B)]
    wt = synth.make_weights(w, seed, device=dev)
    envs = {e: synth.make_env(w, e, seed, device=dev) for e in ids}
    groups = synth.arrival_groups(w, seed + rank, env_ids=ids)
    order = [e for g in groups for e in g]
    pos = {e: i for i, e in enumerate(order)}
    noise = torch.stack([envs[e].noise for e in order]).contiguous()
    out = torch.empty_like(noise)
    kv_bytes = sum(envs[e].kv.numel() * envs[e].kv.element_size() for e in ids)
    inflight = args.inflight
    flags = (B.FLAG_FORCE_SIMT if args.simt else 0) | (B.FLAG_GREEN_CTX if args.green_ctx else 0)
    cfg = B.cfg_for(w, max_group_envs=max(len(g) for g in groups), max_inflight_groups=inflight, flags=flags, device=local)
    gen = B.ActGen(cfg, wt)
    stream = torch.cuda.Stream(dev)

    co_stream, co_buf = None, None
    if args.corunner and q_eff < N_SMS:
        co_stream = torch.cuda.Stream(dev)
        co_buf = torch.zeros(1 << 29, dtype=torch.float32, device=dev)   # 2 GiB

    def step():
        for g in groups:
            lo = pos[g[0]]
            gen.submit(g, [envs[e].kv for e in g], noise[lo:lo + len(g)], out[lo:lo + len(g)], sm_quota=quota,
                       stream=stream, step_index=[envs[e].step for e in g])
        gen.sync()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    n_warm = max(args.min_warmup, args.warmup)
    for _ in range(n_warm):
        step()
    gen.reset_stats()
    barrier()
    sampler = ClockSampler(local)
    if co_stream is not None:
        B.sim_corunner_launch(co_buf, 8 * args.steps, N_SMS - q_eff, co_stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    st0 = gen.stats()
    launches = st0["kernel_launches"]
    if world > 1:
        t = torch.tensor([ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    ms_step = ms / args.steps
    value = world * w.B / (ms_step * 1e-3)

    # ---- roofline of the dominant kernel class: a second pass with events around every launch
    gen.reset_stats()
    gen.set_timing(True)
    for _ in range(args.steps):
        step()
    st = gen.stats()
    gen.set_timing(False)
    cls = st["classes"]
    total_ms = sum(c["ms"] for c in cls.values()) or 1.0
    gemm = cls["gemm"]
    bf16 = w.dtype == "bf16"
    if bf16:
        peak = peaks["bf16_tflops"] * q_eff / N_SMS
        peak_note = "%s bf16 burst %.1f TFLOP/s x quota %d/%d" % (peaks["source"], peaks["bf16_tflops"], q_eff, N_SMS)
        bound = "tensor"
    else:
        peak = FP32_ALU_TFLOPS * q_eff / N_SMS
        peak_note = "fp32 FFMA 148 SMs x 128 lanes x 2 x 1.965 GHz = %.1f TFLOP/s x quota %d/%d" % (FP32_ALU_TFLOPS, q_eff, N_SMS)
        bound = "alu"
    achieved = gemm["flops"] / (gemm["ms"] * 1e-3) / 1e12 if gemm["ms"] > 0 else 0.0
    # DRAM traffic per GEMM launch from the ncu capture of one layer of this model at M = 8192 rows
    # (the committed summary of that capture sits with the other profiles): 0.117 GB of weights per layer, which do not grow with M, plus
    # 0.971 GB of activations, which grow in proportion to the rows; six launches per layer.
    traffic, traffic_note = None, None
    if bf16 and (w.d, w.L, w.H, w.mlp_mult) == (2048, 8, 16, 4) and gemm["launches"] > 0:
        rows_per_launch = st["env_steps"] * w.H / (gemm["launches"] / 6.0 / w.L)
        traffic = (0.117e9 + 0.971e9 * rows_per_launch / 8192.0) / 6.0
        traffic_note = "bytes per launch, ncu capture at M=8192 scaled to M=%d (activation part in proportion)" % round(rows_per_launch)
    roofline = {"bound": bound, "kernel": "gemm", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak if peak else None, "traffic": traffic, "traffic_note": traffic_note,
                "algorithmic_bytes_per_launch": gemm["bytes"] / gemm["launches"] if gemm["launches"] else None,
                "peak_source": peak_note,
                "launches": gemm["launches"], "avg_launch_us": 1e3 * gemm["ms"] / max(1, gemm["launches"]),
                "class_share": {k: round(c["ms"] / total_ms, 4) for k, c in cls.items()},
                "class_ms_per_step": {k: round(c["ms"] / args.steps, 4) for k, c in cls.items()}}
    xa = cls["cross_attn"]
    if xa["ms"] > 0:
        roofline["cross_attn_hbm"] = {"achieved_gbs": xa["bytes"] / (xa["ms"] * 1e-3) / 1e9, "peak_gbs": peaks["hbm_gbs"],
                                      "frac": xa["bytes"] / (xa["ms"] * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    # whole-path fraction of the quota-scaled roofline (the metric's second half)
    flops_step = workload_flops(w, [envs[e] for e in ids])
    t_tensor = flops_step / (peak * 1e12)
    min_bytes = kv_bytes + 2 * noise.numel() * 4 + sum(t.numel() * t.element_size() for t in
                                                       [wt["w_in"], wt["w_out"]] + [v for l in wt["layers"] for v in l.values()])
    t_hbm = min_bytes / (peaks["hbm_gbs"] * 1e9)
    path = {"flops_per_step": flops_step, "t_roof_ms": 1e3 * max(t_tensor, t_hbm), "frac": max(t_tensor, t_hbm) / (ms_step * 1e-3),
            "frac_vs_sustained": (flops_step / (peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * 1e12 * q_eff / N_SMS)) / (ms_step * 1e-3)
            if bf16 else None}

    # ---- end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        h_noise = noise.cpu().pin_memory()
        h_out = torch.empty_like(h_noise).pin_memory()
        h_kv = {e: envs[e].kv.cpu().pin_memory() for e in ids}

        def step_host():
            for g in groups:
                lo = pos[g[0]]
                gen.submit_host(g, [h_kv[e] for e in g], h_noise[lo:lo + len(g)], h_out[lo:lo + len(g)], sm_quota=quota,
                                stream=stream, step_index=[envs[e].step for e in g])
            gen.sync()

        n_e2e = max(1, min(args.steps, 3))
        step_host()
        barrier()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        a0.record(stream)
        for _ in range(n_e2e):
            step_host()
        a1.record(stream)
        barrier()
        wall = (time.perf_counter() - t0) / n_e2e
        ems = a0.elapsed_time(a1) / n_e2e   # device-side span; the wall time is reported beside it
        if world > 1:
            t = torch.tensor([ems], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ems = float(t.item())
        e2e = {"value": world * w.B / (ems * 1e-3), "unit": UNIT, "h2d_bytes_per_step": kv_bytes + noise.numel() * 4,
               "d2h_bytes_per_step": noise.numel() * 4, "ms_per_step": ems, "wall_ms_per_step": wall * 1e3, "steps": n_e2e,
               "equal_to_device_path": bool(torch.equal(h_out.to(dev), out))}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cores = os.cpu_count() or 1
        rate, desc, _ = oracle_sample_rate(w, seed, cores)
        cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}

    gen.destroy()
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": n_warm,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if bf16 else "f32", "data": "synthetic",
            "config": {"workload": "configs[%d] %s" % (args.config, w.name), "envs_per_gpu": w.B, "H": w.H, "A": w.A, "d": w.d,
                       "L": w.L, "heads": w.n_heads, "P": list(w.P), "K": w.K, "d_ctx": w.d_ctx, "groups": len(groups),
                       "group_sizes": [min(map(len, groups)), max(map(len, groups))], "sm_quota": q_eff,
                       "inflight_groups": inflight, "corunner": bool(co_stream is not None),
                       "green_ctx": {"requested": bool(args.green_ctx), "active": bool(st0["green_ctx_active"]), "partition_sms": st0["green_ctx_sms"]},
                       "l2": ("inputs (%.2f GB of prefix planes plus weights) larger than the 126 MB L2" % (kv_bytes / 1e9))
                       if kv_bytes > 126e6 else "inputs fit in L2 and L2 is not flushed: small parity-size case, not a bench line",
                       "seed": seed},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "path_roofline": path,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_pgen_sweep(args):
    """The paper's generation profiling (section 4.3.2: observation batches replayed under different SM
    quotas and batch sizes, stored in a lookup table): chunks/s of one group of B_g environments at
    quota s_g, on the programming model's example grid (20/40/60/80 % x 8/16/32/64).  The table is the
    P_gen input of ebrl_alloc_elastic."""
    import torch
    from paper_2609_27547_b200 import binding as B
    from paper_2609_27547_b200 import synth
    torch.cuda.set_device(0)
    w = synth.WORKLOADS[args.config]
    seed = args.seed or synth.DEFAULT_SEED
    quotas, batches = [20, 40, 60, 80], [8, 16, 32, 64]
    wt = synth.make_weights(w, seed, device="cuda")
    envs = [synth.make_env(w, e, seed, device="cuda") for e in range(max(batches))]
    gen = B.ActGen(B.cfg_for(w, max_group_envs=max(batches), max_inflight_groups=1), wt)
    stream = torch.cuda.Stream()
    noise = torch.stack([e.noise for e in envs]).contiguous()
    out = torch.empty_like(noise)
    rate = []
    for q in quotas:
        sms = max(1, round(N_SMS * q / 100))
        row = []
        for b in batches:
            def step():
                gen.submit(list(range(b)), [e.kv for e in envs[:b]], noise[:b], out[:b], sm_quota=sms, stream=stream)
                gen.sync()
            for _ in range(3):
                step()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.steps):
                step()
            e1.record(stream)
            torch.cuda.synchronize()
            row.append(b * args.steps / (e0.elapsed_time(e1) * 1e-3))
        rate.append(row)
    gen.destroy()
    print(json.dumps({"pgen": {"workload": "configs[%d] %s" % (args.config, w.name), "unit": UNIT, "quota_pct": quotas,
                               "quota_sms": [max(1, round(N_SMS * q / 100)) for q in quotas], "batch": batches, "rate": rate}}))


def main():
    args = parse_args()
    if args.pgen_sweep:
        return run_pgen_sweep(args)
    if args.rollout_sim:
        import torch
        from paper_2609_27547_b200 import rollout_sim as R
        from paper_2609_27547_b200 import synth
        torch.cuda.set_device(0)
        w = synth.WORKLOADS[args.config]
        wt = synth.make_weights(w, args.seed or synth.DEFAULT_SEED, device="cuda")
        n = args.envs or 128
        quota = w.quota if args.quota < 0 else args.quota
        out = [R.run(w, wt, n, max(1, args.steps), pol, quota=quota, max_group=64, sim_steps_per_chunk=w.H).summary()
               for pol in ("chunk", "step")]
        print(json.dumps({"rollout_sim": {"workload": "configs[%d] %s" % (args.config, w.name), "envs": n, "chunks_per_env": max(1, args.steps),
                                          "sm_quota": quota or N_SMS, "simulator": "log-normal step time, mean 40 ms, P99 60 ms, H steps per chunk",
                                          "policies": out}}))
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
