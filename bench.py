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
  in a second pass of the same steps.  ``frac`` is taken against what the quota's SMs can issue at
  the SM clock sampled during that pass (8192 dense bf16 FLOP per clock per SM); the fractions
  against MEASURED_PEAKS.json's burst and sustained figures scaled by quota/SMs (measured on the
  whole, power-capped chip at a lower clock) and against the nominal 2250 TFLOP/s are beside it.
* ``cpu_baseline``: the fp64 oracle as it stands on this machine's host cores, on a bounded sample.
* ``--impl reference`` times that oracle alone (there is no other reference implementation).

``--gpus N`` with N > 1 starts N ranks (one per GPU, through torch.distributed.run on 127.0.0.1)
unless the process already is one of them (RANK / WORLD_SIZE in the environment).  Each rank runs
the same workload shape on its own shard of the job's environment ids (id mod world; environments
are independent, so there is no data-path collective); the ranks meet only for the barriers and
the max-over-ranks of the step time; ``value`` counts the environments of all ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
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
BF16_FLOP_PER_CLK_SM = 8192                        # dense bf16 tcgen05: 2250 TFLOP/s nominal = 148 SMs x 8192 x 1.856 GHz
FP32_FLOP_PER_CLK_SM = 256                         # 128 FFMA lanes x 2
NOMINAL_BF16_TFLOPS = 2250.0


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


def parse_args(argv=None):
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
    ap.add_argument("--fused", action="store_true",
                    help="run every batch through the persistent step kernel (one resident grid for all Euler steps)")
    ap.add_argument("--sm-split", action="store_true",
                    help="harness: the step as one batch on the quota against two half-batches side by side on two streams, "
                         "each on a share of the quota (does an SM split overlap the K/V stream with the projections?)")
    ap.add_argument("--sweep", action="store_true",
                    help="one line per other configuration: configs[0..2], and configs[3] at quotas 148/74/37/16 with and "
                         "without the streaming co-runner (the committed summary of these lines sits with the profiles)")
    ap.add_argument("--stub-step-ms", type=float, default=0.0,
                    help="testing the rank plumbing without a GPU: every step is a sleep of this many ms (+ the rank), "
                         "ranks talk over gloo, the line says \"data\": \"stub\" -- never a measurement")
    return ap.parse_args(argv)


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
        "config": {"workload": synth.workload_label(args.config), "note": "fp64 CPU oracle on host cores; each step is a bounded sample"},
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


class RankContext:
    """One process per GPU: which rank this is, and the only things ranks do together -- a barrier
    and the maximum of a number (the step time).  Environments are independent (section 4.2.2), so
    the data path has no collective; `backend` is "nccl" on GPUs and "gloo" for the CPU test of
    this plumbing."""

    def __init__(self, backend: str, device=None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            if backend == "nccl":
                dist.init_process_group("nccl", device_id=device)
            else:
                dist.init_process_group(backend, rank=self.rank, world_size=self.world)
            self.dist = dist
        self.device = device

    def shard(self, envs_per_rank: int):
        """This rank's environment ids: the job has world x envs_per_rank environments (weak scaling),
        environment e belongs to rank e mod world."""
        from paper_2609_27547_b200 import synth
        return synth.shard_env_ids(self.world * envs_per_rank, self.rank, self.world)

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        if self.device is not None:
            import torch
            torch.cuda.synchronize(self.device)

    def max_over_ranks(self, x: float) -> float:
        if self.dist is None:
            return float(x)
        import torch
        t = torch.tensor([float(x)], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        if self.device is not None:
            t = t.float()
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def job_throughput(ctx: RankContext, envs_per_rank: int, ms_local: float, steps: int):
    """(ms per step = the slowest rank's, whole-job chunks/s = the environments all ranks processed / that time)."""
    ms_step = ctx.max_over_ranks(ms_local) / steps
    return ms_step, ctx.world * envs_per_rank / (ms_step * 1e-3)


def run_stub(args):
    """The rank plumbing of run_ours with the GPU step replaced by a sleep (tests only)."""
    from paper_2609_27547_b200 import synth
    ctx = RankContext("gloo")
    w = synth.WORKLOADS[args.config]
    if args.envs:
        w = synth.scaled(w, B=args.envs)
    seed = args.seed or synth.DEFAULT_SEED
    ids = ctx.shard(w.B)
    groups = synth.arrival_groups(w, seed + ctx.rank, env_ids=ids)
    assert sorted(e for g in groups for e in g) == ids
    ctx.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep((args.stub_step_ms + ctx.rank) * 1e-3)
    ms = (time.perf_counter() - t0) * 1e3
    ctx.barrier()
    ms_step, value = job_throughput(ctx, w.B, ms, args.steps)
    if ctx.dist is not None:
        gathered = [None] * ctx.world
        ctx.dist.all_gather_object(gathered, ids)
    else:
        gathered = [ids]
    if ctx.rank == 0:
        print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": ctx.world, "steps": args.steps,
                          "warmup": 0, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                          "data": "stub", "config": {"workload": synth.workload_label(args.config), "envs_per_gpu": w.B},
                          "shards": gathered, "gpu_launches": 0}))
    ctx.close()


def launch_ranks(args):
    """`--gpus N` outside torchrun: start N ranks of this script on this node."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def run_ours(args, emit=True):
    import torch
    from paper_2609_27547_b200 import binding as B
    from paper_2609_27547_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ctx = RankContext("nccl", dev)
    world, rank = ctx.world, ctx.rank

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
    ids = ctx.shard(w.B)
    wt = synth.make_weights(w, seed, device=dev)
    envs = {e: synth.make_env(w, e, seed, device=dev) for e in ids}
    groups = synth.arrival_groups(w, seed + rank, env_ids=ids)
    order = [e for g in groups for e in g]
    pos = {e: i for i, e in enumerate(order)}
    noise = torch.stack([envs[e].noise for e in order]).contiguous()
    out = torch.empty_like(noise)
    kv_bytes = sum(envs[e].kv.numel() * envs[e].kv.element_size() for e in ids)
    inflight = args.inflight
    flags = (B.FLAG_FORCE_SIMT if args.simt else 0) | (B.FLAG_GREEN_CTX if args.green_ctx else 0) | \
        (B.FLAG_FORCE_FUSED if args.fused else 0)
    cfg = B.cfg_for(w, max_group_envs=max(len(g) for g in groups), max_inflight_groups=inflight, flags=flags, device=local)
    gen = B.ActGen(cfg, wt)
    stream = torch.cuda.Stream(dev)

    def step():
        for g in groups:
            lo = pos[g[0]]
            gen.submit(g, [envs[e].kv for e in g], noise[lo:lo + len(g)], out[lo:lo + len(g)], sm_quota=quota,
                       stream=stream, step_index=[envs[e].step for e in g])
        gen.sync()

    n_warm = max(args.min_warmup, args.warmup)
    tw0 = time.perf_counter()
    for _ in range(n_warm):
        step()
    torch.cuda.synchronize(dev)
    warm_ms_step = (time.perf_counter() - tw0) * 1e3 / max(1, n_warm)

    # the synthetic simulation co-runner on the SMs outside the quota: one launch sized (from the
    # warm-up step time and a timed pass of its own) to outlast the timed region
    co = None
    if args.corunner and q_eff < N_SMS:
        co_stream = gen.rest_stream(quota) if args.green_ctx else None
        fenced = co_stream is not None
        if co_stream is None:
            co_stream = torch.cuda.Stream(dev)
        co_buf = torch.zeros(1 << 29, dtype=torch.float32, device=dev)   # 2 GiB: 4 GiB of traffic per pass
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record(co_stream)
        B.sim_corunner_launch(co_buf, 2, N_SMS - q_eff, co_stream)
        c1.record(co_stream)
        torch.cuda.synchronize(dev)
        pass_ms_alone = c0.elapsed_time(c1) / 2
        co_passes = max(4, int(3.0 * warm_ms_step * args.steps / max(pass_ms_alone, 1e-3)) + 2)
        co = {"stream": co_stream, "buf": co_buf, "passes": co_passes, "fenced": fenced, "pass_ms_alone": pass_ms_alone,
              "e0": torch.cuda.Event(enable_timing=True), "e1": torch.cuda.Event(enable_timing=True)}

    gen.reset_stats()
    ctx.barrier()
    sampler = ClockSampler(local)
    if co is not None:
        co["e0"].record(co["stream"])
        B.sim_corunner_launch(co["buf"], co["passes"], N_SMS - q_eff, co["stream"])
        co["e1"].record(co["stream"])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    co_outlasted = (not co["e1"].query()) if co is not None else None   # still running when the last step's sync returned
    ctx.barrier()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    st0 = gen.stats()
    launches = st0["kernel_launches"]
    ms_step, value = job_throughput(ctx, w.B, ms, args.steps)
    co_report = None
    if co is not None:
        torch.cuda.synchronize(dev)
        co_ms = co["e0"].elapsed_time(co["e1"])
        co_report = {"ctas": N_SMS - q_eff, "passes": co["passes"], "gb_per_pass": 2 * co["buf"].numel() * 4 / 1e9,
                     "achieved_gbs": co["passes"] * 2 * co["buf"].numel() * 4 / (co_ms * 1e-3) / 1e9,
                     "alone_gbs": 2 * co["buf"].numel() * 4 / (co["pass_ms_alone"] * 1e-3) / 1e9,
                     "outlasted_timed_region": bool(co_outlasted),
                     "placement": "remainder SM partition (driver-enforced)" if co["fenced"] else
                                  "primary context: only the grid sizes keep the two apart, the driver may place its CTAs anywhere"}

    # ---- roofline of the dominant kernel class: a second pass with events around every launch
    gen.reset_stats()
    gen.set_timing(True)
    sampler2 = ClockSampler(local)
    for _ in range(args.steps):
        step()
    clocks2 = sampler2.stop()
    st = gen.stats()
    gen.set_timing(False)
    cls = st["classes"]
    total_ms = sum(c["ms"] for c in cls.values()) or 1.0
    gemm = cls["fused"] if cls["fused"]["launches"] else cls["gemm"]
    bf16 = w.dtype == "bf16"
    use_tensor = not args.simt            # fp32 models run their projections on the tensor cores too, as six bf16 products each
    mhz = clocks2.get("sm_mhz") or clocks.get("sm_mhz") or 1965.0
    per_clk = (BF16_FLOP_PER_CLK_SM / (1.0 if bf16 else 6.0)) if use_tensor else FP32_FLOP_PER_CLK_SM
    peak_clock = q_eff * per_clk * mhz * 1e6 / 1e12
    achieved = gemm["flops"] / (gemm["ms"] * 1e-3) / 1e12 if gemm["ms"] > 0 else 0.0
    if use_tensor:
        bound = "tensor"
        div = 1.0 if bf16 else 6.0
        alt = {"measured_burst_x_quota": peaks["bf16_tflops"] * q_eff / N_SMS / div,
               "measured_sustained_x_quota": peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * q_eff / N_SMS / div,
               "nominal_2250_x_quota": NOMINAL_BF16_TFLOPS * q_eff / N_SMS / div}
        if not bf16:
            alt["fp32_ffma_at_max_clock_x_quota"] = FP32_ALU_TFLOPS * q_eff / N_SMS
        peak_note = ("fp32 products as six bf16 tensor-core products each: the bf16 figures divided by 6; " if not bf16 else "") + \
                    ("%d SMs x %d FLOP/clk x %.0f MHz (median SM clock sampled during the per-kernel timing pass); the %s full-chip "
                     "figures (burst %.1f, sustained %.1f TFLOP/s, taken at a power-capped clock) scaled by %d/%d are in frac_vs"
                     % (q_eff, per_clk, mhz, peaks["source"], peaks["bf16_tflops"],
                        peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]), q_eff, N_SMS))
    else:
        bound = "alu"
        alt = {"fp32_ffma_at_max_clock_x_quota": FP32_ALU_TFLOPS * q_eff / N_SMS}
        peak_note = "%d SMs x 128 FFMA lanes x 2 x %.0f MHz (median SM clock sampled during the per-kernel timing pass)" % (q_eff, mhz)
    traffic, traffic_note = gemm_traffic(w, st, gemm)
    roofline = {"bound": bound, "kernel": "fused_steps" if cls["fused"]["launches"] else "gemm", "achieved": achieved, "peak": peak_clock, "unit": "TFLOP/s",
                "frac": achieved / peak_clock if peak_clock else None,
                "frac_vs": {k: achieved / v for k, v in alt.items()}, "peak_alternatives": alt,
                "traffic": traffic, "traffic_note": traffic_note,
                "algorithmic_bytes_per_launch": gemm["bytes"] / gemm["launches"] if gemm["launches"] else None,
                "peak_source": peak_note, "clocks_timing_pass": clocks2,
                "launches": gemm["launches"], "avg_launch_us": 1e3 * gemm["ms"] / max(1, gemm["launches"]),
                "class_share": {k: round(c["ms"] / total_ms, 4) for k, c in cls.items()},
                "class_ms_per_step": {k: round(c["ms"] / args.steps, 4) for k, c in cls.items()}}
    xa = cls["cross_attn"]
    if xa["ms"] > 0:
        roofline["cross_attn_hbm"] = {"achieved_gbs": xa["bytes"] / (xa["ms"] * 1e-3) / 1e9, "peak_gbs": peaks["hbm_gbs"],
                                      "frac": xa["bytes"] / (xa["ms"] * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    # whole-path fraction of the quota-scaled roofline (the metric's second half): the slower of every FLOP at the
    # tensor (or ALU) rate of the quota's SMs and the compulsory bytes at the measured HBM bandwidth, over the step time
    flops_step = workload_flops(w, [envs[e] for e in ids])
    min_bytes = kv_bytes + 2 * noise.numel() * 4 + sum(t.numel() * t.element_size() for t in
                                                       [wt["w_in"], wt["w_out"]] + [v for l in wt["layers"] for v in l.values()])
    t_hbm = min_bytes / (peaks["hbm_gbs"] * 1e9)
    mhz1 = clocks.get("sm_mhz") or mhz
    path_peaks = {"clock_scaled": q_eff * per_clk * mhz1 * 1e6 / 1e12}
    path_peaks.update(alt)
    path = {"flops_per_step": flops_step, "min_bytes_per_step": min_bytes,
            "frac": max(flops_step / (path_peaks["clock_scaled"] * 1e12), t_hbm) / (ms_step * 1e-3),
            "frac_vs": {k: max(flops_step / (v * 1e12), t_hbm) / (ms_step * 1e-3) for k, v in path_peaks.items() if k != "clock_scaled"},
            "t_roof_ms": {k: 1e3 * max(flops_step / (v * 1e12), t_hbm) for k, v in path_peaks.items()},
            "note": "frac: against %d SMs x %d FLOP/clk x the %.0f MHz sampled during the timed steps; "
                    "frac_vs.measured_burst_x_quota is the metric's 'quota-scaled bf16 tensor roofline' with the measured full-chip peak"
                    % (q_eff, per_clk, mhz1)}

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
        ctx.barrier()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        a0.record(stream)
        for _ in range(n_e2e):
            step_host()
        a1.record(stream)
        ctx.barrier()
        wall = (time.perf_counter() - t0) / n_e2e
        ems, evalue = job_throughput(ctx, w.B, a0.elapsed_time(a1), n_e2e)   # device-side span; the wall time is reported beside it
        e2e = {"value": evalue, "unit": UNIT, "h2d_bytes_per_step": kv_bytes + noise.numel() * 4,
               "d2h_bytes_per_step": noise.numel() * 4, "ms_per_step": ems, "wall_ms_per_step": wall * 1e3, "steps": n_e2e,
               "equal_to_device_path": bool(torch.equal(h_out.to(dev), out))}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cores = os.cpu_count() or 1
        rate, desc, _ = oracle_sample_rate(w, seed, cores)
        cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}

    gen.destroy()
    line = None
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": n_warm,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if bf16 else "f32", "data": "synthetic",
            "config": {"workload": synth.workload_label(args.config), "envs_per_gpu": w.B, "H": w.H, "A": w.A, "d": w.d,
                       "L": w.L, "heads": w.n_heads, "P": list(w.P), "K": w.K, "d_ctx": w.d_ctx, "groups": len(groups),
                       "group_sizes": [min(map(len, groups)), max(map(len, groups))], "sm_quota": q_eff,
                       "inflight_groups": inflight, "corunner": co_report if co_report is not None else False,
                       "kernels": "persistent step kernel" if args.fused else ("plain ALU" if args.simt else "one kernel per operation"),
                       "green_ctx": {"requested": bool(args.green_ctx), "active": bool(st0["green_ctx_active"]), "partition_sms": st0["green_ctx_sms"]},
                       "sharding": "environment id mod %d; no data-path collective" % world,
                       "l2": ("inputs (%.2f GB of prefix planes plus weights) larger than the 126 MB L2" % (kv_bytes / 1e9))
                       if kv_bytes > 126e6 else "inputs fit in L2 and L2 is not flushed: small parity-size case, not a bench line",
                       "seed": seed},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "path_roofline": path,
            "cpu_baseline": cpu,
        }
        if emit:
            print(json.dumps(line))
    ctx.close()
    return line


def gemm_traffic(w, st, gemm):
    """DRAM bytes per GEMM launch from the ncu capture recorded beside the other profile summaries
    (a capture of one layer's six GEMMs at a smaller M, scaled to this run's rows: the weight part
    does not grow with M, the activation part grows in proportion).  None when no capture covers
    this model."""
    path = os.path.join(ROOT, "profiles", "gemm_dram_traffic.json")
    if not os.path.exists(path) or gemm["launches"] <= 0:
        return None, None
    with open(path) as f:
        rec = json.load(f)
    for c in rec.get("captures", []):
        m = c["model"]
        if (m["d"], m["L"], m["H"], m["mlp_mult"], m["dtype"]) == (w.d, w.L, w.H, w.mlp_mult, w.dtype):
            rows = st["env_steps"] * w.H / (gemm["launches"] / float(c["gemms_per_layer"]) / w.L)
            per_layer = c["weight_bytes_per_layer"] + c["activation_bytes_per_layer"] * rows / c["rows"]
            return per_layer / c["gemms_per_layer"], ("bytes per launch: %s, M=%d scaled to M=%d (activation part in proportion)"
                                                       % (c["source"], c["rows"], round(rows)))
    return None, None


def run_sweep(args):
    """One JSON line per other configuration (the bench line proper is configs[4])."""
    import copy
    plan = [(0, -1, False), (1, -1, False), (2, -1, False)]
    for q in (148, 74, 37, 16):
        plan.append((3, q, False))
        if q < N_SMS:
            plan.append((3, q, True))
    plan += [(4, 148, False), (4, 37, False)]                 # the bench configuration at other quotas than its own 74
    plan.append((12, -1, False))                              # configurations 2 and 3 on the configs[1] model
    for q in (148, 74, 37, 16):
        plan.append((13, q, False))
        if q < N_SMS:
            plan.append((13, q, True))
    for cfg_i, q, co in plan:
        a = copy.copy(args)
        a.config, a.corunner, a.no_cpu, a.no_e2e, a.quota = cfg_i, co, True, True, q
        a.steps = {1: 10, 4: 3, 12: 10, 13: 5}.get(cfg_i, max(args.steps, 20))
        run_ours(a)


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
    gen = B.ActGen(B.cfg_for(w, max_group_envs=max(batches), max_inflight_groups=1, flags=B.FLAG_FORCE_FUSED if args.fused else 0), wt)
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
    print(json.dumps({"pgen": {"workload": synth.workload_label(args.config), "unit": UNIT, "quota_pct": quotas,
                               "kernels": "persistent step kernel" if args.fused else "one kernel per operation",
                               "quota_sms": [max(1, round(N_SMS * q / 100)) for q in quotas], "batch": batches, "rate": rate}}))


def run_sm_split(args):
    """Can the HBM-bound K/V stream of one half of the environments hide behind the tensor-bound projections of
    the other half?  Times a step (a) as one batch on the whole quota and (b) as two half-batches submitted to two
    streams, each with a share of the quota, so that the two run side by side and drift out of phase (one in
    attention while the other is in its projections).  Same arithmetic per environment in both (bit-identical
    results: checked here)."""
    import torch
    from paper_2609_27547_b200 import binding as B
    from paper_2609_27547_b200 import synth
    torch.cuda.set_device(0)
    w = synth.WORKLOADS[args.config]
    seed = args.seed or synth.DEFAULT_SEED
    quota = args.quota if args.quota >= 0 else w.quota
    quota = quota or N_SMS
    nb = args.envs or w.B
    wt = synth.make_weights(w, seed, device="cuda")
    envs = [synth.make_env(w, e, seed, device="cuda") for e in range(nb)]
    gen = B.ActGen(B.cfg_for(w, max_group_envs=nb, max_inflight_groups=1), wt)
    noise = torch.stack([e.noise for e in envs]).contiguous()
    out = torch.empty_like(noise)
    main_s, side = torch.cuda.Stream(), [torch.cuda.Stream(), torch.cuda.Stream()]
    kv = [e.kv for e in envs]

    def one_batch():
        gen.submit(list(range(nb)), kv, noise, out, sm_quota=quota, stream=main_s)
        gen.sync()

    def split(shares):
        def step():
            ev = torch.cuda.Event()
            ev.record(main_s)
            lo = 0
            for p, q in enumerate(shares):
                hi = nb if p == len(shares) - 1 else lo + nb // len(shares)
                side[p].wait_event(ev)
                gen.submit(list(range(lo, hi)), kv[lo:hi], noise[lo:hi], out[lo:hi], sm_quota=q, stream=side[p])
                done = torch.cuda.Event()
                done.record(side[p])
                main_s.wait_event(done)
                lo = hi
            gen.sync()
        return step

    def timed(step):
        for _ in range(max(args.min_warmup, 1)):
            step()
        mon = ClockSampler(0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(main_s)
        for _ in range(args.steps):
            step()
        e1.record(main_s)
        torch.cuda.synchronize()
        clk = mon.stop()
        return e0.elapsed_time(e1) / args.steps, clk.get("sm_mhz"), out.clone()

    res = {"workload": synth.workload_label(args.config), "envs": nb, "quota": quota, "steps": args.steps, "unit": "ms per step"}
    ms, mhz, ref = timed(one_batch)
    res["one_batch"] = {"ms": ms, "sm_mhz": mhz}
    for shares in ([quota // 2, quota - quota // 2], [quota, quota]):   # the second one occupies 2 x quota SMs: context, not a quota run
        ms, mhz, got = timed(split(shares))
        res["two_half_batches_%d_%d" % tuple(shares)] = {"ms": ms, "sm_mhz": mhz, "bit_identical": bool(torch.equal(got, ref))}
    gen.destroy()
    print(json.dumps({"sm_split": res}))


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return launch_ranks(args)
    if args.stub_step_ms > 0:
        return run_stub(args)
    if args.sweep:
        return run_sweep(args)
    if args.pgen_sweep:
        return run_pgen_sweep(args)
    if args.sm_split:
        return run_sm_split(args)
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
        print(json.dumps({"rollout_sim": {"workload": synth.workload_label(args.config), "envs": n, "chunks_per_env": max(1, args.steps),
                                          "sm_quota": quota or N_SMS, "simulator": "log-normal step time, mean 40 ms, P99 60 ms, H steps per chunk",
                                          "policies": out}}))
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
