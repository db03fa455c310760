"""Multi-GPU plan on CPU: environments are sharded across ranks with no data-path collective;
the only cross-rank step is the max-over-ranks of the timing.  Two gloo ranks."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_27547_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.scaled(synth.WORKLOADS[2], B=50)
    mine = synth.shard_env_ids(w.B, rank, world)
    # every rank draws its own environments without talking to anyone
    chk = sum(float(synth.make_env(w, e).noise.double().sum()) for e in mine)
    groups = synth.arrival_groups(w, synth.DEFAULT_SEED + rank, env_ids=mine)
    assert sorted(e for g in groups for e in g) == mine
    gathered = [None] * world
    dist.all_gather_object(gathered, (mine, chk))
    t = torch.tensor([10.0 + rank])           # a rank's step time; the job's time is the slowest rank's
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        out.put((gathered, float(t.item())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_environments_disjointly():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    gathered, tmax = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    ids = [set(g[0]) for g in gathered]
    assert ids[0].isdisjoint(ids[1]) and ids[0] | ids[1] == set(range(50))
    assert tmax == 11.0
    w = synth.scaled(synth.WORKLOADS[2], B=50)
    total = sum(float(synth.make_env(w, e).noise.double().sum()) for e in range(50))
    assert abs(sum(g[1] for g in gathered) - total) < 1e-9   # the shards together are the whole job


def test_bench_gpus_2_starts_two_ranks_and_aggregates_over_them():
    """`bench.py --gpus 2` outside torchrun starts its own two ranks.  With the GPU step replaced by
    a sleep (--stub-step-ms: rank r sleeps 30 + r ms per step) the rank plumbing runs on CPU over
    gloo: disjoint id-mod-world shards of 2 x B environments, the step time is the slowest rank's,
    and `value` counts the environments of both ranks."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--config", "2", "--envs", "50",
                        "--steps", "4", "--stub-step-ms", "30"], capture_output=True, text=True, timeout=300, env=env)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["data"] == "stub" and d["scaling"] == "weak"
    a, b = (set(x) for x in d["shards"])
    assert a.isdisjoint(b) and a | b == set(range(100)) and all(e % 2 == 0 for e in a)
    assert 31.0 <= d["ms_per_step"] < 60.0                   # the slower rank (31 ms sleeps), not the faster one
    assert abs(d["value"] - 100 / (d["ms_per_step"] * 1e-3)) < 1e-6 * d["value"]


def test_job_throughput_single_rank():
    import bench
    ctx = bench.RankContext("gloo")
    assert ctx.world == 1 and ctx.shard(7) == list(range(7))
    ms_step, value = bench.job_throughput(ctx, 2048, 5580.0, 10)
    assert ms_step == 558.0 and abs(value - 2048 / 0.558) < 1e-9
