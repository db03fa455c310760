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
