"""The seeded input generator: determinism, independence from grouping, distributions."""
import numpy as np
import torch

from paper_2609_27547_b200 import synth


def test_values_depend_only_on_seed_tag_env_index():
    a = synth.normal(7, "x", 3, (1000,))
    b = synth.normal(7, "x", 3, (10, 100))
    assert torch.equal(a, b.reshape(-1))
    assert torch.equal(a[:500], synth.normal(7, "x", 3, (500,)))            # a prefix is a prefix
    assert torch.equal(a, synth.normal(7, "x", 3, (1000,), chunk=64))       # chunking is invisible
    assert not torch.equal(a, synth.normal(8, "x", 3, (1000,)))
    assert not torch.equal(a, synth.normal(7, "y", 3, (1000,)))
    assert not torch.equal(a, synth.normal(7, "x", 4, (1000,)))


def test_normal_moments_and_bf16_rounding():
    x = synth.normal(1, "m", 0, (400000,)).double()
    assert abs(x.mean()) < 5e-3 and abs(x.std() - 1) < 5e-3
    assert abs((x ** 3).mean()) < 2e-2 and abs((x ** 4).mean() - 3) < 5e-2
    f = synth.normal(1, "r", 0, (4096,))
    h = synth.normal(1, "r", 0, (4096,), dtype=torch.bfloat16)
    assert torch.equal(h, f.to(torch.bfloat16))                               # one RNE rounding
    w = synth.normal(1, "w", 0, (256, 64), std=64 ** -0.5)
    assert abs(w.double().var() * 64 - 1) < 0.05                              # variance 1/fan_in


def test_env_inputs_do_not_depend_on_group_or_workload_size():
    w = synth.WORKLOADS[2]
    e1 = synth.make_env(w, 17)
    e2 = synth.make_env(synth.scaled(w, B=20), 17)
    assert e1.P == e2.P and e1.step == e2.step and torch.equal(e1.kv, e2.kv) and torch.equal(e1.noise, e2.noise)
    assert 64 <= e1.P <= 512 and 0 <= e1.step < w.K
    Ps = [synth.uniform_int(synth.DEFAULT_SEED, "prefix_len", e, 64, 512) for e in range(300)]
    assert min(Ps) < 100 and max(Ps) > 470


def test_arrival_groups_partition_the_ids():
    for cfg in (2, 4):
        w = synth.WORKLOADS[cfg]
        g = synth.arrival_groups(w)
        flat = [e for grp in g for e in grp]
        assert sorted(flat) == list(range(w.B))
        assert all(w.group[0] <= len(x) <= w.group[1] for x in g[:-1]) and 1 <= len(g[-1]) <= w.group[1]
        assert flat != list(range(w.B))                                        # shuffled
        assert g == synth.arrival_groups(w) and g != synth.arrival_groups(w, synth.DEFAULT_SEED + 1)
    assert synth.arrival_groups(synth.WORKLOADS[1]) == [list(range(256))]


def test_flop_count_matches_the_configs_table():
    # per-chunk GFLOP of the five configurations (2mnk counting)
    want = {0: 0.120, 1: 9.744, 3: 0.135, 4: 158.56}
    for c, gf in want.items():
        w = synth.WORKLOADS[c]
        assert abs(w.flops_per_env_step(w.P[0]) * w.K / 1e9 - gf) / gf < 5e-3
