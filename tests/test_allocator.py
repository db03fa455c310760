"""The elastic allocator (Algorithm 1, Eq. 2) and the re-balance trigger: the oracle is pinned by
a closed form and by brute force over every integer quota; the library's implementation must make
exactly the oracle's decisions.  CPU only."""
import random

import pytest

from oracle import allocator_oracle as O
from paper_2609_27547_b200 import alloc as A


def _tables(rng, monotone=True):
    q = [20, 40, 60, 80]
    bg, bt = [8, 16, 32, 64], [4, 8, 16]
    def table(nb, scale):
        rows, base = [], [rng.uniform(0.5, 1.5) * scale * (1 + 0.3 * j) for j in range(nb)]
        acc = [0.0] * nb
        for _ in q:
            acc = [a + rng.uniform(0.2, 1.0) * b for a, b in zip(acc, base)] if monotone else [rng.uniform(0.1, 3) * b for b in base]
            rows.append(list(acc))
        return rows
    gen = (q, bg, table(4, 10.0), [2.0, 4.0, 8.0, 16.0])
    train = (q, bt, table(3, 14.0), [10.0, 20.0, 40.0])
    return gen, train


def test_linear_profiles_balance_point_closed_form():
    """P_gen = a s, P_train = b s, simulator never the limit: rollout and training balance where
    a s_g = b (R - s_g), i.e. s_g = b R / (a + b) with R = 100 - s_sim."""
    a, b = 3.0, 5.0
    q = [1, 100]
    gen = O.Profile(q, [1], [[a * 1], [a * 100]], [0.0])
    train = O.Profile(q, [1], [[b * 1], [b * 100]], [0.0])
    r = O.elastic_allocation(64, 4, [10], [1e9], gen, train, 5, 5, 1e9)
    R = 90
    exact = b * R / (a + b)                       # 56.25
    assert r["E"] == 16 and r["s_sim"] == 10
    assert abs(r["s_g"] - exact) <= 1.0 and r["s_g"] + r["s_t"] == R
    assert abs(r["theta"] - a * exact) <= a        # within one percentage point of the optimum
    assert r["iterations"] <= 7                    # ceil(log2(80))


@pytest.mark.parametrize("seed", range(12))
def test_oracle_bisection_equals_brute_force_on_monotone_tables(seed):
    rng = random.Random(seed)
    g, t = _tables(rng)
    gen, train = O.Profile(*g), O.Profile(*t)
    sq, sr = [10, 20, 30], [40.0 * rng.uniform(0.5, 2), 0, 0]
    sr[1] = sr[0] * 1.5; sr[2] = sr[1] * 1.02            # knee at 20 %
    M = rng.choice([30.0, 60.0])
    r = O.elastic_allocation(96, 3, sq, sr, gen, train, 10, 10, M)
    bf = O.brute_force(sq, sr, gen, train, 10, 10, M)
    assert r["s_sim"] == 20 and r["E"] == 32
    assert abs(r["theta"] - bf["theta"]) < 1e-12
    assert gen.mem_gb[list(gen.batch).index(r["B_g"])] + train.mem_gb[list(train.batch).index(r["B_t"])] <= M


def test_eq2_and_special_cases():
    assert O.theta(5.0, 7.0, 6.0) == (5.0, 5.0)          # simulator-bound rollout
    assert O.theta(9.0, 7.0, 6.0) == (7.0, 6.0)          # training-bound
    # a slow simulator caps rollout: everything beyond the minimum goes to training... unless training is slower
    q = [1, 100]
    gen = O.Profile(q, [1], [[10.0], [1000.0]], [0.0])
    train = O.Profile(q, [1], [[1.0], [100.0]], [0.0])
    r = O.elastic_allocation(8, 1, [0], [20.0], gen, train, 5, 5, 1.0)
    assert r["T_r"] <= 20.0 and r["theta"] == pytest.approx(min(r["T_r"], r["T_t"]))
    assert r["s_sim"] == 0 and r["s_g"] + r["s_t"] == 100
    # memory: the big batches do not fit
    gen2 = O.Profile(q, [1, 2], [[1.0, 50.0], [100.0, 5000.0]], [1.0, 100.0])
    r2 = O.elastic_allocation(8, 1, [0], [1e9], gen2, train, 5, 5, 2.0)
    assert r2["B_g"] == 1


@pytest.mark.parametrize("seed", range(20))
def test_library_makes_the_oracles_decisions(seed):
    rng = random.Random(100 + seed)
    g, t = _tables(rng, monotone=(seed % 3 != 0))       # also non-monotone tables: same steps, same answer
    sq = [0] if seed % 2 else [10, 25, 50]
    sr = [rng.uniform(20, 200)] if seed % 2 else sorted(rng.uniform(20, 200) for _ in range(3))
    M = rng.choice([25.0, 48.0, 100.0])
    want = O.elastic_allocation(128, 4, sq, sr, O.Profile(*g), O.Profile(*t), 8, 12, M)
    got = A.elastic_allocation(128, 4, sq, sr, g, t, 8, 12, M)
    for k in ("E", "s_sim", "s_g", "s_t", "B_g", "B_t", "iterations"):
        assert got[k] == want[k], k
    for k in ("T_s", "T_g", "T_t", "T_r", "theta"):
        assert abs(got[k] - want[k]) <= 1e-12 * max(1.0, abs(want[k])), k


def test_library_lookup_and_rejections():
    g, _ = _tables(random.Random(1))
    p, keep = A.make_profile(*g)
    op = O.Profile(*g)
    for s in (1, 20, 33, 40, 79, 80, 100):
        for j in range(4):
            assert abs(A.profile_rate(p, s, j) - op.at(s, j)) < 1e-12
    bad = ([40, 20], [1], [[1.0], [2.0]], [0.0])                           # unsorted grid
    ok = ([20, 40], [1], [[1.0], [2.0]], [0.0])
    assert A.elastic_allocation(8, 1, [0], [1.0], bad, ok, 5, 5, 1.0) is None
    assert A.elastic_allocation(8, 1, [0], [1.0], ok, ok, 60, 50, 1.0) is None   # empty quota interval
    assert A.elastic_allocation(8, 1, [0], [1.0], ok, ([20, 40], [1], [[1.0], [2.0]], [5.0]), 5, 5, 1.0) is None   # nothing fits
    assert A.elastic_allocation(0, 1, [0], [1.0], ok, ok, 5, 5, 1.0) is None


def test_rebalance_trigger():
    """20-step moving averages; fire when the gap exceeds 15 % of the faster stage for 20 steps in a row."""
    ro = [100.0] * 30 + [100.0] * 60
    tr = [95.0] * 30 + [70.0] * 60                       # balanced, then training falls behind
    want = O.rebalance_trigger(ro, tr)
    assert sum(want[:30]) == 0 and sum(want) >= 1
    first = want.index(1)
    # the averaged gap crosses 15 % a few steps after step 30 and must then persist for 20 steps
    assert 30 + 20 <= first + 1 <= 30 + 20 + 20
    r = A.Rebalance()
    got = [r.push(a, b) for a, b in zip(ro, tr)]
    assert got == want
    rng = random.Random(5)
    ro = [rng.uniform(50, 150) for _ in range(400)]
    tr = [rng.uniform(50, 150) * (0.6 if 100 < i < 250 else 1.0) for i in range(400)]
    r2 = A.Rebalance(window=10, streak=7, threshold=0.2)
    assert [r2.push(a, b) for a, b in zip(ro, tr)] == O.rebalance_trigger(ro, tr, 10, 7, 0.2)
    a, b, s = r2.averages()
    assert abs(a - sum(ro[-10:]) / 10) < 1e-9 and abs(b - sum(tr[-10:]) / 10) < 1e-9
