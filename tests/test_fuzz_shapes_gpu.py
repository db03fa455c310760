"""Seeded random model shapes through the C ABI against the fp64 oracle.

The fixed parity cases pick their shapes by hand; this file draws sixteen small models from a seeded
generator -- head_dim 32 / 64 / 128, 1..8 heads, 1..16 query tokens, 1..14 action dimensions, 1..3
layers, 1..4 Euler steps, MLP widths 1x / 2x / 4x, ragged prefixes, both dtypes, mixed step indices
-- so that every kernel family (tensor-core and plain-ALU projections, the three attention kernels,
embedding and head) meets shapes nobody chose for it.  Each case is compared element-wise with the
oracle within the dtype's tolerance, then re-run under a random SM quota and a random partition
into groups, which must reproduce the first result bit for bit.
"""
import numpy as np
import pytest

from paper_2609_27547_b200 import synth
from helpers import chunk_rel_err, oracle_run
from gpu_helpers import Runner, TOL, stack

pytestmark = pytest.mark.gpu


def _draw(case: int):
    rng = np.random.RandomState(7000 + case)
    hd = int(rng.choice([32, 64, 128]))
    heads = [n for n in (1, 2, 4, 8) if (hd * n) % 128 == 0 and hd * n <= 1024]
    n_heads = int(rng.choice(heads))
    lo = int(rng.randint(1, 41))
    w = synth.scaled(synth.WORKLOADS[0],
                     B=int(rng.randint(1, 15)), dtype=str(rng.choice(["f32", "bf16"])), H=int(rng.randint(1, 17)),
                     A=int(rng.randint(1, 15)), d=hd * n_heads, n_heads=n_heads, L=int(rng.randint(1, 4)),
                     K=int(rng.randint(1, 5)), P=(lo, lo + int(rng.randint(0, 121))), mixed_steps=bool(rng.randint(0, 2)),
                     mlp_mult=int(rng.choice([1, 2, 4])))
    return w, rng


@pytest.mark.parametrize("case", range(16))
def test_random_shape_against_the_oracle(case):
    w, rng = _draw(case)
    seed = synth.DEFAULT_SEED + case
    wt = synth.make_weights(w, seed, random_gains=True)
    envs = [synth.make_env(w, e, seed) for e in range(w.B)]
    ref = oracle_run(w, wt, envs)
    ids = list(range(w.B))
    r = Runner(w, wt, envs)
    got = stack(r.run([ids]), ids)
    err = chunk_rel_err(got, ref)
    assert err <= TOL[w.dtype], (w, err)
    # another quota, another partition, another arrival order: the same bits
    order = [int(x) for x in rng.permutation(w.B)]
    cuts = sorted(set(int(x) for x in rng.randint(1, w.B + 1, size=3)) | {w.B})
    groups, lo = [], 0
    for hi in cuts:
        if hi > lo:
            groups.append(order[lo:hi])
            lo = hi
    again = stack(r.run(groups, quota=int(rng.randint(1, 149))), ids)
    r.close()
    assert np.array_equal(again, got), (w, groups)
