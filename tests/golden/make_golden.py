"""Writes the stored oracle outputs under tests/golden/.  Calls only the oracle (and the seeded
input generator); never the CUDA path.

    python tests/golden/make_golden.py

oracle_cfg0_first4.txt: the tiny fp32 configuration (16 envs, H=8, A=7, d=256, L=2, 4 heads,
P=32, K=4), default seed, environments 0..3, final action chunks in fp64, one row per
(environment, action token).  The paper prints no worked example; this file is a regression
fixture for the oracle, not a pin of it.
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
sys.path.insert(0, os.path.dirname(HERE))

from paper_2609_27547_b200 import synth  # noqa: E402
from helpers import oracle_run  # noqa: E402


def main():
    w = synth.WORKLOADS[0]
    wt = synth.make_weights(w, synth.DEFAULT_SEED)
    envs = [synth.make_env(w, e, synth.DEFAULT_SEED) for e in range(4)]
    out = oracle_run(w, wt, envs)
    np.savetxt(os.path.join(HERE, "oracle_cfg0_first4.txt"), out.reshape(-1, w.A), fmt="%.17e",
               header="oracle a_K, cfg0 tiny fp32, seed %d, envs 0..3, rows = (env, token)" % synth.DEFAULT_SEED)


if __name__ == "__main__":
    main()
