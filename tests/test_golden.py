"""The frozen oracle answer on the smallest configuration (a drift detector for the
oracle and the input recipe; the paper itself prints no numerical example)."""
import os

import numpy as np

import oracle
from gdn_inputs import config

HERE = os.path.dirname(os.path.abspath(__file__))


def test_oracle_matches_frozen_values():
    cfg = config("prefill_tiny", seed=0)
    t = cfg["tokens"]
    out, fin = oracle.prefill(t.q, t.k, t.v, t.g, t.beta, cfg["cu_seqlens"], None)
    n = 0
    for line in open(os.path.join(HERE, "golden", "prefill_tiny_oracle.txt")):
        if line.startswith("#"):
            continue
        f = line.split()
        if f[0] == "out":
            got = out[int(f[1]), 0, int(f[2])]
        elif f[0] == "state":
            got = fin[0, 0, int(f[1]), int(f[2])]
        elif f[0] == "out_fro":
            got = np.linalg.norm(out)
        else:
            got = np.linalg.norm(fin)
        want = float(f[-1])
        assert abs(got - want) <= 1e-12 * max(1.0, abs(want)), line
        n += 1
    assert n == 13
