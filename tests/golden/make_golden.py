"""Writes tests/golden/prefill_tiny_oracle.txt from the CPU oracle alone.

The paper prints no worked numerical example, so there is no paper-given fixture to
store.  This file freezes the oracle's own answer on the smallest workload
configuration (1 sequence, 64 tokens, one head, d=128, seed 0) so that any later
change to the oracle's arithmetic or to the input recipe shows up as a diff.  It
calls only `oracle/` and `gdn_inputs/`; run it as `python tests/golden/make_golden.py`.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from gdn_inputs import config  # noqa: E402

ROWS = [(0, 0), (0, 127), (1, 5), (17, 64), (63, 0), (63, 127)]
STATE = [(0, 0), (3, 100), (64, 64), (127, 0), (127, 127)]


def compute():
    cfg = config("prefill_tiny", seed=0)
    t = cfg["tokens"]
    out, fin = oracle.prefill(t.q, t.k, t.v, t.g, t.beta, cfg["cu_seqlens"], None, threads=1)
    lines = ["# prefill_tiny, seed 0; fp64 oracle; '%r' round-trips exactly"]
    for (i, r) in ROWS:
        lines.append("out %d %d %r" % (i, r, float(out[i, 0, r])))
    for (r, c) in STATE:
        lines.append("state %d %d %r" % (r, c, float(fin[0, 0, r, c])))
    lines.append("out_fro %r" % float(np.linalg.norm(out)))
    lines.append("state_fro %r" % float(np.linalg.norm(fin)))
    return "\n".join(lines) + "\n"


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "prefill_tiny_oracle.txt")
    with open(path, "w") as f:
        f.write(compute())
    print("wrote", path)
