"""Token-serial prefill kernel against the fp64 CPU oracle."""
import numpy as np
import pytest

import oracle
from gdn_inputs import config, make_cu_seqlens, make_state, make_tokens
from paper_2607_16831_b200 import harness

pytestmark = pytest.mark.gpu


def check(cfg, what):
    res = harness.run_prefill(cfg, recurrent=True)
    ref_o, ref_s = oracle.prefill(*harness.token_arrays(cfg["tokens"]), cfg["cu_seqlens"], cfg["initial_state"])
    return harness.assert_close(res["out"], ref_o, res["final_state"], ref_s, what)


def test_recurrent_tiny():
    e = check(config("prefill_tiny"), "recurrent tiny")
    assert e["state_rel_fro"] < 1e-5


def test_recurrent_varlen_small():
    check(config("prefill_varlen", N=5, max_len=150, Hqk=2, Hv=4), "recurrent varlen")


def test_recurrent_zero_length_sequence():
    tok = make_tokens(70, 2, 4, seed=3)
    cfg = dict(tokens=tok, cu_seqlens=make_cu_seqlens([30, 0, 40]), initial_state=make_state(3, 4, seed=3), N=3)
    res = harness.run_prefill(cfg, recurrent=True)
    np.testing.assert_array_equal(res["final_state"][1], cfg["initial_state"][1].astype(np.float64))
    check(cfg, "recurrent zero-length")
