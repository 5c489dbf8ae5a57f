"""Sequence-parallel prefill (runs of chunks advanced side by side, joined by the scan over
chunk-run transitions) against the fp64 CPU oracle, through the C ABI.

The library picks the number of runs from (sequences x value heads) and the longest sequence, so
the shapes below are what selects 2, 3, 4, 5 and 8 runs; GDN_PREFILL_MAX_SEGMENTS=1 switches the
split off for the A/B comparison."""
import os

import numpy as np
import pytest

import oracle
from gdn_inputs import config, make_cu_seqlens, make_state, make_tokens
from paper_2607_16831_b200 import harness

pytestmark = pytest.mark.gpu


def custom(lengths, Hqk, Hv, seed, initial=True, **tok_kw):
    T = int(np.sum(lengths))
    tok = make_tokens(T, Hqk, Hv, seed=seed, **tok_kw)
    init = make_state(len(lengths), Hv, seed=seed) if initial else None
    return dict(kind="prefill", tokens=tok, cu_seqlens=make_cu_seqlens(lengths), initial_state=init, N=len(lengths))


def check(cfg, what, **kw):
    res = harness.run_prefill(cfg, **kw)
    assert res["device_status"] == 0, "%s: a bounded device wait ran out" % what
    ref_o, ref_s = oracle.prefill(*harness.token_arrays(cfg["tokens"]), cfg["cu_seqlens"], cfg["initial_state"])
    e = harness.assert_close(res["out"], ref_o, res["final_state"] if kw.get("want_final", True) else None,
                             ref_s if kw.get("want_final", True) else None, what)
    print(what, e)
    return e, res


# (lengths, Hqk, Hv): runs chosen = min((148 / (N Hv) + 1) / 2, 8, chunks of the longest sequence / 8)
SHAPES = [
    ([1024], 4, 8, "16 chunks -> 2 runs"),
    ([2048], 4, 8, "32 chunks -> 4 runs"),
    ([4096], 4, 8, "64 chunks -> 8 runs"),
    ([2000], 4, 8, "ragged tail, 32 chunks -> 4 runs of 8"),
    ([2434], 2, 4, "39 chunks -> 4 runs (10, 10, 10, 9), ragged"),
    ([2200], 8, 16, "35 chunks, 16 heads -> 4 runs (9, 9, 9, 8)"),
    ([3000, 1400], 4, 8, "two sequences -> 5 runs each; the short one has runs of 5, 5, 5, 5, 2 chunks"),
    ([1800, 0, 64], 2, 4, "an empty sequence and a one-chunk sequence beside one split into 3 runs"),
    ([1024], 8, 8, "one value head per key head"),
    ([1024], 2, 8, "four value heads per key head"),
    ([1024], 1, 3, "three value heads on one key head (an unpaired head in the intra-chunk kernel)"),
]


@pytest.mark.parametrize("lengths,Hqk,Hv,what", SHAPES)
@pytest.mark.parametrize("gate_mean", [2.0, 6.0])
def test_split_prefill_matches_oracle(lengths, Hqk, Hv, what, gate_mean):
    # gate_mean 6 (weak decay): the state entering a run matters for all of its tokens
    check(custom(lengths, Hqk, Hv, seed=len(lengths) * 1000 + lengths[0], gate_mean=gate_mean), what)


def test_split_prefill_zero_initial_state_and_no_final_state():
    cfg = custom([2048], 4, 8, seed=3, initial=False, gate_mean=5.0)
    check(cfg, "zero initial state, 4 runs")
    check(cfg, "final state not requested, 4 runs", want_final=False)
    cfg2 = custom([1024], 4, 8, seed=4, gate_mean=5.0)
    check(cfg2, "final state not requested, 2 runs", want_final=False)


def test_split_prefill_full_size_long_sequence():
    """The T=4096, 16/32-head workload takes the two-run path."""
    check(config("prefill_long", initial=True, gate_mean=5.0), "prefill_long weak decay, 2 runs")


def test_split_and_unsplit_agree():
    cfg = custom([2048], 4, 8, seed=21, gate_mean=6.0)
    _, a = check(cfg, "4 runs")
    os.environ["GDN_PREFILL_MAX_SEGMENTS"] = "1"
    try:
        _, b = check(cfg, "1 run")
    finally:
        del os.environ["GDN_PREFILL_MAX_SEGMENTS"]
    assert harness.rel_fro(a["out"], b["out"]) < 8e-3
    assert harness.rel_fro(a["final_state"], b["final_state"]) < 5e-3
    # the two paths round differently; identical bits would mean the split was not taken
    assert not np.array_equal(a["out"], b["out"])


def test_split_prefill_correlated_keys():
    """Keys sharing a common direction: transitions far from a multiple of the identity."""
    check(custom([2048], 4, 8, seed=23, gate_mean=6.0, key_correlation=0.5), "correlated keys, 4 runs")


def test_split_prefill_repeated_calls_reuse_workspace():
    cfg = custom([1024], 4, 8, seed=29, gate_mean=4.0)
    _, a = check(cfg, "first call")
    _, b = check(cfg, "second call")
    np.testing.assert_array_equal(a["out"], b["out"])
    np.testing.assert_array_equal(a["final_state"], b["final_state"])


@pytest.mark.parametrize("gate_mean", [-4.0, -12.0])
def test_split_prefill_strong_decay_underflows_cleanly(gate_mean):
    """g ~ -4 (-12) per token: cumulative decays underflow to zero inside a chunk, the transition of a
    run is exactly zero, and nothing may turn into NaN or Inf on the way."""
    cfg = custom([2048], 4, 8, seed=37, gate_mean=gate_mean)
    _, res = check(cfg, "strong decay, 4 runs")
    assert np.isfinite(res["out"]).all() and np.isfinite(res["final_state"]).all()


def test_split_prefill_long_ragged_sequence():
    """20,001 tokens at 2/4 heads: 313 chunks in 8 runs of 40 (the last one 33 with a one-token tail)."""
    check(custom([20001], 2, 4, seed=41, gate_mean=5.0), "long ragged sequence, 8 runs")


def test_split_prefill_quarter_million_tokens():
    """262,161 tokens at 2/4 heads (4097 chunks, a 1 GB workspace, 8 runs of 513 chunks with a 17-token tail):
    offsets beyond 32 bits in bytes, long chains, weak decay so that the state is carried all the way."""
    check(custom([262144 + 17], 2, 4, seed=43, gate_mean=5.0), "quarter of a million tokens, 8 runs")
