"""Sequences of a packed batch must not see each other's values.

A ragged last chunk is fetched as a whole 64-token TMA box, which also brings in the first
tokens of the next sequence.  Those rows only ever meet exact zeros in the products, which is
harmless for finite values and fatal for NaN / Inf (0 x NaN = NaN).  The kernels clear them in
shared memory; here non-finite values are planted in the first tokens of sequence 1 and
sequence 0 must come out bit-identical to the run with finite values there.
"""
import copy

import numpy as np
import pytest

import oracle
from gdn_inputs import make_cu_seqlens, make_state, make_tokens
from paper_2607_16831_b200 import harness

pytestmark = pytest.mark.gpu

BF16_NAN, BF16_INF = np.uint16(0x7FC0), np.uint16(0x7F80)


@pytest.fixture(autouse=True)
def chunked_path_only(monkeypatch):
    monkeypatch.setenv("GDN_PREFILL_SHORT_FALLBACK", "0")


def run(tok, lengths, init):
    return harness.run_prefill(dict(tokens=tok, cu_seqlens=make_cu_seqlens(lengths), initial_state=init))


def bits(a):
    return np.ascontiguousarray(a).view(np.uint64) if a.dtype == np.float64 else a


@pytest.mark.parametrize("lengths,Hqk,Hv", [([100, 70], 2, 4), ([1, 64], 1, 2), ([130, 5, 63], 2, 2),
                                            ([1100, 40], 1, 1)])   # the last one: sequence 0 runs as several runs of chunks
@pytest.mark.parametrize("field,poison", [("q", BF16_NAN), ("k", BF16_NAN), ("k", BF16_INF), ("v", BF16_NAN),
                                          ("v", BF16_INF), ("g", np.float32("nan")), ("g", np.float32("-inf")),
                                          ("beta", np.float32("nan")), ("beta", np.float32("inf"))])
def test_nonfinite_tokens_of_the_next_sequence_do_not_leak(lengths, Hqk, Hv, field, poison):
    T = int(np.sum(lengths))
    tok = make_tokens(T, Hqk, Hv, seed=3, gate_mean=4.0)
    init = make_state(len(lengths), Hv, seed=3)
    clean = run(tok, lengths, init)
    assert clean["device_status"] == 0

    bad = copy.deepcopy(tok)
    t1 = lengths[0]
    getattr(bad, field)[t1:t1 + min(8, lengths[1])] = poison   # the first tokens of sequence 1, every head
    res = run(bad, lengths, init)
    assert res["device_status"] == 0

    # sequence 0 (and every later sequence but 1): bit-identical to the clean run
    keep = np.ones(T, dtype=bool)
    keep[t1:t1 + lengths[1]] = False
    np.testing.assert_array_equal(bits(res["out"][keep]), bits(clean["out"][keep]))
    seqs = [n for n in range(len(lengths)) if n != 1]
    np.testing.assert_array_equal(bits(res["final_state"][seqs]), bits(clean["final_state"][seqs]))
    # and right: sequence 0 against the oracle on its own tokens
    ref_o, ref_s = oracle.prefill(tok.q[:t1], tok.k[:t1], tok.v[:t1], tok.g[:t1], tok.beta[:t1],
                                  make_cu_seqlens([t1]), init[:1])
    harness.assert_close(res["out"][:t1], ref_o, res["final_state"][:1], ref_s, "sequence 0 next to a poisoned sequence")
