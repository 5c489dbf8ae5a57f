"""gdn_prefill's short-sequence dispatch: when no sequence is longer than one chunk and the
token-serial kernel is the faster one by the library's cost model, gdn_prefill runs it instead of
the chunked kernels.  Either way the result must match the fp64 oracle."""
import numpy as np
import pytest

import oracle
from gdn_inputs import make_cu_seqlens, make_state, make_tokens
from paper_2607_16831_b200 import harness

pytestmark = pytest.mark.gpu


def custom(lengths, Hqk, Hv, seed):
    T = int(np.sum(lengths))
    tok = make_tokens(T, Hqk, Hv, seed=seed)
    return dict(kind="prefill", tokens=tok, cu_seqlens=make_cu_seqlens(lengths),
                initial_state=make_state(len(lengths), Hv, seed=seed), N=len(lengths))


def oracle_check(cfg, res, what):
    assert res["device_status"] == 0
    ref_o, ref_s = oracle.prefill(*harness.token_arrays(cfg["tokens"]), cfg["cu_seqlens"], cfg["initial_state"])
    return harness.assert_close(res["out"], ref_o, res["final_state"], ref_s, what)


# (lengths, Hqk, Hv, token-serial expected by the cost model)
CASES = [
    ([4], 4, 8, True),
    ([16, 3, 9, 1], 4, 8, True),
    ([32], 4, 8, True),
    ([64], 4, 8, False),            # one full chunk: the chunked kernels win
    ([8] * 64, 4, 8, True),         # many tiny sequences
    ([32] * 64, 4, 8, False),       # many sequences of half a chunk: several waves of the serial kernel
    ([65, 3], 4, 8, False),         # anything longer than a chunk stays chunked
    ([5, 0, 7], 2, 4, True),        # with an empty sequence
]


@pytest.mark.parametrize("lengths,Hqk,Hv,serial", CASES)
def test_short_sequence_dispatch(lengths, Hqk, Hv, serial, monkeypatch):
    cfg = custom(lengths, Hqk, Hv, seed=len(lengths) + lengths[0])
    auto = harness.run_prefill(cfg)
    oracle_check(cfg, auto, "gdn_prefill (dispatching) %s" % (lengths[:4],))
    rec = harness.run_prefill(cfg, recurrent=True)
    monkeypatch.setenv("GDN_PREFILL_SHORT_FALLBACK", "0")
    chunked = harness.run_prefill(cfg)
    oracle_check(cfg, chunked, "gdn_prefill (chunked only) %s" % (lengths[:4],))
    same_as_serial = np.array_equal(auto["out"], rec["out"]) and np.array_equal(auto["final_state"], rec["final_state"])
    same_as_chunked = np.array_equal(auto["out"], chunked["out"]) and np.array_equal(auto["final_state"], chunked["final_state"])
    # the two kernels round differently, so bit equality tells which one ran
    assert same_as_serial == serial, "expected the %s path" % ("token-serial" if serial else "chunked")
    assert same_as_chunked == (not serial)
