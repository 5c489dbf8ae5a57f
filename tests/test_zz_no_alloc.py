"""gdn_prefill_static -- the prefill entry point for callers that may not allocate device
memory (its scratch is a fixed array inside the library) -- must give what the recurrence gives,
what gdn_prefill gives, and must not allocate.

Collected last on purpose (the file name sorts after every other test file): a run that stops
at the first failure has then already exercised everything else.  The test is self-contained,
so it also passes when run alone in a fresh process, where its first call is the one that
looks up the scratch address on the device.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _run_both(lengths, Hqk, Hv, seed):
    import torch

    import oracle
    import paper_2607_16831_b200 as gdn
    from gdn_inputs import make_cu_seqlens, make_state, make_tokens
    from paper_2607_16831_b200 import harness

    T = int(np.sum(lengths))
    tok = make_tokens(T, Hqk, Hv, seed=seed, gate_mean=4.0)
    d = harness.to_device(tok)
    cu_np = make_cu_seqlens(lengths)
    cu = torch.from_numpy(cu_np).cuda()
    N = len(lengths)
    init_np = make_state(N, Hv, seed=seed)
    init = torch.from_numpy(init_np).cuda()
    max_len = int(max(lengths))
    assert gdn.gdn_prefill_workspace_bytes(T, N, Hqk, Hv) <= gdn.PREFILL_STATIC_SCRATCH_BYTES

    def fresh():
        return (torch.full((T, Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda"),
                torch.full((N, Hv, 128, 128), float("nan"), dtype=torch.float32, device="cuda"))

    out_a, fin_a = fresh()
    ws = harness.alloc_workspace(T, N, Hqk, Hv)
    gdn.gdn_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, init, out_a, fin_a, max_len, ws)
    out_b, fin_b = fresh()
    out_c, fin_c = fresh()
    # warm-up call: on a fresh process this is the one that looks up the scratch address
    gdn.gdn_prefill_static(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, init, out_c, fin_c, max_len)
    torch.cuda.synchronize()
    # the measured call: neither the driver's free-memory figure nor torch's allocator may move
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    gdn.gdn_prefill_static(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, init, out_b, fin_b, max_len)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "gdn_prefill_static changed the device's free memory by %d bytes" % (free0 - free1)
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    # no bounded wait ran out in the static scratch (None = that scratch's status word)
    assert gdn.gdn_last_device_status(None) == 0
    ref_o, ref_s = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, cu_np, init_np)
    return (harness.bf16_to_numpy(out_a), fin_a.cpu().numpy().astype(np.float64),
            harness.bf16_to_numpy(out_b), fin_b.cpu().numpy().astype(np.float64), ref_o, ref_s)


def test_static_scratch_prefill_matches_oracle_and_workspace_prefill_twice_in_a_row():
    from paper_2607_16831_b200 import harness

    # two problems in a row: the second finds the first one's leftovers in the shared scratch and
    # must not be affected by them
    for lengths, Hqk, Hv, seed in (([100, 64, 30], 2, 4, 1), ([17, 200], 1, 2, 2)):
        out_a, fin_a, out_b, fin_b, ref_o, ref_s = _run_both(lengths, Hqk, Hv, seed)
        # against the fp64 oracle, at the tolerances of every other parity test
        e = harness.assert_close(out_b, ref_o, fin_b, ref_s, "static-scratch prefill vs oracle")
        assert e["out_nan"] == 0 and e["state_nan"] == 0
        # against the entry point with a caller workspace (same kernels, same inputs)
        e = harness.assert_close(out_b, out_a, fin_b, fin_a, "static-scratch prefill vs workspace prefill")
        assert e["out_max_abs"] <= harness.OUT_MAX_ABS and e["out_rel_fro"] <= harness.OUT_REL_FRO
        assert e["state_rel_fro"] <= harness.STATE_REL_FRO


def test_static_scratch_prefill_refuses_oversized_problems():
    import torch

    import paper_2607_16831_b200 as gdn

    T, Hqk, Hv = 4096, 16, 32  # needs ~85 MB of workspace: more than the fixed scratch
    assert gdn.gdn_prefill_workspace_bytes(T, 1, Hqk, Hv) > gdn.PREFILL_STATIC_SCRATCH_BYTES
    q = torch.zeros((T, Hqk, 128), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros((T, Hv, 128), dtype=torch.bfloat16, device="cuda")
    gb = torch.zeros((T, Hv), dtype=torch.float32, device="cuda")
    cu = torch.tensor([0, T], dtype=torch.int32, device="cuda")
    out = torch.empty_like(v)
    with pytest.raises(gdn.GdnError) as err:
        gdn.gdn_prefill_static(q, q, v, gb, gb, cu, None, out, None, T)
    assert err.value.status == 4  # GDN_ERR_WORKSPACE


def test_static_scratch_status_word_is_readable():
    """The scratch's address is private to the library; gdn_last_device_status(None) reads its status word
    (a static call comes first, so the test also stands alone in a fresh process)."""
    import paper_2607_16831_b200 as gdn

    _run_both([70], 1, 1, 3)
    assert gdn.gdn_last_device_status(None) == 0
