"""Chunked (tcgen05/TMA) prefill parity against the fp64 CPU oracle, through the C ABI."""
import numpy as np
import pytest

import oracle
from gdn_inputs import config, make_cu_seqlens, make_state, make_tokens
from paper_2607_16831_b200 import harness

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def chunked_path_only(monkeypatch):
    """These tests are about the chunked kernels: keep gdn_prefill from handing the shortest
    shapes to the token-serial kernel (tests/test_prefill_dispatch_gpu.py covers that hand-over)."""
    monkeypatch.setenv("GDN_PREFILL_SHORT_FALLBACK", "0")


def check(cfg, what, **kw):
    res = harness.run_prefill(cfg, **kw)
    assert res["device_status"] == 0, "%s: a bounded device wait ran out" % what
    ref_o, ref_s = oracle.prefill(*harness.token_arrays(cfg["tokens"]), cfg["cu_seqlens"], cfg["initial_state"])
    e = harness.assert_close(res["out"], ref_o, res["final_state"], ref_s, what)
    print(what, e)
    return e


def custom(lengths, Hqk, Hv, seed, initial=True, **tok_kw):
    T = int(np.sum(lengths))
    tok = make_tokens(T, Hqk, Hv, seed=seed, **tok_kw)
    init = make_state(len(lengths), Hv, seed=seed) if initial else None
    return dict(kind="prefill", tokens=tok, cu_seqlens=make_cu_seqlens(lengths), initial_state=init, N=len(lengths))


def test_prefill_tiny_config():
    check(config("prefill_tiny"), "prefill tiny (1 x 64, 1 head)")


@pytest.mark.parametrize("T", [1, 63, 64, 65, 130])
def test_prefill_single_sequence_lengths(T):
    check(custom([T], 1, 2, seed=T), "prefill T=%d" % T)


def test_prefill_two_chunks_no_initial_state():
    check(custom([128], 2, 4, seed=5, initial=False), "prefill 128 zero-init")


def test_prefill_varlen_small_with_empty_sequence():
    cfg = custom([70, 0, 1, 200, 64], 2, 4, seed=7)
    res = harness.run_prefill(cfg)
    np.testing.assert_array_equal(res["final_state"][1], cfg["initial_state"][1].astype(np.float64))
    check(cfg, "prefill varlen small")


def test_prefill_weak_decay_carries_state_across_chunks():
    # mean log-gate ~ -0.0025: the initial state is still visible after 8 chunks
    e = check(custom([512], 2, 4, seed=11, gate_mean=6.0), "prefill weak decay")
    assert e["state_rel_fro"] < 2.5e-3


def test_prefill_matches_token_serial_kernel():
    cfg = custom([300, 77], 2, 4, seed=13)
    a = harness.run_prefill(cfg)
    b = harness.run_prefill(cfg, recurrent=True)
    assert harness.rel_fro(a["out"], b["out"]) < 8e-3
    assert harness.rel_fro(a["final_state"], b["final_state"]) < 5e-3


def test_prefill_final_state_not_requested():
    cfg = custom([100], 1, 1, seed=17)
    res = harness.run_prefill(cfg, want_final=False)
    ref_o, _ = oracle.prefill(*harness.token_arrays(cfg["tokens"]), cfg["cu_seqlens"], cfg["initial_state"])
    harness.assert_close(res["out"], ref_o, None, None, "prefill no final")


def test_prefill_split_invariance_through_state_handoff():
    """prefill(x[0:T]) == prefill(x[0:T1]) then prefill(x[T1:T]) from the returned state."""
    tok = make_tokens(200, 2, 4, seed=19, gate_mean=4.0)
    init = make_state(1, 4, seed=19)
    full = harness.run_prefill(dict(tokens=tok, cu_seqlens=make_cu_seqlens([200]), initial_state=init))
    T1 = 90
    from gdn_inputs import Tokens
    def part(a, b):
        return Tokens(q=tok.q[a:b], k=tok.k[a:b], v=tok.v[a:b], g=tok.g[a:b], beta=tok.beta[a:b], Hqk=2, Hv=4, dk=128, dv=128)
    r1 = harness.run_prefill(dict(tokens=part(0, T1), cu_seqlens=make_cu_seqlens([T1]), initial_state=init))
    r2 = harness.run_prefill(dict(tokens=part(T1, 200), cu_seqlens=make_cu_seqlens([200 - T1]),
                                  initial_state=r1["final_state"].astype(np.float32)))
    assert harness.rel_fro(np.concatenate([r1["out"], r2["out"]]), full["out"]) < 8e-3
    assert harness.rel_fro(r2["final_state"], full["final_state"]) < 5e-3


def test_prefill_long_config_both_initial_states():
    check(config("prefill_long"), "prefill long zero-init")
    check(config("prefill_long", initial=True), "prefill long with initial state")


def test_prefill_long_weak_decay():
    check(config("prefill_long", initial=True, gate_mean=6.0), "prefill long weak decay")


def test_prefill_varlen_config():
    check(config("prefill_varlen"), "prefill varlen 16 x U[1,2048]")


@pytest.mark.parametrize("Hqk,Hv", [(2, 2), (1, 4), (1, 3), (3, 6)])
def test_prefill_head_groupings(Hqk, Hv):
    """G = Hv/Hqk of 1, 4, 3 (odd: the last pair of value heads is half empty) and 2."""
    check(custom([90, 130], Hqk, Hv, seed=23 + Hv), "prefill heads %d/%d" % (Hqk, Hv))


def test_prefill_correlated_keys_stress():
    """Keys sharing a common direction make the intra-chunk triangular system far from the identity."""
    e = check(custom([256], 2, 4, seed=29, gate_mean=6.0, key_correlation=0.5), "prefill correlated keys")
    assert e["state_rel_fro"] < 4e-3


def test_prefill_final_state_may_alias_initial_state_and_guard_bands_stay_intact():
    import torch
    import paper_2607_16831_b200 as gdn

    cfg = custom([70, 33], 2, 4, seed=31)
    tok = cfg["tokens"]
    d = harness.to_device(tok)
    cu_np = np.asarray(cfg["cu_seqlens"], dtype=np.int32)
    cu = torch.from_numpy(cu_np).cuda()
    T, N, Hv = tok.T, 2, 4
    pad = 64  # canary rows around the outputs
    out_buf = torch.full((T + 2 * pad, Hv, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    st_buf = torch.full((N + 2, Hv, 128, 128), 7.0, dtype=torch.float32, device="cuda")
    st_buf[1:N + 1] = torch.from_numpy(cfg["initial_state"]).cuda()
    out, state = out_buf[pad:pad + T], st_buf[1:N + 1]
    ws = harness.alloc_workspace(T, N, tok.Hqk, Hv)
    gdn.gdn_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, state, out, state, int(np.max(np.diff(cu_np))), ws)
    torch.cuda.synchronize()
    assert gdn.gdn_last_device_status(ws) == 0
    ref_o, ref_s = oracle.prefill(*harness.token_arrays(tok), cfg["cu_seqlens"], cfg["initial_state"])
    harness.assert_close(harness.bf16_to_numpy(out), ref_o, state.cpu().numpy().astype(np.float64), ref_s, "in-place state")
    assert torch.all(out_buf[:pad] == 7.0) and torch.all(out_buf[pad + T:] == 7.0), "wrote outside `out`"
    assert torch.all(st_buf[0] == 7.0) and torch.all(st_buf[N + 1] == 7.0), "wrote outside `final_state`"


def test_prefill_workspace_errors_are_reported_before_any_launch():
    import torch
    import paper_2607_16831_b200 as gdn

    cfg = custom([64], 1, 1, seed=37)
    tok = cfg["tokens"]
    d = harness.to_device(tok)
    cu = torch.from_numpy(np.asarray(cfg["cu_seqlens"], dtype=np.int32)).cuda()
    out = torch.empty((64, 1, 128), dtype=torch.bfloat16, device="cuda")
    ws = harness.alloc_workspace(64, 1, 1, 1)
    for bad in (None, ws[: ws.numel() // 2], ws[16:]):  # missing, too small, misaligned
        with pytest.raises(gdn.GdnError) as err:
            gdn.gdn_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, None, out, None, 64, bad)
        assert err.value.status == 4


def test_prefill_malformed_cu_seqlens_stays_in_bounds():
    """Offsets beyond total_tokens are clamped on the device: results are unspecified but no
    access leaves the buffers (the canaries survive and the call completes)."""
    import torch
    import paper_2607_16831_b200 as gdn

    tok = make_tokens(100, 1, 2, seed=41)
    d = harness.to_device(tok)
    cu = torch.tensor([0, 60, 500], dtype=torch.int32, device="cuda")  # claims 500 tokens, only 100 exist
    out_buf = torch.full((100 + 128, 2, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    fin = torch.empty((2, 2, 128, 128), dtype=torch.float32, device="cuda")
    ws = harness.alloc_workspace(100, 2, 1, 2)
    gdn.gdn_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, None, out_buf[:100], fin, 100, ws)
    torch.cuda.synchronize()
    assert gdn.gdn_last_device_status(ws) == 0
    assert torch.all(out_buf[100:] == 7.0)
    assert torch.isfinite(fin).all()


@pytest.mark.parametrize("gate_mean", [-4.0, -12.0])
def test_prefill_strong_decay_underflows_cleanly(gate_mean):
    """g ~ -4 (-12) per token: every cumulative decay factor underflows inside a chunk; the decay
    differences are formed before the exponential, so nothing may overflow or turn into NaN."""
    cfg = custom([300, 64, 700], 2, 4, seed=43, gate_mean=gate_mean)
    check(cfg, "strong decay")
    res = harness.run_prefill(cfg)
    assert np.isfinite(res["out"]).all() and np.isfinite(res["final_state"]).all()


def test_prefill_all_sequences_empty_passes_states_through():
    from gdn_inputs import Tokens
    N, Hqk, Hv = 3, 2, 4
    empty = Tokens(q=np.zeros((0, Hqk, 128), np.uint16), k=np.zeros((0, Hqk, 128), np.uint16),
                   v=np.zeros((0, Hv, 128), np.uint16), g=np.zeros((0, Hv), np.float32),
                   beta=np.zeros((0, Hv), np.float32), Hqk=Hqk, Hv=Hv, dk=128, dv=128)
    init = make_state(N, Hv, seed=47)
    res = harness.run_prefill(dict(tokens=empty, cu_seqlens=make_cu_seqlens([0] * N), initial_state=init))
    np.testing.assert_array_equal(res["final_state"], init.astype(np.float64))
    res = harness.run_prefill(dict(tokens=empty, cu_seqlens=make_cu_seqlens([0] * N), initial_state=None))
    assert np.count_nonzero(res["final_state"]) == 0


def test_prefill_beta_zero_is_pure_decay_closed_form():
    """beta = 0: nothing is written, S_T = exp(sum g) S_0 and o_t = exp(gamma_t) S_0 q_t -- checked
    against that closed form in fp64, not against the oracle (T = 300 spans five chunks)."""
    from gdn_inputs import bf16_bits_to_f32
    T, Hqk, Hv = 300, 2, 4
    tok = make_tokens(T, Hqk, Hv, seed=53, gate_mean=4.0)
    tok.beta[:] = 0.0
    init = make_state(1, Hv, seed=53)
    res = harness.run_prefill(dict(tokens=tok, cu_seqlens=make_cu_seqlens([T]), initial_state=init))
    q = bf16_bits_to_f32(tok.q).astype(np.float64)
    gam = np.cumsum(tok.g.astype(np.float64), axis=0)  # [T, Hv]
    S0 = init[0].astype(np.float64)                    # [Hv, dv, dk]
    ref_o = np.stack([np.exp(gam[:, h])[:, None] * (q[:, h // 2, :] @ S0[h].T) for h in range(Hv)], axis=1)
    ref_s = np.exp(gam[-1])[:, None, None] * S0
    harness.assert_close(res["out"], ref_o, res["final_state"], ref_s[None], "beta = 0 closed form")


def test_prefill_onehot_keys_associative_recall():
    """g = 0, beta = 1, distinct one-hot keys: the state stores v_j in column j exactly, a query
    equal to an earlier key returns that value, a repeated key overwrites."""
    from gdn_inputs import Tokens, f32_to_bf16_bits, bf16_bits_to_f32
    T, Hv = 100, 2
    rng = np.random.default_rng(59)
    cols = np.concatenate([rng.permutation(128)[:90], rng.integers(0, 128, 10)])  # the last ten repeat keys
    k = np.zeros((T, 1, 128), np.float32)
    k[np.arange(T), 0, cols] = 1.0
    ask = np.array([cols[rng.integers(0, t + 1)] for t in range(T)])             # a key seen so far
    q = np.zeros((T, 1, 128), np.float32)
    q[np.arange(T), 0, ask] = 1.0
    v = rng.standard_normal((T, Hv, 128)).astype(np.float32)
    tok = Tokens(q=f32_to_bf16_bits(q), k=f32_to_bf16_bits(k), v=f32_to_bf16_bits(v), g=np.zeros((T, Hv), np.float32),
                 beta=np.ones((T, Hv), np.float32), Hqk=1, Hv=Hv, dk=128, dv=128)
    res = harness.run_prefill(dict(tokens=tok, cu_seqlens=make_cu_seqlens([T]), initial_state=None))
    vb = bf16_bits_to_f32(tok.v).astype(np.float64)
    ref_o = np.stack([vb[max(s for s in range(t + 1) if cols[s] == ask[t])] for t in range(T)])  # latest write wins
    ref_s = np.zeros((1, Hv, 128, 128))
    for c in range(128):
        writes = [s for s in range(T) if cols[s] == c]
        if writes:
            ref_s[0, :, :, c] = vb[writes[-1]]
    # the chunked path rounds its intermediate operands to bf16, so "exactly" means within the tolerances
    e = harness.assert_close(res["out"], ref_o, res["final_state"], ref_s, "one-hot recall")
    assert e["out_rel_fro"] < 5e-3 and e["state_rel_fro"] < 2e-3
    # the token-serial kernel keeps everything in fp32: there the recall is exact to bf16 rounding of the output
    rec = harness.run_prefill(dict(tokens=tok, cu_seqlens=make_cu_seqlens([T]), initial_state=None), recurrent=True)
    np.testing.assert_array_equal(rec["out"], ref_o)
    np.testing.assert_allclose(rec["final_state"], ref_s, rtol=0, atol=1e-6)


@pytest.mark.parametrize("lengths,Hqk,Hv", [([300, 0, 65], 2, 4), ([2048], 4, 8), ([70] * 12, 1, 2)])
def test_prefill_does_not_depend_on_what_the_workspace_and_outputs_held(lengths, Hqk, Hv):
    """Nothing is read before it is written: the same call over a workspace and output buffers filled with
    different garbage gives the same bits (a read of uninitialised scratch, or a result that is only
    partly written, shows up as a difference)."""
    import torch
    import paper_2607_16831_b200 as gdn
    from gdn_inputs import make_cu_seqlens, make_state, make_tokens
    T, N = int(np.sum(lengths)), len(lengths)
    tok = make_tokens(T, Hqk, Hv, seed=17, gate_mean=4.0)
    d = harness.to_device(tok)
    cu = torch.from_numpy(make_cu_seqlens(lengths)).cuda()
    init = torch.from_numpy(make_state(N, Hv, seed=17)).cuda()
    got = []
    for fill in (0x00, 0xFF, 0x5A):
        ws = harness.alloc_workspace(T, N, Hqk, Hv)
        ws.fill_(fill)
        out = torch.full((T, Hv, 128), 0, dtype=torch.int16, device="cuda").fill_(fill * 257 - 65536 * (fill > 127))
        fin = torch.empty((N, Hv, 128, 128), dtype=torch.float32, device="cuda").view(torch.int32).fill_(fill * 0x01010101 - (1 << 32) * (fill > 127)).view(torch.float32)
        gdn.gdn_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, init, out.view(torch.bfloat16), fin, int(max(lengths)), ws)
        torch.cuda.synchronize()
        assert gdn.gdn_last_device_status(ws) == 0
        got.append((out.cpu().numpy().copy(), fin.view(torch.int32).cpu().numpy().copy()))
    for o, f in got[1:]:
        np.testing.assert_array_equal(o, got[0][0])
        np.testing.assert_array_equal(f, got[0][1])


@pytest.mark.parametrize("persistent", ["0", "1"])
@pytest.mark.parametrize("lengths,Hqk,Hv", [([70, 0, 1, 200, 64, 129, 5, 300], 2, 4), ([64] * 40 + [1, 65], 1, 8),
                                            ([1100, 40, 700], 1, 2)])
def test_prefill_chain_kernel_forms_agree_with_the_oracle(monkeypatch, persistent, lengths, Hqk, Hv):
    """The chain kernel has two forms -- one thread block per chain, or persistent thread blocks that walk
    several chains each (what gdn_prefill picks for many short sequences).  Both are forced here on batches
    that mix empty, one-token, ragged and multi-chunk sequences (and, in the last case, sequences that are
    cut into runs), with more chains than the persistent form has thread blocks in the second case."""
    monkeypatch.setenv("GDN_PREFILL_PERSISTENT", persistent)
    check(custom(lengths, Hqk, Hv, seed=41, gate_mean=4.0), "prefill, persistent=%s, %d sequences" % (persistent, len(lengths)))
