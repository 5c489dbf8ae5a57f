"""Entry points with the operator's whole front end fused in (raw gates, q/k L2 normalisation, scale on q)
against the fp64 oracle's fused form on the same seeded inputs.  q and k are rescaled per token by powers
of two (exact in bf16), so their norms are far from 1 and differ from token to token."""
import os

import numpy as np
import pytest

import oracle
from gdn_inputs import (bf16_bits_to_f32, config, f32_to_bf16_bits, make_cu_seqlens, make_raw_gates, make_state,
                        make_tokens)
from paper_2607_16831_b200 import harness

pytestmark = pytest.mark.gpu


def _dev(x):
    import torch
    return None if x is None else torch.from_numpy(np.ascontiguousarray(x)).cuda()


def unnormalised(tok, seed):
    """q, k bits with per-(token, head) norms spread over 2^-3 .. 2^3."""
    rng = np.random.default_rng(seed + 12345)
    T, Hqk = tok.q.shape[0], tok.q.shape[1]
    pk = (2.0 ** rng.integers(-3, 4, size=(T, Hqk, 1))).astype(np.float32)
    pq = (2.0 ** rng.integers(-1, 6, size=(T, Hqk, 1))).astype(np.float32)   # tok.q has norm 1/sqrt(128)
    return f32_to_bf16_bits(bf16_bits_to_f32(tok.q) * pq), f32_to_bf16_bits(bf16_bits_to_f32(tok.k) * pk)


def run_prefill_fused(lengths, Hqk, Hv, seed, raw, scale, l2norm, initial=True, **tok_kw):
    import torch
    import paper_2607_16831_b200 as gdn
    T, N = int(np.sum(lengths)), len(lengths)
    tok = make_tokens(T, Hqk, Hv, seed=seed, **tok_kw)
    qb, kb = unnormalised(tok, seed) if l2norm else (tok.q, tok.k)
    if raw:
        a, b, A_log, dt_bias = make_raw_gates(T, Hv, seed=seed)
    else:
        a, b, A_log, dt_bias = tok.g, tok.beta, None, None
    init = make_state(N, Hv, seed=seed) if initial else None
    cu_np = make_cu_seqlens(lengths)
    out = torch.full((T, Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    fin = torch.full((N, Hv, 128, 128), float("nan"), dtype=torch.float32, device="cuda")
    ws = harness.alloc_workspace(T, N, Hqk, Hv)
    gdn.gdn_prefill_fused(harness.bf16_to_device(qb), harness.bf16_to_device(kb), harness.bf16_to_device(tok.v),
                          _dev(a), _dev(b), _dev(A_log), _dev(dt_bias), _dev(cu_np), _dev(init), out, fin,
                          int(max(lengths)) if T else 0, ws, scale=scale, qk_l2norm=l2norm)
    torch.cuda.synchronize()
    assert gdn.gdn_last_device_status(ws) == 0
    ref_o, ref_s = oracle.prefill_fused(qb, kb, tok.v, a, b, A_log, dt_bias, cu_np, init, scale=scale,
                                        qk_l2norm=l2norm)
    return harness.bf16_to_numpy(out), ref_o, fin.cpu().numpy().astype(np.float64), ref_s


@pytest.mark.parametrize("B", [1, 5, 64])
@pytest.mark.parametrize("raw,scale,l2norm", [(True, 0.5, True), (False, 1.0, True), (False, 0.25, False)])
def test_decode_fused_matches_oracle(B, raw, scale, l2norm):
    import torch
    import paper_2607_16831_b200 as gdn
    cfg = config("decode_sweep", B=B, seed=B)
    tok = cfg["tokens"]
    qb, kb = unnormalised(tok, B) if l2norm else (tok.q, tok.k)
    if raw:
        a, b, A_log, dt_bias = make_raw_gates(B, tok.Hv, seed=B)
    else:
        a, b, A_log, dt_bias = tok.g, tok.beta, None, None
    s_in = _dev(cfg["state"])
    s_out = torch.full_like(s_in, float("nan"))
    out = torch.full((B, tok.Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    gdn.gdn_decode_fused(harness.bf16_to_device(qb), harness.bf16_to_device(kb), harness.bf16_to_device(tok.v), _dev(a),
                         _dev(b), _dev(A_log), _dev(dt_bias), s_in, s_out, out, scale=scale, qk_l2norm=l2norm)
    torch.cuda.synchronize()
    ref_o, ref_s = oracle.decode_fused(qb, kb, tok.v, a, b, A_log, dt_bias, cfg["state"], scale=scale, qk_l2norm=l2norm)
    e = harness.assert_close(harness.bf16_to_numpy(out), ref_o, s_out.cpu().numpy().astype(np.float64), ref_s,
                             "decode fused B=%d" % B)
    assert e["state_rel_fro"] < 2e-6


@pytest.mark.parametrize("B,T", [(1, 3), (6, 4), (40, 2)])
@pytest.mark.parametrize("raw,scale,l2norm", [(True, 0.5, True), (False, 0.25, False)])
def test_decode_multi_fused_matches_oracle(B, T, raw, scale, l2norm):
    """T tokens per item in one pass over the state, with the front end: the oracle's fused prefill over B
    sequences of length T from the same states."""
    import torch
    import paper_2607_16831_b200 as gdn
    Hqk, Hv = 4, 8
    tok = make_tokens(B * T, Hqk, Hv, seed=300 + B + T, gate_mean=3.0)
    qb, kb = unnormalised(tok, B + T) if l2norm else (tok.q, tok.k)
    if raw:
        a, b, A_log, dt_bias = make_raw_gates(B * T, Hv, seed=B + T)
    else:
        a, b, A_log, dt_bias = tok.g, tok.beta, None, None
    st = make_state(B, Hv, seed=300 + B)
    shp = lambda bits, H: harness.bf16_to_device(bits).view(B, T, H, 128)
    s_in = _dev(st)
    s_out = torch.full_like(s_in, float("nan"))
    out = torch.full((B, T, Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    gdn.gdn_decode_multi_fused(shp(qb, Hqk), shp(kb, Hqk), shp(tok.v, Hv), _dev(a).view(B, T, Hv), _dev(b).view(B, T, Hv),
                               _dev(A_log), _dev(dt_bias), s_in, s_out, out, scale=scale, qk_l2norm=l2norm)
    torch.cuda.synchronize()
    ref_o, ref_s = oracle.prefill_fused(qb, kb, tok.v, a, b, A_log, dt_bias, make_cu_seqlens([T] * B), st, scale=scale,
                                        qk_l2norm=l2norm)
    e = harness.assert_close(harness.bf16_to_numpy(out).reshape(B * T, Hv, 128), ref_o,
                             s_out.cpu().numpy().astype(np.float64), ref_s, "decode multi fused B=%d T=%d" % (B, T))
    assert e["state_rel_fro"] < 5e-6


CASES = [
    ([64], 1, 1, "one chunk"),
    ([200, 1, 77], 2, 4, "ragged chunks, three sequences"),
    ([1024], 16, 32, "full head count"),
    ([1024], 1, 3, "an unpaired value head"),
    ([2048], 4, 8, "split into 4 runs"),
    ([130, 0, 64, 63, 65, 700, 2, 90, 300, 31], 2, 4, "ten sequences (chunk-table kernel), one empty"),
]


@pytest.mark.parametrize("lengths,Hqk,Hv,what", CASES)
@pytest.mark.parametrize("raw,scale,l2norm", [(True, 0.5, True), (False, 1.0, True), (False, 0.25, False)])
def test_prefill_fused_matches_oracle(lengths, Hqk, Hv, what, raw, scale, l2norm):
    os.environ["GDN_PREFILL_SHORT_FALLBACK"] = "0"
    try:
        o, ro, s, rs = run_prefill_fused(lengths, Hqk, Hv, seed=len(lengths) * 100 + Hv, raw=raw, scale=scale,
                                         l2norm=l2norm, gate_mean=4.0)
    finally:
        del os.environ["GDN_PREFILL_SHORT_FALLBACK"]
    print(what, harness.assert_close(o, ro, s, rs, "prefill fused: " + what))


@pytest.mark.parametrize("lengths,Hqk,Hv", [([9], 1, 2), ([40, 3, 17, 33], 4, 8), ([5] * 40, 4, 8)])
def test_prefill_fused_short_sequences_take_the_token_serial_kernel(lengths, Hqk, Hv):
    """max_seqlen <= 64: the dispatch picks the token-serial kernel, which carries the same front end."""
    o, ro, s, rs = run_prefill_fused(lengths, Hqk, Hv, seed=77, raw=True, scale=0.5, l2norm=True)
    e = harness.assert_close(o, ro, s, rs, "prefill fused, token-serial")
    assert e["state_rel_fro"] < 1e-5   # fp32 recurrence: far tighter than the chunked path


def test_prefill_fused_weak_decay_correlated_keys():
    o, ro, s, rs = run_prefill_fused([1500], 4, 8, seed=5, raw=False, scale=0.7, l2norm=True, gate_mean=6.0,
                                     key_correlation=0.5)
    harness.assert_close(o, ro, s, rs, "prefill fused, correlated keys, weak decay")


def test_prefill_fused_zero_vectors_stay_zero():
    """A token whose k (or q) is all zeros: the normalised vector is zero, the state only decays at that token
    (its output is zero for a zero q); nothing turns into NaN."""
    import torch
    import paper_2607_16831_b200 as gdn
    T, Hqk, Hv = 192, 2, 4
    tok = make_tokens(T, Hqk, Hv, seed=9)
    qb, kb = unnormalised(tok, 9)
    qb[10] = 0; kb[10] = 0; kb[70, 1] = 0; qb[130, 0] = 0
    init = make_state(1, Hv, seed=9)
    cu_np = make_cu_seqlens([T])
    out = torch.full((T, Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    fin = torch.full((1, Hv, 128, 128), float("nan"), dtype=torch.float32, device="cuda")
    ws = harness.alloc_workspace(T, 1, Hqk, Hv)
    gdn.gdn_prefill_fused(harness.bf16_to_device(qb), harness.bf16_to_device(kb), harness.bf16_to_device(tok.v),
                          _dev(tok.g), _dev(tok.beta), None, None, _dev(cu_np), _dev(init), out, fin, T, ws,
                          scale=1.0, qk_l2norm=True)
    torch.cuda.synchronize()
    ref_o, ref_s = oracle.prefill_fused(qb, kb, tok.v, tok.g, tok.beta, None, None, cu_np, init, scale=1.0, qk_l2norm=True)
    o = harness.bf16_to_numpy(out)
    assert np.isfinite(o).all() and (o[10] == 0).all() and (o[130, :2] == 0).all()
    harness.assert_close(o, ref_o, fin.cpu().numpy().astype(np.float64), ref_s, "zero vectors")


def test_fused_switched_off_is_the_plain_entry_point_bit_for_bit():
    import torch
    import paper_2607_16831_b200 as gdn
    cfg = config("prefill_tiny", T=256, Hv=2)
    res = harness.run_prefill(cfg)
    tok = cfg["tokens"]
    d = harness.to_device(tok)
    T = tok.q.shape[0]
    out = torch.empty((T, tok.Hv, 128), dtype=torch.bfloat16, device="cuda")
    fin = torch.empty((1, tok.Hv, 128, 128), dtype=torch.float32, device="cuda")
    ws = harness.alloc_workspace(T, 1, tok.Hqk, tok.Hv)
    gdn.gdn_prefill_fused(d["q"], d["k"], d["v"], d["g"], d["beta"], None, None, _dev(cfg["cu_seqlens"]), None, out, fin,
                          T, ws, scale=1.0, qk_l2norm=False)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(harness.bf16_to_numpy(out), res["out"])
    np.testing.assert_array_equal(fin.cpu().numpy().astype(np.float64), res["final_state"])


def test_fused_entry_points_reject_bad_arguments():
    import torch
    import paper_2607_16831_b200 as gdn
    cfg = config("decode_sweep", B=1)
    tok = cfg["tokens"]
    a, b, A_log, dt_bias = make_raw_gates(1, tok.Hv)
    d = harness.to_device(tok)
    s = _dev(cfg["state"])
    out = torch.empty((1, tok.Hv, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gdn.GdnError) as err:   # exactly one of A_log, dt_bias
        gdn.gdn_decode_fused(d["q"], d["k"], d["v"], _dev(a), _dev(b), None, _dev(dt_bias), s, s, out)
    assert err.value.status == 1
    with pytest.raises(gdn.GdnError) as err:   # scale not finite
        gdn.gdn_decode_fused(d["q"], d["k"], d["v"], _dev(a), _dev(b), _dev(A_log), _dev(dt_bias), s, s, out,
                             scale=float("nan"))
    assert err.value.status == 2
