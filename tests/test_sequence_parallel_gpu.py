"""The sequence-parallel building blocks (gdn_prefill_partial, gdn_state_scan, gdn_prefill_apply)
on the GPU against the fp64 oracle, and W emulated ranks run one after the other on one GPU
through the same host logic the multi-rank path uses (no process waits on another)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_16831_b200 as gdn
from gdn_inputs import make_cu_seqlens, make_state, make_tokens
from paper_2607_16831_b200 import harness
from paper_2607_16831_b200.sequence_parallel import CudaBackend, finish_piece, split_tokens

pytestmark = pytest.mark.gpu


def piece(tok, lo, hi):
    from gdn_inputs import Tokens

    return Tokens(q=tok.q[lo:hi], k=tok.k[lo:hi], v=tok.v[lo:hi], g=tok.g[lo:hi], beta=tok.beta[lo:hi],
                  Hqk=tok.Hqk, Hv=tok.Hv, dk=128, dv=128)


def test_partial_gives_zero_state_run_and_transition():
    lens = [200, 0, 65]
    Hqk, Hv = 2, 4
    tok = make_tokens(sum(lens), Hqk, Hv, seed=31, gate_mean=4.0)
    d = harness.to_device(tok)
    cu_np = make_cu_seqlens(lens)
    cu = torch.from_numpy(cu_np).cuda()
    T, N = tok.T, len(lens)
    out0 = torch.full((T, Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    qt = torch.full_like(out0, float("nan"))
    H = torch.full((N, Hv, 128, 128), float("nan"), dtype=torch.float32, device="cuda")
    P = torch.full_like(H, float("nan"))
    ws = harness.alloc_workspace(T, N, Hqk, Hv)
    gdn.gdn_prefill_partial(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, out0, qt, H, P, max(lens), ws)
    assert gdn.gdn_last_device_status(ws) == 0
    ref_o, ref_H = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, cu_np, None)
    eye = np.broadcast_to(np.eye(128, dtype=np.float32), (N, Hv, 128, 128)).copy()
    ref_qt, ref_P = oracle.prefill(tok.q, tok.k, np.zeros_like(tok.v), tok.g, tok.beta, cu_np, eye)
    harness.assert_close(harness.bf16_to_numpy(out0), ref_o, H.cpu().numpy().astype(np.float64), ref_H, "partial: zero-state run")
    harness.assert_close(harness.bf16_to_numpy(qt), ref_qt, P.cpu().numpy().astype(np.float64), ref_P, "partial: identity run")
    # the empty sequence: H = 0, P = I exactly
    assert torch.count_nonzero(H[1]).item() == 0
    assert torch.equal(P[1].cpu(), torch.from_numpy(eye[1]))


@pytest.mark.parametrize("steps,N,Hv", [(0, 1, 2), (1, 2, 4), (3, 1, 8), (7, 3, 2)])
def test_state_scan_matches_fp64_products(steps, N, Hv):
    rng = np.random.default_rng(steps * 10 + N)
    S0 = rng.standard_normal((N, Hv, 128, 128)).astype(np.float32)
    P = (rng.standard_normal((steps, N, Hv, 128, 128)) / np.sqrt(128)).astype(np.float32)
    H = rng.standard_normal((steps, N, Hv, 128, 128)).astype(np.float32)
    ref = S0.astype(np.float64)
    for i in range(steps):
        ref = ref @ P[i].astype(np.float64) + H[i]
    S_out = torch.full((N, Hv, 128, 128), float("nan"), dtype=torch.float32, device="cuda")
    gdn.gdn_state_scan(torch.from_numpy(S0).cuda(), torch.from_numpy(P).cuda() if steps else None,
                       torch.from_numpy(H).cuda() if steps else None, S_out)
    got = S_out.cpu().numpy().astype(np.float64)
    assert harness.rel_fro(got, ref) < 1e-6
    # from the zero state, in place of S0 = NULL
    if steps:
        S_out2 = torch.empty_like(S_out)
        gdn.gdn_state_scan(None, torch.from_numpy(P).cuda(), torch.from_numpy(H).cuda(), S_out2)
        ref0 = np.zeros_like(ref)
        for i in range(steps):
            ref0 = ref0 @ P[i].astype(np.float64) + H[i]
        assert harness.rel_fro(S_out2.cpu().numpy().astype(np.float64), ref0) < 1e-6


def test_apply_adds_state_times_carried_queries():
    lens = [130, 64, 1]
    Hv = 4
    T, N = sum(lens), len(lens)
    rng = np.random.default_rng(7)
    from gdn_inputs import bf16_bits_to_f32, f32_to_bf16_bits

    qt_bits = f32_to_bf16_bits(rng.standard_normal((T, Hv, 128)).astype(np.float32) * 0.1)
    o_bits = f32_to_bf16_bits(rng.standard_normal((T, Hv, 128)).astype(np.float32))
    S = rng.standard_normal((N, Hv, 128, 128)).astype(np.float32)
    cu_np = make_cu_seqlens(lens)
    qt = harness.bf16_to_device(qt_bits)
    out = harness.bf16_to_device(o_bits)
    ws = harness.alloc_workspace(T, N, Hv, Hv)
    gdn.gdn_prefill_apply(torch.from_numpy(S).cuda(), qt, out, torch.from_numpy(cu_np).cuda(), max(lens), ws)
    assert gdn.gdn_last_device_status(ws) == 0
    ref = bf16_bits_to_f32(o_bits).astype(np.float64)
    qf = bf16_bits_to_f32(qt_bits).astype(np.float64)
    for n in range(N):
        a, b = cu_np[n], cu_np[n + 1]
        ref[a:b] += np.einsum("hvk,thk->thv", S[n].astype(np.float64), qf[a:b])
    got = harness.bf16_to_numpy(out)
    # S enters the product as bf16, the sum is rounded to bf16: a few 1e-3 relative
    assert harness.rel_fro(got, ref) < 5e-3


@pytest.mark.parametrize("world", [2, 3, 4])
@pytest.mark.parametrize("T,gate_mean,initial", [(1000, 2.0, True), (1536, 6.0, True), (700, 5.0, False), (40, 5.0, True)])
def test_emulated_ranks_match_the_oracle(world, T, gate_mean, initial):
    """(T = 40 with several ranks: all pieces but the first are empty.)"""
    Hqk, Hv = 2, 4
    tok = make_tokens(T, Hqk, Hv, seed=T + world, gate_mean=gate_mean)
    init = make_state(1, Hv, seed=T) if initial else None
    spans = split_tokens(T, world)
    be = [CudaBackend() for _ in range(world)]
    parts = []
    for r, (lo, hi) in enumerate(spans):  # phase 1 on every "rank"
        d = harness.to_device(piece(tok, lo, hi))
        parts.append(be[r].partial(d["q"], d["k"], d["v"], d["g"], d["beta"]))
    P_all = [p[3] for p in parts]  # what the all_gather would deliver
    H_all = [p[2] for p in parts]
    S0 = None if init is None else torch.from_numpy(init).cuda()
    out = np.zeros((T, Hv, 128), dtype=np.float64)
    finals = []
    for r, (lo, hi) in enumerate(spans):  # phase 2 on every "rank"
        o, fin = finish_piece(be[r], r, S0, parts[r][0], parts[r][1], P_all, H_all)
        out[lo:hi] = harness.bf16_to_numpy(o)
        finals.append(fin.cpu().numpy().astype(np.float64))
    torch.cuda.synchronize()
    ref_o, ref_s = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, make_cu_seqlens([T]), init)
    for fin in finals:
        harness.assert_close(out, ref_o, fin, ref_s, "sequence-parallel, %d emulated ranks" % world)


def test_state_scan_with_no_steps_copies_the_state_every_time():
    """steps = 0 leaves the kernel's loop empty: the result must still be written (repeated, because the
    failure this guards against depended on what shared memory happened to hold)."""
    S0 = torch.randn((2, 3, 128, 128), dtype=torch.float32, device="cuda")
    for _ in range(50):
        S_out = torch.full_like(S0, float("nan"))
        gdn.gdn_state_scan(S0, None, None, S_out)
        assert torch.equal(S_out, S0)
    S_out = torch.full_like(S0, float("nan"))
    gdn.gdn_state_scan(None, None, None, S_out)
    assert torch.count_nonzero(S_out).item() == 0
