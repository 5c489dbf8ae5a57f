"""Seeded random shapes through the prefill entry points against the fp64 oracle: sequence counts, lengths
(empty, shorter than a chunk, ragged, several chunks, long enough to be split into runs), head groupings,
decay strengths, with and without an initial state, plain and fused front end.  Every case also runs twice
over differently filled scratch and must give the same bits."""
import numpy as np
import pytest

import oracle
from gdn_inputs import bf16_bits_to_f32, f32_to_bf16_bits, make_cu_seqlens, make_raw_gates, make_state, make_tokens
from paper_2607_16831_b200 import harness

pytestmark = pytest.mark.gpu


def draw_case(seed):
    rng = np.random.default_rng(1000 + seed)
    N = int(rng.choice([1, 1, 2, 3, 5, 9, 12]))
    Hqk, G = int(rng.choice([1, 2, 4])), int(rng.choice([1, 2, 2, 3, 4]))
    kind = int(rng.integers(0, 3))
    if kind == 0:
        lens = rng.integers(0, 200, size=N)
    elif kind == 1:
        lens = rng.integers(1, 900, size=N)
    else:
        lens = np.array([int(rng.choice([64, 128, 1024, 1, 63, 65, 1536, 512]))] * N)
    if int(lens.sum()) * Hqk * G > 40000:  # keep the oracle fast
        lens = np.maximum(lens // 4, (lens > 0).astype(lens.dtype))
    if lens.sum() == 0:
        lens[0] = 7
    return dict(lens=[int(x) for x in lens], Hqk=Hqk, Hv=Hqk * G, gate_mean=float(rng.choice([2.0, 5.0, 7.0, -2.0])),
                initial=bool(rng.random() < 0.7), fused=bool(rng.random() < 0.4), raw=bool(rng.random() < 0.5))


@pytest.mark.parametrize("seed", range(32))
def test_random_prefill_case_matches_oracle_and_is_deterministic(seed):
    import torch
    import paper_2607_16831_b200 as gdn
    c = draw_case(seed)
    lens, Hqk, Hv = c["lens"], c["Hqk"], c["Hv"]
    T, N = int(np.sum(lens)), len(lens)
    tok = make_tokens(T, Hqk, Hv, seed=seed, gate_mean=c["gate_mean"])
    init = make_state(N, Hv, seed=seed) if c["initial"] else None
    cu_np = make_cu_seqlens(lens)
    qb, kb = tok.q, tok.k
    scale, l2norm = 1.0, False
    a, b, A_log, dt_bias = tok.g, tok.beta, None, None
    if c["fused"]:
        rng = np.random.default_rng(seed)
        pw = (2.0 ** rng.integers(-2, 3, size=(T, Hqk, 1))).astype(np.float32)
        qb = f32_to_bf16_bits(bf16_bits_to_f32(tok.q) * pw * np.float32(8.0))
        kb = f32_to_bf16_bits(bf16_bits_to_f32(tok.k) * pw)
        scale, l2norm = 0.5, True
        if c["raw"]:
            a, b, A_log, dt_bias = make_raw_gates(T, Hv, seed=seed)
    dev = lambda x: None if x is None else torch.from_numpy(np.ascontiguousarray(x)).cuda()
    dq, dk, dv = harness.bf16_to_device(qb), harness.bf16_to_device(kb), harness.bf16_to_device(tok.v)
    da, db, dA, ddt, dcu, dinit = dev(a), dev(b), dev(A_log), dev(dt_bias), dev(cu_np), dev(init)
    got = []
    for fill in (0x00, 0xA5):
        ws = harness.alloc_workspace(T, N, Hqk, Hv)
        ws.fill_(fill)
        out = torch.full((T, Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
        fin = torch.full((N, Hv, 128, 128), float("nan"), dtype=torch.float32, device="cuda")
        if c["fused"]:
            gdn.gdn_prefill_fused(dq, dk, dv, da, db, dA, ddt, dcu, dinit, out, fin, int(max(lens)), ws, scale=scale,
                                  qk_l2norm=l2norm)
        else:
            gdn.gdn_prefill(dq, dk, dv, da, db, dcu, dinit, out, fin, int(max(lens)), ws)
        torch.cuda.synchronize()
        assert gdn.gdn_last_device_status(ws) == 0
        got.append((harness.bf16_to_numpy(out), fin.cpu().numpy().astype(np.float64)))
    np.testing.assert_array_equal(got[0][0], got[1][0])
    np.testing.assert_array_equal(got[0][1], got[1][1])
    if c["fused"]:
        ref_o, ref_s = oracle.prefill_fused(qb, kb, tok.v, a, b, A_log, dt_bias, cu_np, init, scale=scale, qk_l2norm=l2norm)
    else:
        ref_o, ref_s = oracle.prefill(qb, kb, tok.v, a, b, cu_np, init)
    harness.assert_close(got[0][0], ref_o, got[0][1], ref_s, "random case %d: %r" % (seed, c))
