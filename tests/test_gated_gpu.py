"""Entry points with the gate arithmetic fused in (raw a, b, A_log, dt_bias), against the fp64
oracle's raw-gate form on the same seeded inputs."""
import numpy as np
import pytest

import oracle
from gdn_inputs import config, make_cu_seqlens, make_raw_gates, make_state, make_tokens
from paper_2607_16831_b200 import harness

pytestmark = pytest.mark.gpu


def _dev(x):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


@pytest.mark.parametrize("B", [1, 5, 64])
def test_decode_gated_matches_oracle(B):
    import torch
    import paper_2607_16831_b200 as gdn
    cfg = config("decode_sweep", B=B, seed=B)
    tok = cfg["tokens"]
    a, b, A_log, dt_bias = make_raw_gates(B, tok.Hv, seed=B)
    d = harness.to_device(tok)
    s_in = _dev(cfg["state"])
    s_out = torch.full_like(s_in, float("nan"))
    out = torch.full((B, tok.Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    gdn.gdn_decode_gated(d["q"], d["k"], d["v"], _dev(a), _dev(b), _dev(A_log), _dev(dt_bias), s_in, s_out, out)
    torch.cuda.synchronize()
    ref_o, ref_s = oracle.decode_gated(tok.q, tok.k, tok.v, a, b, A_log, dt_bias, cfg["state"])
    e = harness.assert_close(harness.bf16_to_numpy(out), ref_o, s_out.cpu().numpy().astype(np.float64), ref_s,
                             "decode gated B=%d" % B)
    assert e["state_rel_fro"] < 2e-6


@pytest.mark.parametrize("lengths,Hqk,Hv", [([64], 1, 1), ([200, 1, 77], 2, 4), ([1024], 16, 32)])
def test_prefill_gated_matches_oracle(lengths, Hqk, Hv):
    import torch
    import paper_2607_16831_b200 as gdn
    T, N = int(np.sum(lengths)), len(lengths)
    tok = make_tokens(T, Hqk, Hv, seed=T)
    a, b, A_log, dt_bias = make_raw_gates(T, Hv, seed=T)
    init = make_state(N, Hv, seed=T)
    cu_np = make_cu_seqlens(lengths)
    d = harness.to_device(tok)
    out = torch.full((T, Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    fin = torch.full((N, Hv, 128, 128), float("nan"), dtype=torch.float32, device="cuda")
    ws = harness.alloc_workspace(T, N, Hqk, Hv)
    gdn.gdn_prefill_gated(d["q"], d["k"], d["v"], _dev(a), _dev(b), _dev(A_log), _dev(dt_bias), _dev(cu_np),
                          _dev(init), out, fin, int(max(lengths)), ws)
    torch.cuda.synchronize()
    assert gdn.gdn_last_device_status(ws) == 0
    ref_o, ref_s = oracle.prefill_gated(tok.q, tok.k, tok.v, a, b, A_log, dt_bias, cu_np, init)
    harness.assert_close(harness.bf16_to_numpy(out), ref_o, fin.cpu().numpy().astype(np.float64), ref_s,
                         "prefill gated %r" % (lengths,))


def test_gated_entry_points_reject_missing_gate_parameters():
    import torch
    import paper_2607_16831_b200 as gdn
    cfg = config("decode_sweep", B=1)
    tok = cfg["tokens"]
    a, b, A_log, dt_bias = make_raw_gates(1, tok.Hv)
    d = harness.to_device(tok)
    s = _dev(cfg["state"])
    out = torch.empty((1, tok.Hv, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gdn.GdnError) as err:
        gdn.gdn_decode_gated(d["q"], d["k"], d["v"], _dev(a), _dev(b), None, _dev(dt_bias), s, s, out)
    assert err.value.status == 1
