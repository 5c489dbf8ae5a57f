"""Decode parity: the CUDA kernel (through the C ABI) against the fp64 CPU oracle,
element by element on the same seeded inputs."""
import numpy as np
import pytest

import oracle
from gdn_inputs import config
from paper_2607_16831_b200 import harness

pytestmark = pytest.mark.gpu


def check(cfg, **kw):
    res = harness.run_decode(cfg, **kw)
    ref_o, ref_s = oracle.decode(*harness.token_arrays(cfg["tokens"]), cfg["state"])
    e = harness.assert_close(res["out"], ref_o, res["state_out"], ref_s, "decode B=%d %r" % (cfg["B"], kw))
    # fp32 arithmetic on an fp32 state: far tighter than the acceptance bounds
    assert e["state_rel_fro"] < 1e-6, e
    assert e["out_rel_fro"] < 4e-3, e  # bf16 output rounding alone is ~1.7e-3
    return e


def test_decode_b64_full_config():
    check(config("decode_b64", B=64))


@pytest.mark.parametrize("B", [1, 8, 32, 128, 256])
def test_decode_batch_sweep(B):
    check(config("decode_sweep", B=B))


@pytest.mark.parametrize("B", [2, 3, 5])
def test_decode_ragged_batches_and_in_place(B):
    check(config("decode_sweep", B=B, seed=B))
    check(config("decode_sweep", B=B, seed=B), in_place=True)


def test_decode_all_launch_shapes_agree():
    import paper_2607_16831_b200 as gdn
    cfg = config("decode_sweep", B=3, seed=9)
    for variant in range(gdn.gdn_decode_num_variants()):
        check(cfg, variant=variant)


def test_decode_other_head_groupings():
    check(config("decode_sweep", B=2, Hqk=4, Hv=8))
    check(config("decode_sweep", B=2, Hqk=4, Hv=4))
    check(config("decode_sweep", B=2, Hqk=1, Hv=4))


def test_decode_layout_with_onehot_keys():
    """A transposed state layout cannot pass: key = e_5, so only column 5 of every row changes."""
    import torch
    cfg = config("decode_sweep", B=1, Hqk=1, Hv=1)
    tok = cfg["tokens"]
    tok.k[:] = 0
    tok.k[0, 0, 5] = 0x3F80  # bf16 1.0
    tok.g[:] = 0.0
    tok.beta[:] = 1.0
    res = harness.run_decode(cfg)
    s_in = cfg["state"][0, 0].astype(np.float64)
    v = harness.bf16_to_numpy(harness.bf16_to_device(tok.v))[0, 0]
    expect = s_in.copy()
    expect[:, 5] = v
    np.testing.assert_allclose(res["state_out"][0, 0], expect, rtol=0, atol=1e-7)


def test_decode_empty_batch_is_ok():
    import torch
    import paper_2607_16831_b200 as gdn
    e = torch.empty((0, 16, 128), dtype=torch.bfloat16, device="cuda")
    ev = torch.empty((0, 32, 128), dtype=torch.bfloat16, device="cuda")
    eg = torch.empty((0, 32), dtype=torch.float32, device="cuda")
    es = torch.empty((0, 32, 128, 128), dtype=torch.float32, device="cuda")
    gdn.gdn_decode(e, e, ev, eg, eg, es, es, ev)


def test_decode_guard_bands_stay_intact():
    import torch
    import paper_2607_16831_b200 as gdn
    cfg = config("decode_sweep", B=3, seed=21)
    tok = cfg["tokens"]
    d = harness.to_device(tok)
    s_in = torch.from_numpy(cfg["state"]).cuda()
    so_buf = torch.full((5, 32, 128, 128), 7.0, dtype=torch.float32, device="cuda")
    o_buf = torch.full((5, 32, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    gdn.gdn_decode(d["q"], d["k"], d["v"], d["g"], d["beta"], s_in, so_buf[1:4], o_buf[1:4])
    torch.cuda.synchronize()
    assert torch.all(so_buf[0] == 7.0) and torch.all(so_buf[4] == 7.0)
    assert torch.all(o_buf[0] == 7.0) and torch.all(o_buf[4] == 7.0)
    ref_o, ref_s = oracle.decode(*harness.token_arrays(tok), cfg["state"])
    harness.assert_close(harness.bf16_to_numpy(o_buf[1:4]), ref_o, so_buf[1:4].cpu().numpy().astype(np.float64), ref_s, "decode guard")


def test_decode_then_prefill_state_handoff():
    """T decode calls from a state == one prefill of the same T tokens from that state."""
    import torch
    import paper_2607_16831_b200 as gdn
    from gdn_inputs import make_cu_seqlens, make_state, make_tokens
    T, Hqk, Hv = 9, 2, 4
    tok = make_tokens(T, Hqk, Hv, seed=25, gate_mean=4.0)
    init = make_state(1, Hv, seed=25)
    pre = harness.run_prefill(dict(tokens=tok, cu_seqlens=make_cu_seqlens([T]), initial_state=init))
    d = harness.to_device(tok)
    s = torch.from_numpy(init).cuda()
    outs = []
    for t in range(T):
        o = torch.empty((1, Hv, 128), dtype=torch.bfloat16, device="cuda")
        gdn.gdn_decode(d["q"][t:t + 1], d["k"][t:t + 1], d["v"][t:t + 1], d["g"][t:t + 1], d["beta"][t:t + 1], s, s, o)
        outs.append(harness.bf16_to_numpy(o))
    torch.cuda.synchronize()
    dec_out = np.concatenate(outs, axis=0)
    assert harness.rel_fro(dec_out, pre["out"]) < 8e-3
    assert harness.rel_fro(s.cpu().numpy().astype(np.float64), pre["final_state"]) < 5e-3


@pytest.mark.parametrize("B,T", [(1, 2), (3, 4), (64, 3), (2, 0)])
def test_decode_multi_token(B, T):
    """T tokens per item in one state pass == the oracle run over B sequences of length T."""
    import torch
    import paper_2607_16831_b200 as gdn
    from gdn_inputs import make_cu_seqlens, make_state, make_tokens
    Hqk, Hv = 16, 32
    tok = make_tokens(B * T, Hqk, Hv, seed=100 + B + T, gate_mean=3.0)
    st = make_state(B, Hv, seed=100 + B)
    d = harness.to_device(tok)
    shp = lambda x, H: x.view(B, T, H, 128)
    s_in = torch.from_numpy(st).cuda()
    s_out = torch.full_like(s_in, float("nan"))
    out = torch.full((B, T, Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    gdn.gdn_decode_multi(shp(d["q"], Hqk), shp(d["k"], Hqk), shp(d["v"], Hv), d["g"].view(B, T, Hv),
                         d["beta"].view(B, T, Hv), s_in, s_out, out)
    torch.cuda.synchronize()
    ref_o, ref_s = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, make_cu_seqlens([T] * B), st)
    got_o = harness.bf16_to_numpy(out).reshape(B * T, Hv, 128)
    e = harness.assert_close(got_o, ref_o, s_out.cpu().numpy().astype(np.float64), ref_s, "decode multi B=%d T=%d" % (B, T))
    assert e["state_rel_fro"] < 2e-6


@pytest.mark.parametrize("B,slices,streams", [(5, 3, 2), (16, 8, 3), (2, 8, 3)])
def test_decode_from_host_buffers_in_slices(B, slices, streams):
    """host_pipeline.HostDecode: pinned host buffers in, slices of the batch on several streams,
    pinned host buffers out; then a second step on the state kept on the device."""
    import torch
    from gdn_inputs import config
    from paper_2607_16831_b200.host_pipeline import HostDecode

    cfg = config("decode_sweep", B=B)
    tok, st = cfg["tokens"], cfg["state"]
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h = [pin(tok.q.view(np.int16)), pin(tok.k.view(np.int16)), pin(tok.v.view(np.int16)), pin(tok.g), pin(tok.beta)]
    h_state = pin(st)
    h_out = torch.full((B, tok.Hv, 128), -1, dtype=torch.int16).pin_memory()
    h_state_out = torch.full_like(h_state, float("nan")).pin_memory()
    pipe = HostDecode(B, tok.Hqk, tok.Hv, slices=slices, streams=streams)
    pipe.step(*h, h_state, h_state_out, h_out)
    torch.cuda.synchronize()
    ref_o, ref_s = oracle.decode(*harness.token_arrays(tok), st)
    got_o = harness.bf16_to_numpy(h_out.view(torch.bfloat16))
    harness.assert_close(got_o, ref_o, h_state_out.numpy().astype(np.float64), ref_s, "host decode B=%d" % B)
    # second step from the state that stayed on the device == oracle from the first step's state
    pipe.swap()
    pipe.step(*h, None, h_state_out, h_out)
    torch.cuda.synchronize()
    ref_o2, ref_s2 = oracle.decode(*harness.token_arrays(tok), ref_s.astype(np.float32))
    harness.assert_close(harness.bf16_to_numpy(h_out.view(torch.bfloat16)), ref_o2,
                         h_state_out.numpy().astype(np.float64), ref_s2, "host decode, second step")


@pytest.mark.parametrize("B,slices,streams", [(12, 4, 2), (7, 8, 3), (3, 1, 1)])
def test_host_decode_steps_enqueued_back_to_back(B, slices, streams):
    """Five steps with different inputs enqueued without synchronising in between (they overlap on the device:
    one step's copies back run while the next step's inputs come in), each with its own host output buffers;
    every step must match the oracle on its own inputs: the reuse of the device buffers is ordered."""
    import torch
    from gdn_inputs import config
    from paper_2607_16831_b200.host_pipeline import HostDecode

    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    steps = []
    for s in range(5):
        cfg = config("decode_sweep", B=B, seed=40 + s)
        tok, st = cfg["tokens"], cfg["state"]
        steps.append(dict(tok=tok, st=st,
                          h=[pin(tok.q.view(np.int16)), pin(tok.k.view(np.int16)), pin(tok.v.view(np.int16)), pin(tok.g),
                             pin(tok.beta)],
                          h_state=pin(st),
                          h_out=torch.full((B, tok.Hv, 128), -1, dtype=torch.int16).pin_memory(),
                          h_state_out=torch.full((B, tok.Hv, 128, 128), float("nan"), dtype=torch.float32).pin_memory()))
    pipe = HostDecode(B, steps[0]["tok"].Hqk, steps[0]["tok"].Hv, slices=slices, streams=streams)
    for x in steps:
        pipe.step(*x["h"], x["h_state"], x["h_state_out"], x["h_out"])
    torch.cuda.current_stream().synchronize()  # the caller's stream waits for every step's last copy
    for s, x in enumerate(steps):
        ref_o, ref_s = oracle.decode(*harness.token_arrays(x["tok"]), x["st"])
        harness.assert_close(harness.bf16_to_numpy(x["h_out"].view(torch.bfloat16)), ref_o,
                             x["h_state_out"].numpy().astype(np.float64), ref_s, "host decode, step %d of 5" % s)
