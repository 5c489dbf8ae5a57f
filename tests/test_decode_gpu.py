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
