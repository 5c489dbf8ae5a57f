"""The C-ABI library: loads without a GPU, exports every symbol the header declares, and
rejects bad arguments on the host before touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def gdn():
    from paper_2607_16831_b200 import build
    build.build()
    import paper_2607_16831_b200 as g
    return g


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gdn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gdn_[a-z_0-9]+)\s*\(", text)))


def test_header_and_binding_agree(gdn):
    names = declared_functions()
    assert sorted(gdn.EXPORTS) == names
    L = gdn.lib()
    for n in names:
        assert getattr(L, n) is not None


def test_status_strings(gdn):
    assert gdn.status_string(0) == "GDN_OK"
    for code, name in gdn.STATUS_NAMES.items():
        assert gdn.status_string(code).startswith(name)
    assert "UNKNOWN" in gdn.status_string(99)


def test_host_side_argument_checks(gdn):
    L = gdn.lib()
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(0x1004)
    # decode
    assert L.gdn_decode(None, None, None, None, None, None, None, None, 0, 16, 32, 128, 128, None) == 0
    assert L.gdn_decode(None, fake, fake, fake, fake, fake, fake, fake, 2, 16, 32, 128, 128, None) == 1
    assert L.gdn_decode(fake, fake, fake, fake, fake, fake, fake, fake, -1, 16, 32, 128, 128, None) == 2
    assert L.gdn_decode(fake, fake, fake, fake, fake, fake, fake, fake, 2, 16, 33, 128, 128, None) == 2
    assert L.gdn_decode(fake, fake, fake, fake, fake, fake, fake, fake, 2, 16, 32, 64, 128, None) == 3
    assert L.gdn_decode(fake, fake, fake, fake, fake, odd, fake, fake, 2, 16, 32, 128, 128, None) == 5
    assert L.gdn_decode_variant(fake, fake, fake, fake, fake, fake, fake, fake, 2, 16, 32, 128, 128, 99, None) == 2
    # prefill
    assert L.gdn_prefill_workspace_bytes(4096, 1, 16, 32, 128, 128) > 0
    assert L.gdn_prefill_workspace_bytes(4096, 1, 16, 32, 64, 128) == 0
    args = [fake] * 9
    assert L.gdn_prefill(*args, 0, 0, 0, 16, 32, 128, 128, None, 0, None) == 0
    assert L.gdn_prefill(*args, 100, 2, 101, 16, 32, 128, 128, fake, 1 << 30, None) == 2  # max_seqlen > total
    assert L.gdn_prefill(*args, 100, 2, 10, 16, 32, 128, 128, fake, 1 << 30, None) == 2   # 2*10 < 100
    assert L.gdn_prefill(*args, 100, 0, 0, 16, 32, 128, 128, fake, 1 << 30, None) == 2
    a = list(args); a[5] = None
    assert L.gdn_prefill(*a, 100, 2, 60, 16, 32, 128, 128, fake, 1 << 30, None) == 1     # cu_seqlens NULL
    a = list(args); a[0] = odd
    assert L.gdn_prefill(*a, 100, 2, 60, 16, 32, 128, 128, fake, 1 << 30, None) == 5
    assert L.gdn_prefill_recurrent(*args, 100, 2, 101, 16, 32, 128, 128, None) == 2
    # fused front end
    assert L.gdn_decode_fused(fake, fake, fake, fake, fake, None, fake, fake, fake, fake, 2, 16, 32, 128, 128, 1.0, 1, None) == 1
    assert L.gdn_decode_fused(fake, fake, fake, fake, fake, None, None, fake, fake, fake, 2, 16, 32, 128, 128,
                              float("inf"), 1, None) == 2
    assert L.gdn_decode_fused(fake, fake, fake, fake, fake, None, None, fake, fake, fake, 0, 16, 32, 128, 128, 1.0, 1, None) == 0
    assert L.gdn_decode_multi_fused(fake, fake, fake, fake, fake, fake, None, fake, fake, fake, 2, 3, 16, 32, 128, 128,
                                    1.0, 1, None) == 1
    assert L.gdn_decode_multi_fused(fake, fake, fake, fake, fake, None, None, fake, fake, fake, 2, -1, 16, 32, 128, 128,
                                    1.0, 1, None) == 2
    assert L.gdn_decode_multi_fused(fake, fake, fake, fake, fake, None, None, fake, fake, fake, 2, 3, 16, 32, 128, 128,
                                    float("inf"), 0, None) == 2
    assert L.gdn_decode_multi(fake, fake, odd, fake, fake, fake, fake, fake, 2, 3, 16, 32, 128, 128, None) == 5
    fa = [fake] * 11
    assert L.gdn_prefill_fused(*fa, 100, 2, 60, 16, 32, 128, 128, float("nan"), 0, fake, 1 << 30, None) == 2
    a = list(fa); a[5] = None   # A_log without dt_bias
    assert L.gdn_prefill_fused(*a, 100, 2, 60, 16, 32, 128, 128, 1.0, 1, fake, 1 << 30, None) == 1
    a = list(fa); a[1] = odd
    assert L.gdn_prefill_fused(*a, 100, 2, 60, 16, 32, 128, 128, 1.0, 1, fake, 1 << 30, None) == 5
    assert L.gdn_prefill_fused(*fa, 0, 0, 0, 16, 32, 128, 128, 1.0, 1, None, 0, None) == 0
    # sequence-parallel building blocks
    pa = [fake] * 10
    assert L.gdn_prefill_partial(*pa, 0, 0, 0, 16, 32, 128, 128, None, 0, None) == 0
    assert L.gdn_prefill_partial(*pa, 100, 2, 101, 16, 32, 128, 128, fake, 1 << 30, None) == 2
    assert L.gdn_prefill_partial(*pa, 100, 2, 60, 16, 32, 64, 128, fake, 1 << 30, None) == 3
    a = list(pa); a[5] = None
    assert L.gdn_prefill_partial(*a, 100, 2, 60, 16, 32, 128, 128, fake, 1 << 30, None) == 1   # cu_seqlens NULL
    a = list(pa); a[2] = odd
    assert L.gdn_prefill_partial(*a, 100, 2, 60, 16, 32, 128, 128, fake, 1 << 30, None) == 5
    assert L.gdn_state_scan(fake, fake, fake, 3, fake, 0, 32, 128, 128, None) == 0             # no sequences
    assert L.gdn_state_scan(fake, fake, fake, -1, fake, 1, 32, 128, 128, None) == 2
    assert L.gdn_state_scan(fake, fake, fake, 3, None, 1, 32, 128, 128, None) == 1
    assert L.gdn_state_scan(fake, None, fake, 3, fake, 1, 32, 128, 128, None) == 1
    assert L.gdn_state_scan(fake, odd, fake, 3, fake, 1, 32, 128, 128, None) == 5
    assert L.gdn_state_scan(fake, fake, fake, 3, fake, 1, 32, 128, 64, None) == 3
    assert L.gdn_prefill_apply(fake, fake, fake, fake, 0, 0, 0, 32, 128, 128, None, 0, None) == 0
    assert L.gdn_prefill_apply(fake, fake, fake, fake, 100, 2, 101, 32, 128, 128, fake, 1 << 30, None) == 2
    assert L.gdn_prefill_apply(None, fake, fake, fake, 100, 2, 60, 32, 128, 128, fake, 1 << 30, None) == 1
    assert L.gdn_prefill_apply(fake, fake, odd, fake, 100, 2, 60, 32, 128, 128, fake, 1 << 30, None) == 5


def test_workspace_size_grows_with_tokens(gdn):
    a = gdn.gdn_prefill_workspace_bytes(64, 1, 1, 1)
    b = gdn.gdn_prefill_workspace_bytes(4096, 1, 16, 32)
    c = gdn.gdn_prefill_workspace_bytes(4096, 16, 16, 32)
    d = gdn.gdn_prefill_workspace_bytes(8192, 16, 16, 32)
    e = gdn.gdn_prefill_workspace_bytes(8192, 1, 16, 32)
    # few long sequences get extra room for the sequence-parallel scan, so b may exceed c
    assert 0 < a < b < e and a < c < d


class _FakeTensor:
    """Stands in for a CUDA tensor on a box without a GPU: the binding's checks only look at
    attributes, and every case below is rejected before a pointer is taken."""

    def __init__(self, shape, dtype, strides=None, device="cuda:0", cuda=True):
        import torch

        self.shape = tuple(shape)
        self.dtype = dtype
        self.is_cuda = cuda
        self.device = torch.device(device)
        self._contig = strides is None
        self._strides = strides

    def dim(self):
        return len(self.shape)

    def is_contiguous(self):
        return self._contig

    def stride(self):
        return self._strides or ()

    def data_ptr(self):
        raise AssertionError("a rejected tensor's pointer must never be taken")


def test_binding_rejects_tensors_the_c_abi_would_misread(gdn, monkeypatch):
    import torch

    monkeypatch.setattr(gdn, "_chk_current", lambda dev: None)
    bf, f32, i32 = torch.bfloat16, torch.float32, torch.int32
    B, Hqk, Hv = 2, 2, 4
    F = _FakeTensor

    def decode_args(**over):
        a = dict(q=F((B, Hqk, 128), bf), k=F((B, Hqk, 128), bf), v=F((B, Hv, 128), bf), g=F((B, Hv), f32),
                 beta=F((B, Hv), f32), state_in=F((B, Hv, 128, 128), f32), state_out=F((B, Hv, 128, 128), f32),
                 out=F((B, Hv, 128), bf))
        a.update(over)
        return [a[n] for n in ("q", "k", "v", "g", "beta", "state_in", "state_out", "out")]

    bad = [
        dict(q=F((B, Hqk, 128), bf, strides=(512, 256, 1))),              # a strided slice such as q[:, ::2]
        dict(state_in=F((B, Hv, 128, 128), f32, strides=(65536, 16384, 1, 128))),  # a transposed state
        dict(k=F((B, Hqk, 128), torch.float16)),                          # fp16 is not bf16
        dict(g=F((B, Hv), torch.float64)),
        dict(v=F((B, Hv, 128), bf, cuda=False, device="cpu")),
        dict(out=F((B, Hv, 64), bf)),                                     # wrong head size
        dict(state_out=F((B + 1, Hv, 128, 128), f32)),                    # batch disagrees
        dict(beta=F((B, Hv), f32, device="cuda:1")),                      # another device
        dict(q=None),
    ]
    for over in bad:
        with pytest.raises(ValueError):
            gdn.gdn_decode(*decode_args(**over))

    T, N = 100, 2

    def prefill_args(**over):
        a = dict(q=F((T, Hqk, 128), bf), k=F((T, Hqk, 128), bf), v=F((T, Hv, 128), bf), g=F((T, Hv), f32),
                 beta=F((T, Hv), f32), cu=F((N + 1,), i32), init=F((N, Hv, 128, 128), f32), out=F((T, Hv, 128), bf),
                 fin=F((N, Hv, 128, 128), f32))
        a.update(over)
        return [a[n] for n in ("q", "k", "v", "g", "beta", "cu", "init", "out", "fin")]

    ws = F((1 << 20,), torch.uint8)
    bad = [
        dict(cu=F((N + 1,), torch.int64)),                                # int64 offsets
        dict(init=F((N + 1, Hv, 128, 128), f32)),                         # N disagrees with cu_seqlens
        dict(fin=F((N, Hv, 128, 128), f32, strides=(1, 1, 1, 1))),
        dict(out=F((T - 1, Hv, 128), bf)),
        dict(v=F((T, Hv, 128), bf, strides=(1024, 256, 2))),
    ]
    for over in bad:
        with pytest.raises(ValueError):
            gdn.gdn_prefill(*prefill_args(**over), 60, ws)
        with pytest.raises(ValueError):
            gdn.gdn_prefill_static(*prefill_args(**over), 60)
    with pytest.raises(ValueError):
        gdn.gdn_prefill(*prefill_args(), 60, F((1 << 20,), torch.float32))  # the workspace is bytes
    with pytest.raises(ValueError):
        gdn.gdn_prefill_gated(*prefill_args()[:5], F((Hv + 1,), f32), F((Hv,), f32), *prefill_args()[5:], 60, ws)
