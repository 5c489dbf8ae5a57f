"""Python binding of libgdn (argument marshalling only; every step runs in the CUDA kernels).

The functions mirror the C entry points of include/gdn.h one to one and take torch CUDA
tensors (torch is used for device memory and streams only).  There is no CPU fallback:
if libgdn.so is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libgdn.so")

GDN_OK = 0
STATUS_NAMES = {0: "GDN_OK", 1: "GDN_ERR_NULL", 2: "GDN_ERR_SHAPE", 3: "GDN_ERR_UNSUPPORTED",
                4: "GDN_ERR_WORKSPACE", 5: "GDN_ERR_ALIGN", 6: "GDN_ERR_CUDA"}

# Every symbol include/gdn.h declares.
EXPORTS = ("gdn_status_string", "gdn_decode", "gdn_decode_variant", "gdn_decode_num_variants",
           "gdn_prefill_workspace_bytes", "gdn_prefill", "gdn_prefill_recurrent", "gdn_prefill_static",
           "gdn_decode_gated", "gdn_prefill_gated", "gdn_decode_fused", "gdn_prefill_fused", "gdn_decode_multi", "gdn_decode_multi_fused",
           "gdn_prefill_partial", "gdn_state_scan", "gdn_prefill_apply",
           "gdn_last_device_status")


class GdnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s" % (where, status_string(status)))


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libgdn.so (built in-tree by paper_2607_16831_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libgdn.so is not built: run `python -m paper_2607_16831_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        P, I, Z = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.gdn_status_string.argtypes = [I]
        L.gdn_status_string.restype = ctypes.c_char_p
        L.gdn_decode.argtypes = [P] * 8 + [I] * 5 + [P]
        L.gdn_decode.restype = I
        L.gdn_decode_variant.argtypes = [P] * 8 + [I] * 6 + [P]
        L.gdn_decode_variant.restype = I
        L.gdn_decode_num_variants.argtypes = []
        L.gdn_decode_num_variants.restype = I
        L.gdn_prefill_workspace_bytes.argtypes = [I] * 6
        L.gdn_prefill_workspace_bytes.restype = Z
        L.gdn_prefill.argtypes = [P] * 9 + [I] * 7 + [P, Z, P]
        L.gdn_prefill.restype = I
        L.gdn_prefill_recurrent.argtypes = [P] * 9 + [I] * 7 + [P]
        L.gdn_prefill_recurrent.restype = I
        L.gdn_prefill_static.argtypes = [P] * 9 + [I] * 7 + [P]
        L.gdn_prefill_static.restype = I
        L.gdn_decode_multi.argtypes = [P] * 8 + [I] * 6 + [P]
        L.gdn_decode_multi.restype = I
        L.gdn_decode_gated.argtypes = [P] * 10 + [I] * 5 + [P]
        L.gdn_decode_gated.restype = I
        L.gdn_prefill_gated.argtypes = [P] * 11 + [I] * 7 + [P, Z, P]
        L.gdn_prefill_gated.restype = I
        F = ctypes.c_float
        L.gdn_decode_fused.argtypes = [P] * 10 + [I] * 5 + [F, I, P]
        L.gdn_decode_fused.restype = I
        L.gdn_prefill_fused.argtypes = [P] * 11 + [I] * 7 + [F, I, P, Z, P]
        L.gdn_prefill_fused.restype = I
        L.gdn_decode_multi_fused.argtypes = [P] * 10 + [I] * 6 + [F, I, P]
        L.gdn_decode_multi_fused.restype = I
        L.gdn_prefill_partial.argtypes = [P] * 10 + [I] * 7 + [P, Z, P]
        L.gdn_prefill_partial.restype = I
        L.gdn_state_scan.argtypes = [P, P, P, I, P, I, I, I, I, P]
        L.gdn_state_scan.restype = I
        L.gdn_prefill_apply.argtypes = [P] * 4 + [I] * 6 + [P, Z, P]
        L.gdn_prefill_apply.restype = I
        L.gdn_last_device_status.argtypes = [P, ctypes.POINTER(I), P]
        L.gdn_last_device_status.restype = I
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().gdn_status_string(int(status)).decode()


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


_DT = {}


def _dtypes():
    if not _DT:
        import torch

        _DT.update(bf16=torch.bfloat16, f32=torch.float32, i32=torch.int32, u8=torch.uint8)
    return _DT


def _chk(name: str, t, dtype: str, shape=None, optional: bool = False, device=None):
    """The C ABI takes bare pointers, so a strided view, a wrong dtype or a tensor on another device
    would be read as garbage without any error.  Everything handed over is checked here: CUDA,
    contiguous, the expected dtype, the expected shape (None entries are free), one device.
    Returns the tensor's device (or `device` when the tensor is None)."""
    if t is None:
        if optional:
            return device
        raise ValueError("%s is required" % name)
    if not getattr(t, "is_cuda", False):
        raise ValueError("%s must be a CUDA tensor" % name)
    if t.dtype is not (_DT or _dtypes())[dtype]:
        raise ValueError("%s must be %s, got %s" % (name, _DT[dtype], t.dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous (got strides %s for shape %s)" % (name, tuple(t.stride()), tuple(t.shape)))
    if shape is not None:
        ts = t.shape
        if len(ts) != len(shape) or any(e is not None and e != a for e, a in zip(shape, ts)):
            raise ValueError("%s must have shape %s, got %s" % (name, tuple(shape), tuple(t.shape)))
    if device is not None and t.device != device:
        raise ValueError("%s is on %s, the other tensors are on %s" % (name, t.device, device))
    return t.device


def _chk_current(device) -> None:
    import torch

    if device is not None and device.index != torch.cuda.current_device():
        raise ValueError("tensors are on %s but the current CUDA device is %d" % (device, torch.cuda.current_device()))


def _chk_tokens(q, k, v, g, beta, lead, names=("g", "beta")):
    """q,k bf16 [*lead,Hqk,128]; v bf16 [*lead,Hv,128]; g,beta fp32 [*lead,Hv].  Returns (Hqk, Hv, device)."""
    n = len(lead)
    if q is None or q.dim() != n + 2 or v is None or v.dim() != n + 2:
        raise ValueError("q and v must have %d dimensions" % (n + 2))
    Hqk, Hv = int(q.shape[n]), int(v.shape[n])
    dev = _chk("q", q, "bf16", (*lead, Hqk, 128))
    _chk("k", k, "bf16", (*lead, Hqk, 128), device=dev)
    _chk("v", v, "bf16", (*lead, Hv, 128), device=dev)
    _chk(names[0], g, "f32", (*lead, Hv), device=dev)
    _chk(names[1], beta, "f32", (*lead, Hv), device=dev)
    return Hqk, Hv, dev


def _chk_raw_gates(A_log, dt_bias, Hv, dev, required: bool):
    # a missing gate parameter is the library's to report (GDN_ERR_NULL); what is present is checked here
    _chk("A_log", A_log, "f32", (Hv,), optional=True, device=dev)
    _chk("dt_bias", dt_bias, "f32", (Hv,), optional=True, device=dev)


def _chk_prefill(q, k, v, g, beta, cu_seqlens, initial_state, out, final_state, workspace, names=("g", "beta")):
    if q is None or q.dim() != 3:
        raise ValueError("q must have 3 dimensions")
    T = int(q.shape[0])
    Hqk, Hv, dev = _chk_tokens(q, k, v, g, beta, (T,), names)
    _chk("cu_seqlens", cu_seqlens, "i32", (None,), device=dev)
    N = int(cu_seqlens.shape[0]) - 1
    if N < 0:
        raise ValueError("cu_seqlens must have at least one entry")
    _chk("initial_state", initial_state, "f32", (N, Hv, 128, 128), optional=True, device=dev)
    _chk("out", out, "bf16", (T, Hv, 128), device=dev)
    _chk("final_state", final_state, "f32", (N, Hv, 128, 128), optional=True, device=dev)
    _chk("workspace", workspace, "u8", (None,), optional=True, device=dev)
    _chk_current(dev)
    return T, N, Hqk, Hv


def _chk_decode(q, k, v, g, beta, state_in, state_out, out, lead_tokens=(), names=("g", "beta")):
    if q is None or q.dim() < 1:
        raise ValueError("q must be a tensor")
    B = int(q.shape[0])
    Hqk, Hv, dev = _chk_tokens(q, k, v, g, beta, (B, *lead_tokens), names)
    _chk("state_in", state_in, "f32", (B, Hv, 128, 128), device=dev)
    _chk("state_out", state_out, "f32", (B, Hv, 128, 128), device=dev)
    _chk("out", out, "bf16", (B, *lead_tokens, Hv, 128), device=dev)
    _chk_current(dev)
    return B, Hqk, Hv, dev


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch

        stream = torch.cuda.current_stream()
    s = int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)
    return s or None


def _check(rc: int, where: str) -> None:
    if rc != GDN_OK:
        raise GdnError(rc, where)


def gdn_decode(q, k, v, g, beta, state_in, state_out, out, stream=None, variant: int = -1) -> None:
    """q,k: bf16 [B,Hqk,128]; v,out: bf16 [B,Hv,128]; g,beta: fp32 [B,Hv];
    state_in/state_out: fp32 [B,Hv,128,128].  Enqueues on `stream` (default: current)."""
    _chk_decode(q, k, v, g, beta, state_in, state_out, out)
    B, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    args = [_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(state_in), _ptr(state_out), _ptr(out),
            B, Hqk, Hv, dk, dv]
    if variant < 0:
        _check(lib().gdn_decode(*args, _stream(stream)), "gdn_decode")
    else:
        _check(lib().gdn_decode_variant(*args, variant, _stream(stream)), "gdn_decode_variant")


def gdn_decode_num_variants() -> int:
    return int(lib().gdn_decode_num_variants())


def gdn_prefill_workspace_bytes(total_tokens: int, num_seqs: int, Hqk: int, Hv: int, dk: int = 128,
                                dv: int = 128) -> int:
    return int(lib().gdn_prefill_workspace_bytes(total_tokens, num_seqs, Hqk, Hv, dk, dv))


def gdn_prefill(q, k, v, g, beta, cu_seqlens, initial_state, out, final_state, max_seqlen: int, workspace,
                stream=None) -> None:
    """q,k: bf16 [T,Hqk,128]; v,out: bf16 [T,Hv,128]; g,beta: fp32 [T,Hv]; cu_seqlens: int32 [N+1]
    (device); initial_state/final_state: fp32 [N,Hv,128,128] or None; workspace: a uint8 CUDA
    tensor of at least gdn_prefill_workspace_bytes(...) bytes, 1024-byte aligned."""
    _chk_prefill(q, k, v, g, beta, cu_seqlens, initial_state, out, final_state, workspace)
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().gdn_prefill(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(cu_seqlens), _ptr(initial_state),
                           _ptr(out), _ptr(final_state), T, N, int(max_seqlen), Hqk, Hv, dk, dv, _ptr(workspace),
                           wbytes, _stream(stream))
    _check(rc, "gdn_prefill")


def gdn_prefill_recurrent(q, k, v, g, beta, cu_seqlens, initial_state, out, final_state, max_seqlen: int,
                          stream=None) -> None:
    _chk_prefill(q, k, v, g, beta, cu_seqlens, initial_state, out, final_state, None)
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    rc = lib().gdn_prefill_recurrent(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(cu_seqlens),
                                     _ptr(initial_state), _ptr(out), _ptr(final_state), T, N, int(max_seqlen),
                                     Hqk, Hv, dk, dv, _stream(stream))
    _check(rc, "gdn_prefill_recurrent")


def gdn_prefill_partial(q, k, v, g, beta, cu_seqlens, out0, qt, H, P, max_seqlen: int, workspace, stream=None) -> None:
    """A piece of every sequence without its entering state: out0 = H_t q_t, qt = M_t q_t (bf16
    [T,Hv,128]); H, P fp32 [N,Hv,128,128] with S_end = S_in P + H."""
    _T, _N, _, _Hv = _chk_prefill(q, k, v, g, beta, cu_seqlens, None, out0, None, workspace)
    _chk("qt", qt, "bf16", (_T, _Hv, 128), device=q.device)
    _chk("H", H, "f32", (_N, _Hv, 128, 128), device=q.device)
    _chk("P", P, "f32", (_N, _Hv, 128, 128), device=q.device)
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().gdn_prefill_partial(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(cu_seqlens), _ptr(out0),
                                   _ptr(qt), _ptr(H), _ptr(P), T, N, int(max_seqlen), Hqk, Hv, dk, dv,
                                   _ptr(workspace), wbytes, _stream(stream))
    _check(rc, "gdn_prefill_partial")


def gdn_state_scan(S0, P, H, S_out, stream=None) -> None:
    """S_out = (...((S0 P[0] + H[0]) P[1] + H[1])...); P, H fp32 [steps,N,Hv,128,128]; S0 fp32
    [N,Hv,128,128] or None (zeros)."""
    steps = 0 if P is None else int(P.shape[0])
    dev = _chk("S_out", S_out, "f32", (None, None, 128, 128))
    N, Hv, dv, dk = S_out.shape
    _chk("S0", S0, "f32", (N, Hv, 128, 128), optional=True, device=dev)
    _chk("P", P, "f32", (steps, N, Hv, 128, 128), optional=True, device=dev)
    _chk("H", H, "f32", (steps, N, Hv, 128, 128), optional=steps == 0, device=dev)
    _chk_current(dev)
    rc = lib().gdn_state_scan(_ptr(S0), _ptr(P), _ptr(H), steps, _ptr(S_out), N, Hv, dk, dv, _stream(stream))
    _check(rc, "gdn_state_scan")


def gdn_prefill_apply(S_in, qt, out, cu_seqlens, max_seqlen: int, workspace, stream=None) -> None:
    """out[t] += S_in qt[t] for every token of every sequence (out holds gdn_prefill_partial's out0)."""
    dev = _chk("qt", qt, "bf16", (None, None, 128))
    T, Hv, dk = qt.shape
    N = cu_seqlens.shape[0] - 1
    _chk("S_in", S_in, "f32", (N, Hv, 128, 128), device=dev)
    _chk("out", out, "bf16", (T, Hv, 128), device=dev)
    _chk("cu_seqlens", cu_seqlens, "i32", (None,), device=dev)
    _chk("workspace", workspace, "u8", (None,), optional=True, device=dev)
    _chk_current(dev)
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().gdn_prefill_apply(_ptr(S_in), _ptr(qt), _ptr(out), _ptr(cu_seqlens), T, N, int(max_seqlen), Hv, dk,
                                 out.shape[2], _ptr(workspace), wbytes, _stream(stream))
    _check(rc, "gdn_prefill_apply")


def gdn_decode_multi(q, k, v, g, beta, state_in, state_out, out, stream=None) -> None:
    """T tokens per batch item in one pass over the state: q,k bf16 [B,T,Hqk,128]; v,out bf16
    [B,T,Hv,128]; g,beta fp32 [B,T,Hv]; states fp32 [B,Hv,128,128]."""
    _chk_decode(q, k, v, g, beta, state_in, state_out, out, lead_tokens=(int(q.shape[1]),) if q is not None and q.dim() == 4 else (0,))
    B, T, Hqk, dk = q.shape
    _, _, Hv, dv = v.shape
    rc = lib().gdn_decode_multi(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(state_in), _ptr(state_out),
                                _ptr(out), B, T, Hqk, Hv, dk, dv, _stream(stream))
    _check(rc, "gdn_decode_multi")


def gdn_decode_gated(q, k, v, a, b, A_log, dt_bias, state_in, state_out, out, stream=None) -> None:
    """gdn_decode with the gate arithmetic fused in: a,b fp32 [B,Hv] raw gate inputs, A_log and
    dt_bias fp32 [Hv]; alpha = exp(-exp(A_log) softplus(a + dt_bias)), beta = sigmoid(b)."""
    _, _, _Hv, _dev = _chk_decode(q, k, v, a, b, state_in, state_out, out, names=("a", "b"))
    _chk_raw_gates(A_log, dt_bias, _Hv, _dev, required=True)
    B, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    rc = lib().gdn_decode_gated(_ptr(q), _ptr(k), _ptr(v), _ptr(a), _ptr(b), _ptr(A_log), _ptr(dt_bias),
                                _ptr(state_in), _ptr(state_out), _ptr(out), B, Hqk, Hv, dk, dv, _stream(stream))
    _check(rc, "gdn_decode_gated")


def gdn_prefill_gated(q, k, v, a, b, A_log, dt_bias, cu_seqlens, initial_state, out, final_state, max_seqlen: int,
                      workspace, stream=None) -> None:
    """gdn_prefill with the gate arithmetic fused in (see gdn_decode_gated)."""
    _, _, _, _Hv = _chk_prefill(q, k, v, a, b, cu_seqlens, initial_state, out, final_state, workspace, names=("a", "b"))
    _chk_raw_gates(A_log, dt_bias, _Hv, q.device, required=True)
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().gdn_prefill_gated(_ptr(q), _ptr(k), _ptr(v), _ptr(a), _ptr(b), _ptr(A_log), _ptr(dt_bias),
                                 _ptr(cu_seqlens), _ptr(initial_state), _ptr(out), _ptr(final_state), T, N,
                                 int(max_seqlen), Hqk, Hv, dk, dv, _ptr(workspace), wbytes, _stream(stream))
    _check(rc, "gdn_prefill_gated")


def gdn_decode_fused(q, k, v, a, b, A_log, dt_bias, state_in, state_out, out, scale: float = 1.0,
                     qk_l2norm: bool = False, stream=None) -> None:
    """gdn_decode with the operator's front end fused in: raw gates as in gdn_decode_gated (A_log =
    dt_bias = None: a, b are g and beta), q and k divided by sqrt(sum of squares + 1e-6) when
    qk_l2norm, q multiplied by scale."""
    _, _, _Hv, _dev = _chk_decode(q, k, v, a, b, state_in, state_out, out, names=("a", "b"))
    _chk_raw_gates(A_log, dt_bias, _Hv, _dev, required=False)
    B, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    rc = lib().gdn_decode_fused(_ptr(q), _ptr(k), _ptr(v), _ptr(a), _ptr(b), _ptr(A_log), _ptr(dt_bias),
                                _ptr(state_in), _ptr(state_out), _ptr(out), B, Hqk, Hv, dk, dv, float(scale),
                                int(bool(qk_l2norm)), _stream(stream))
    _check(rc, "gdn_decode_fused")


def gdn_decode_multi_fused(q, k, v, a, b, A_log, dt_bias, state_in, state_out, out, scale: float = 1.0,
                           qk_l2norm: bool = False, stream=None) -> None:
    """gdn_decode_multi with the front end of gdn_decode_fused (a, b fp32 [B,T,Hv])."""
    _, _, _Hv, _dev = _chk_decode(q, k, v, a, b, state_in, state_out, out, names=("a", "b"),
                                  lead_tokens=(int(q.shape[1]),) if q is not None and q.dim() == 4 else (0,))
    _chk_raw_gates(A_log, dt_bias, _Hv, _dev, required=False)
    B, T, Hqk, dk = q.shape
    _, _, Hv, dv = v.shape
    rc = lib().gdn_decode_multi_fused(_ptr(q), _ptr(k), _ptr(v), _ptr(a), _ptr(b), _ptr(A_log), _ptr(dt_bias),
                                      _ptr(state_in), _ptr(state_out), _ptr(out), B, T, Hqk, Hv, dk, dv, float(scale),
                                      int(bool(qk_l2norm)), _stream(stream))
    _check(rc, "gdn_decode_multi_fused")


def gdn_prefill_fused(q, k, v, a, b, A_log, dt_bias, cu_seqlens, initial_state, out, final_state, max_seqlen: int,
                      workspace, scale: float = 1.0, qk_l2norm: bool = False, stream=None) -> None:
    """gdn_prefill with the operator's front end fused in (see gdn_decode_fused)."""
    _, _, _, _Hv = _chk_prefill(q, k, v, a, b, cu_seqlens, initial_state, out, final_state, workspace, names=("a", "b"))
    _chk_raw_gates(A_log, dt_bias, _Hv, q.device, required=False)
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().gdn_prefill_fused(_ptr(q), _ptr(k), _ptr(v), _ptr(a), _ptr(b), _ptr(A_log), _ptr(dt_bias),
                                 _ptr(cu_seqlens), _ptr(initial_state), _ptr(out), _ptr(final_state), T, N,
                                 int(max_seqlen), Hqk, Hv, dk, dv, float(scale), int(bool(qk_l2norm)),
                                 _ptr(workspace), wbytes, _stream(stream))
    _check(rc, "gdn_prefill_fused")


PREFILL_STATIC_SCRATCH_BYTES = 32 * 1024 * 1024


def gdn_prefill_static(q, k, v, g, beta, cu_seqlens, initial_state, out, final_state, max_seqlen: int,
                       stream=None) -> None:
    """gdn_prefill for callers that cannot allocate device memory (a frozen memory pool, an
    allocation-free request path): no workspace argument, the scratch is a fixed
    PREFILL_STATIC_SCRATCH_BYTES array inside the library.  Raises GdnError(GDN_ERR_WORKSPACE)
    when gdn_prefill_workspace_bytes(...) for the problem exceeds it.  Calls on one device must
    not overlap on the GPU: they share that one array.  gdn_last_device_status(None) reads the
    status word of that array."""
    _chk_prefill(q, k, v, g, beta, cu_seqlens, initial_state, out, final_state, None)
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    rc = lib().gdn_prefill_static(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(cu_seqlens),
                                  _ptr(initial_state), _ptr(out), _ptr(final_state), T, N, int(max_seqlen),
                                  Hqk, Hv, dk, dv, _stream(stream))
    _check(rc, "gdn_prefill_static")


def gdn_last_device_status(workspace, stream=None) -> int:
    """Reads and clears the device status word of a prefill workspace (None: the fixed scratch of
    gdn_prefill_static on the current device).  0 = no kernel gave up on a bounded wait."""
    _chk("workspace", workspace, "u8", (None,), optional=True)
    val = ctypes.c_int(0)
    _check(lib().gdn_last_device_status(_ptr(workspace), ctypes.byref(val), _stream(stream)),
           "gdn_last_device_status")
    return int(val.value)
