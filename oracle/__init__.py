"""CPU oracle for the gated delta-rule recurrence -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares nothing with the CUDA library and never imports it.

`prefill` / `decode` call the plain fp64 token-by-token C implementation in
`gdn_oracle.c` (compiled here with gcc on first use).  `reformulations` holds
independent fp64 restatements (the paper's K x V form, an explicit matrix
product, the chunked WY/UT form) that the pin tests compare it with.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gdn_oracle.c")
_LIB = os.path.join(_HERE, "libgdn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile gdn_oracle.c -> libgdn_oracle.so (gcc -O2, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.c_void_p
        I = ctypes.c_int
        lib.gdn_oracle_prefill.argtypes = [P] * 9 + [I] * 6
        lib.gdn_oracle_prefill.restype = I
        lib.gdn_oracle_decode.argtypes = [P] * 8 + [I] * 6
        lib.gdn_oracle_decode.restype = I
        lib.gdn_oracle_prefill_gated.argtypes = [P] * 11 + [I] * 6
        lib.gdn_oracle_prefill_gated.restype = I
        lib.gdn_oracle_decode_gated.argtypes = [P] * 10 + [I] * 6
        lib.gdn_oracle_decode_gated.restype = I
        D = ctypes.c_double
        lib.gdn_oracle_prefill_fused.argtypes = [P] * 11 + [I] * 5 + [D, I, I]
        lib.gdn_oracle_prefill_fused.restype = I
        lib.gdn_oracle_decode_fused.argtypes = [P] * 10 + [I] * 5 + [D, I, I]
        lib.gdn_oracle_decode_fused.restype = I
        _lib = lib
    return _lib


def default_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def prefill(q, k, v, g, beta, cu_seqlens, initial_state=None, want_final=True,
            threads: Optional[int] = None) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """q,k: uint16(bf16) [T,Hqk,dk]; v: uint16 [T,Hv,dv]; g,beta: fp32 [T,Hv];
    cu_seqlens: int32 [N+1]; initial_state: fp32 [N,Hv,dv,dk] or None.
    Returns (out fp64 [T,Hv,dv], final_state fp64 [N,Hv,dv,dk] or None)."""
    q, k, v = _c(q, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    g, beta = _c(g, np.float32), _c(beta, np.float32)
    cu = _c(cu_seqlens, np.int32)
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu.shape[0] - 1
    assert k.shape == q.shape and v.shape[0] == T and g.shape == (T, Hv) and beta.shape == (T, Hv)
    assert cu[0] == 0 and cu[-1] == T and np.all(np.diff(cu) >= 0)
    if initial_state is not None:
        initial_state = _c(initial_state, np.float32)
        assert initial_state.shape == (N, Hv, dv, dk)
    out = np.zeros((T, Hv, dv), dtype=np.float64)
    fin = np.zeros((N, Hv, dv, dk), dtype=np.float64) if want_final else None
    rc = _load().gdn_oracle_prefill(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(cu),
                                    _ptr(initial_state), _ptr(out), _ptr(fin), N, Hqk, Hv, dk, dv,
                                    threads or default_threads())
    if rc != 0:
        raise ValueError("gdn_oracle_prefill: bad arguments")
    return out, fin


def decode(q, k, v, g, beta, state_in, threads: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """One token per batch item.  state_in: fp32 [B,Hv,dv,dk].
    Returns (out fp64 [B,Hv,dv], state_out fp64 [B,Hv,dv,dk])."""
    q, k, v = _c(q, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    g, beta = _c(g, np.float32), _c(beta, np.float32)
    state_in = _c(state_in, np.float32)
    B, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    assert state_in.shape == (B, Hv, dv, dk)
    out = np.zeros((B, Hv, dv), dtype=np.float64)
    so = np.zeros((B, Hv, dv, dk), dtype=np.float64)
    rc = _load().gdn_oracle_decode(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(state_in),
                                   _ptr(so), _ptr(out), B, Hqk, Hv, dk, dv, threads or default_threads())
    if rc != 0:
        raise ValueError("gdn_oracle_decode: bad arguments")
    return out, so


def prefill_gated(q, k, v, a, b, A_log, dt_bias, cu_seqlens, initial_state=None, want_final=True,
                  threads: Optional[int] = None):
    """As `prefill`, with the raw gate inputs: a,b fp32 [T,Hv]; A_log, dt_bias fp32 [Hv];
    alpha = exp(-exp(A_log) softplus(a + dt_bias)), beta = sigmoid(b) in fp64."""
    q, k, v = _c(q, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    a, b = _c(a, np.float32), _c(b, np.float32)
    A_log, dt_bias = _c(A_log, np.float32), _c(dt_bias, np.float32)
    cu = _c(cu_seqlens, np.int32)
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu.shape[0] - 1
    assert a.shape == (T, Hv) and b.shape == (T, Hv) and A_log.shape == (Hv,) and dt_bias.shape == (Hv,)
    if initial_state is not None:
        initial_state = _c(initial_state, np.float32)
    out = np.zeros((T, Hv, dv), dtype=np.float64)
    fin = np.zeros((N, Hv, dv, dk), dtype=np.float64) if want_final else None
    rc = _load().gdn_oracle_prefill_gated(_ptr(q), _ptr(k), _ptr(v), _ptr(a), _ptr(b), _ptr(A_log), _ptr(dt_bias),
                                          _ptr(cu), _ptr(initial_state), _ptr(out), _ptr(fin), N, Hqk, Hv, dk, dv,
                                          threads or default_threads())
    if rc != 0:
        raise ValueError("gdn_oracle_prefill_gated: bad arguments")
    return out, fin


def decode_gated(q, k, v, a, b, A_log, dt_bias, state_in, threads: Optional[int] = None):
    q, k, v = _c(q, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    a, b = _c(a, np.float32), _c(b, np.float32)
    A_log, dt_bias = _c(A_log, np.float32), _c(dt_bias, np.float32)
    state_in = _c(state_in, np.float32)
    B, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    out = np.zeros((B, Hv, dv), dtype=np.float64)
    so = np.zeros((B, Hv, dv, dk), dtype=np.float64)
    rc = _load().gdn_oracle_decode_gated(_ptr(q), _ptr(k), _ptr(v), _ptr(a), _ptr(b), _ptr(A_log), _ptr(dt_bias),
                                         _ptr(state_in), _ptr(so), _ptr(out), B, Hqk, Hv, dk, dv,
                                         threads or default_threads())
    if rc != 0:
        raise ValueError("gdn_oracle_decode_gated: bad arguments")
    return out, so


def prefill_fused(q, k, v, a, b, A_log, dt_bias, cu_seqlens, initial_state=None, scale=1.0, qk_l2norm=False,
                  want_final=True, threads: Optional[int] = None):
    """As `prefill_gated` with the fused front end: with qk_l2norm, q and k of every (token, head)
    are divided by sqrt(sum of squares + 1e-6); q is then multiplied by `scale` (all in fp64).
    A_log = dt_bias = None: a and b are the log-decay g and beta themselves."""
    q, k, v = _c(q, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    a, b = _c(a, np.float32), _c(b, np.float32)
    if A_log is not None:
        A_log, dt_bias = _c(A_log, np.float32), _c(dt_bias, np.float32)
    cu = _c(cu_seqlens, np.int32)
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu.shape[0] - 1
    assert a.shape == (T, Hv) and b.shape == (T, Hv)
    if initial_state is not None:
        initial_state = _c(initial_state, np.float32)
    out = np.zeros((T, Hv, dv), dtype=np.float64)
    fin = np.zeros((N, Hv, dv, dk), dtype=np.float64) if want_final else None
    rc = _load().gdn_oracle_prefill_fused(_ptr(q), _ptr(k), _ptr(v), _ptr(a), _ptr(b), _ptr(A_log), _ptr(dt_bias),
                                          _ptr(cu), _ptr(initial_state), _ptr(out), _ptr(fin), N, Hqk, Hv, dk, dv,
                                          float(scale), int(bool(qk_l2norm)), threads or default_threads())
    if rc != 0:
        raise ValueError("gdn_oracle_prefill_fused: bad arguments")
    return out, fin


def decode_fused(q, k, v, a, b, A_log, dt_bias, state_in, scale=1.0, qk_l2norm=False,
                 threads: Optional[int] = None):
    q, k, v = _c(q, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    a, b = _c(a, np.float32), _c(b, np.float32)
    if A_log is not None:
        A_log, dt_bias = _c(A_log, np.float32), _c(dt_bias, np.float32)
    state_in = _c(state_in, np.float32)
    B, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    out = np.zeros((B, Hv, dv), dtype=np.float64)
    so = np.zeros((B, Hv, dv, dk), dtype=np.float64)
    rc = _load().gdn_oracle_decode_fused(_ptr(q), _ptr(k), _ptr(v), _ptr(a), _ptr(b), _ptr(A_log), _ptr(dt_bias),
                                         _ptr(state_in), _ptr(so), _ptr(out), B, Hqk, Hv, dk, dv, float(scale),
                                         int(bool(qk_l2norm)), threads or default_threads())
    if rc != 0:
        raise ValueError("gdn_oracle_decode_fused: bad arguments")
    return out, so
