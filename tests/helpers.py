"""Shared test helpers: exact single-head views of packed inputs, error norms."""
import numpy as np

from gdn_inputs import bf16_bits_to_f32, f32_to_bf16_bits


def round_bf16(x):
    """fp64/fp32 array -> (bits uint16, exact fp64 value of the rounded bf16)."""
    bits = f32_to_bf16_bits(np.asarray(x, dtype=np.float32))
    return bits, bf16_bits_to_f32(bits).astype(np.float64)


def head_view(tok, t0, t1, h):
    """fp64 single-head arrays (q,k,v,g,beta) for tokens [t0,t1) and value head h."""
    hq = h // (tok.Hv // tok.Hqk)
    q = bf16_bits_to_f32(tok.q[t0:t1, hq]).astype(np.float64)
    k = bf16_bits_to_f32(tok.k[t0:t1, hq]).astype(np.float64)
    v = bf16_bits_to_f32(tok.v[t0:t1, h]).astype(np.float64)
    g = tok.g[t0:t1, h].astype(np.float64)
    b = tok.beta[t0:t1, h].astype(np.float64)
    return q, k, v, g, b


def rel_fro(a, ref):
    a = np.asarray(a, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref.ravel())
    num = np.linalg.norm((a - ref).ravel())
    if den == 0.0:
        return 0.0 if num == 0.0 else np.inf
    return num / den


def max_abs(a, ref):
    return float(np.max(np.abs(np.asarray(a, dtype=np.float64) - np.asarray(ref, dtype=np.float64)))) if np.size(ref) else 0.0
