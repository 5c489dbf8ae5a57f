"""Seeded synthetic inputs for the gated delta-rule workloads.

This module only *draws* inputs (random numbers, normalisation of the drawn
vectors, rounding to the storage dtypes).  It holds none of the recurrence's
arithmetic and imports neither the CPU oracle nor the CUDA library, so both can
consume exactly the same bytes.

Storage conventions (the library's boundary):
  q, k : bf16 [T, Hqk, dk]   held as numpy uint16 bit patterns
  v    : bf16 [T, Hv,  dv]   held as numpy uint16 bit patterns
  g    : fp32 [T, Hv]        log-decay, alpha = exp(g), g <= 0
  beta : fp32 [T, Hv]
  state: fp32 [N, Hv, dv, dk] (K contiguous)

Recipe (one numpy PCG64 generator per call, draw order fixed):
  q, k, v ~ N(0,1) in fp32; q and k are L2-normalised per (token, head) in fp32,
  q is then scaled by 1/sqrt(dk); all three are rounded to bf16 (nearest-even).
  g = log(sigmoid(x)) with x ~ N(gate_mean, 1), evaluated as -softplus(-x) in fp32.
  beta = sigmoid(N(0,1)) in fp32.  States ~ N(0, sd 0.02) in fp32.
Draw order: q, k, v, x, beta-logits, state, (sequence lengths are drawn from a
second generator seeded with seed+1 so they do not shift the tensor draws).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

__all__ = [
    "f32_to_bf16_bits",
    "bf16_bits_to_f32",
    "Tokens",
    "make_tokens",
    "make_state",
    "make_cu_seqlens",
    "make_varlen_lengths",
    "make_raw_gates",
    "config",
    "CONFIG_NAMES",
]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp32."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Tokens:
    """One packed batch of token inputs (decode: T = B, one token per item)."""

    q: np.ndarray  # uint16 [T,Hqk,dk]
    k: np.ndarray  # uint16 [T,Hqk,dk]
    v: np.ndarray  # uint16 [T,Hv,dv]
    g: np.ndarray  # float32 [T,Hv]
    beta: np.ndarray  # float32 [T,Hv]
    Hqk: int = 0
    Hv: int = 0
    dk: int = 0
    dv: int = 0
    meta: dict = field(default_factory=dict)

    @property
    def T(self) -> int:
        return int(self.q.shape[0])


def _log_sigmoid_f32(x: np.ndarray) -> np.ndarray:
    # log(sigmoid(x)) = -softplus(-x) = -(max(-x,0) + log1p(exp(-|x|)))
    x = x.astype(np.float32)
    return (-(np.maximum(-x, np.float32(0)) + np.log1p(np.exp(-np.abs(x))))).astype(np.float32)


def _sigmoid_f32(x: np.ndarray) -> np.ndarray:
    x = x.astype(np.float32)
    return (np.float32(1) / (np.float32(1) + np.exp(-x))).astype(np.float32)


def make_tokens(
    T: int,
    Hqk: int,
    Hv: int,
    dk: int = 128,
    dv: int = 128,
    seed: int = 0,
    gate_mean: float = 2.0,
    key_correlation: float = 0.0,
    rng: Optional[np.random.Generator] = None,
) -> Tokens:
    """Draw q,k,v,g,beta for T packed tokens.

    gate_mean: mean of x in g = log(sigmoid(x)); 2.0 is the workload's value
      (forgets in ~50 tokens), 6.0 gives a weak decay (mean g ~ -0.0025) that
      makes inter-chunk state propagation visible in long sequences.
    key_correlation in [0,1): mixes a per-head common direction into every key
      before normalisation, which makes the intra-chunk triangular system far
      from the identity (a stress input, not one of the workload configs).
    """
    if rng is None:
        rng = np.random.default_rng(seed)
    q = rng.standard_normal((T, Hqk, dk), dtype=np.float32)
    k = rng.standard_normal((T, Hqk, dk), dtype=np.float32)
    v = rng.standard_normal((T, Hv, dv), dtype=np.float32)
    x = rng.standard_normal((T, Hv), dtype=np.float32) + np.float32(gate_mean)
    b = rng.standard_normal((T, Hv), dtype=np.float32)
    if key_correlation > 0.0:
        common = np.random.default_rng(seed + 7919).standard_normal((1, Hqk, dk), dtype=np.float32)
        c = np.float32(key_correlation)
        k = (np.float32(1) - c) * k + c * np.float32(np.sqrt(dk)) * common / np.linalg.norm(
            common, axis=-1, keepdims=True
        ).astype(np.float32)
    eps = np.float32(1e-12)
    q = q / np.maximum(np.linalg.norm(q, axis=-1, keepdims=True), eps)
    k = k / np.maximum(np.linalg.norm(k, axis=-1, keepdims=True), eps)
    q = q * np.float32(1.0 / np.sqrt(dk))
    return Tokens(
        q=f32_to_bf16_bits(q),
        k=f32_to_bf16_bits(k),
        v=f32_to_bf16_bits(v),
        g=_log_sigmoid_f32(x),
        beta=_sigmoid_f32(b),
        Hqk=Hqk,
        Hv=Hv,
        dk=dk,
        dv=dv,
        meta={"seed": seed, "gate_mean": gate_mean, "key_correlation": key_correlation},
    )


def make_raw_gates(T: int, Hv: int, seed: int = 0):
    """Raw gate inputs of the paper's gate parameterisation: a, b fp32 [T,Hv] ~ N(0,1);
    A_log = log(U(1,16)) and dt_bias = softplus^-1(dt), dt log-uniform in [1e-3, 1e-1], fp32 [Hv]
    (the usual initialisation of this layer), so exp(A_log) softplus(a + dt_bias) stays within a
    few units.  Returns (a, b, A_log, dt_bias)."""
    rng = np.random.default_rng(seed + 15485863)
    a = rng.standard_normal((T, Hv), dtype=np.float32)
    b = rng.standard_normal((T, Hv), dtype=np.float32)
    A_log = np.log(rng.uniform(1.0, 16.0, size=Hv)).astype(np.float32)
    dt = np.exp(rng.uniform(np.log(1e-3), np.log(1e-1), size=Hv))
    dt_bias = (dt + np.log(-np.expm1(-dt))).astype(np.float32)
    return a, b, A_log, dt_bias


def make_state(N: int, Hv: int, dk: int = 128, dv: int = 128, seed: int = 0, sd: float = 0.02,
               rng: Optional[np.random.Generator] = None) -> np.ndarray:
    """fp32 [N,Hv,dv,dk] ~ N(0, sd)."""
    if rng is None:
        rng = np.random.default_rng(seed + 104729)
    s = rng.standard_normal((N, Hv, dv, dk), dtype=np.float32)
    s *= np.float32(sd)
    return s


def make_varlen_lengths(num_seqs: int, lo: int = 1, hi: int = 2048, seed: int = 0, chunk: int = 64) -> np.ndarray:
    """Lengths uniform in [lo,hi]; redraws (seed+1, seed+2, ...) until at least
    one length is not a multiple of the chunk size."""
    s = seed + 1
    while True:
        rng = np.random.default_rng(s)
        lens = rng.integers(lo, hi + 1, size=num_seqs, dtype=np.int64)
        if hi < chunk or np.any(lens % chunk != 0):
            return lens.astype(np.int32)
        s += 1


def make_cu_seqlens(lengths) -> np.ndarray:
    lengths = np.asarray(lengths, dtype=np.int64)
    cu = np.zeros(len(lengths) + 1, dtype=np.int64)
    np.cumsum(lengths, out=cu[1:])
    assert cu[-1] < 2**31
    return cu.astype(np.int32)


CONFIG_NAMES = ("prefill_tiny", "decode_b64", "decode_sweep", "prefill_long", "prefill_varlen")


def config(name: str, seed: int = 0, **over) -> dict:
    """The five workload configurations, as dictionaries of numpy arrays.

    prefill_tiny   : N=1, T=64, Hqk=Hv=1, zero initial state.
    decode_b64     : B=64, Hqk=16, Hv=32, state ~ N(0,0.02); `B=` overrides the
                     batch (the sweep uses B in {1,8,32,128,256}).
    prefill_long   : N=1, T=4096, 16/32 heads; `initial=True` adds an N(0,0.02) state.
    prefill_varlen : N=16, lengths U[1,2048], per-sequence N(0,0.02) states.
    Overrides: Hqk, Hv, dk, dv, T, B, N, max_len, gate_mean, initial.
    """
    dk = over.get("dk", 128)
    dv = over.get("dv", 128)
    gate_mean = over.get("gate_mean", 2.0)
    if name == "prefill_tiny":
        Hqk, Hv, T = over.get("Hqk", 1), over.get("Hv", 1), over.get("T", 64)
        tok = make_tokens(T, Hqk, Hv, dk, dv, seed, gate_mean)
        return dict(kind="prefill", tokens=tok, cu_seqlens=make_cu_seqlens([T]), initial_state=None, N=1)
    if name in ("decode_b64", "decode_sweep"):
        B = over.get("B", 64)
        Hqk, Hv = over.get("Hqk", 16), over.get("Hv", 32)
        tok = make_tokens(B, Hqk, Hv, dk, dv, seed, gate_mean)
        return dict(kind="decode", tokens=tok, state=make_state(B, Hv, dk, dv, seed), B=B)
    if name == "prefill_long":
        Hqk, Hv, T = over.get("Hqk", 16), over.get("Hv", 32), over.get("T", 4096)
        tok = make_tokens(T, Hqk, Hv, dk, dv, seed, gate_mean)
        init = make_state(1, Hv, dk, dv, seed) if over.get("initial", False) else None
        return dict(kind="prefill", tokens=tok, cu_seqlens=make_cu_seqlens([T]), initial_state=init, N=1)
    if name == "prefill_varlen":
        N = over.get("N", 16)
        Hqk, Hv = over.get("Hqk", 16), over.get("Hv", 32)
        lens = make_varlen_lengths(N, 1, over.get("max_len", 2048), seed)
        cu = make_cu_seqlens(lens)
        tok = make_tokens(int(cu[-1]), Hqk, Hv, dk, dv, seed, gate_mean)
        return dict(kind="prefill", tokens=tok, cu_seqlens=cu, initial_state=make_state(N, Hv, dk, dv, seed), N=N)
    raise KeyError(name)
