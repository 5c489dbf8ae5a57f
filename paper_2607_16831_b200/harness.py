"""Host-side harness: moves seeded numpy inputs to the device, calls the binding, brings
results back, and compares against reference arrays handed in by the caller.  It never
imports the CPU oracle; tests, the smoke check and the benchmark pass the oracle's
arrays in."""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import (gdn_decode, gdn_last_device_status, gdn_prefill, gdn_prefill_recurrent,
               gdn_prefill_workspace_bytes)

# Acceptance tolerances: bf16 outputs within max-abs 2e-2 and relative Frobenius 1e-2;
# fp32 states within relative Frobenius 5e-3.
OUT_MAX_ABS = 2e-2
OUT_REL_FRO = 1e-2
STATE_REL_FRO = 5e-3


def token_arrays(tok):
    return tok.q, tok.k, tok.v, tok.g, tok.beta


def bf16_to_device(bits: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def bf16_to_numpy(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> float64 numpy (exact)."""
    return t.detach().float().cpu().numpy().astype(np.float64)


def to_device(tok, device="cuda"):
    return dict(
        q=bf16_to_device(tok.q, device), k=bf16_to_device(tok.k, device), v=bf16_to_device(tok.v, device),
        g=torch.from_numpy(tok.g).to(device), beta=torch.from_numpy(tok.beta).to(device))


def alloc_workspace(total_tokens: int, num_seqs: int, Hqk: int, Hv: int, device="cuda") -> torch.Tensor:
    n = gdn_prefill_workspace_bytes(total_tokens, num_seqs, Hqk, Hv)
    buf = torch.empty(n + 1024, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 1024
    return buf[off:off + n]


def run_decode(cfg, variant: int = -1, in_place: bool = False, device="cuda"):
    tok = cfg["tokens"]
    d = to_device(tok, device)
    s_in = torch.from_numpy(cfg["state"]).to(device)
    s_out = s_in if in_place else torch.full_like(s_in, float("nan"))
    out = torch.full((tok.T, tok.Hv, tok.dv), float("nan"), dtype=torch.bfloat16, device=device)
    gdn_decode(d["q"], d["k"], d["v"], d["g"], d["beta"], s_in, s_out, out, variant=variant)
    torch.cuda.synchronize()
    return dict(out=bf16_to_numpy(out), state_out=s_out.cpu().numpy().astype(np.float64))


def run_prefill(cfg, recurrent: bool = False, want_final: bool = True, device="cuda"):
    tok = cfg["tokens"]
    d = to_device(tok, device)
    cu_np = np.asarray(cfg["cu_seqlens"], dtype=np.int32)
    cu = torch.from_numpy(cu_np).to(device)
    N = cu_np.shape[0] - 1
    max_len = int(np.max(np.diff(cu_np))) if N > 0 else 0
    init = None if cfg.get("initial_state") is None else torch.from_numpy(cfg["initial_state"]).to(device)
    out = torch.full((tok.T, tok.Hv, tok.dv), float("nan"), dtype=torch.bfloat16, device=device)
    fin = torch.full((N, tok.Hv, tok.dv, tok.dk), float("nan"), dtype=torch.float32, device=device) if want_final else None
    status = 0
    if recurrent:
        gdn_prefill_recurrent(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, init, out, fin, max_len)
    else:
        ws = alloc_workspace(tok.T, N, tok.Hqk, tok.Hv, device)
        gdn_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, init, out, fin, max_len, ws)
        if tok.T > 0 and N > 0:
            status = gdn_last_device_status(ws)
    torch.cuda.synchronize()
    return dict(out=bf16_to_numpy(out), final_state=None if fin is None else fin.cpu().numpy().astype(np.float64),
                device_status=status)


def rel_fro(a: np.ndarray, ref: np.ndarray) -> float:
    den = float(np.linalg.norm(ref.ravel()))
    num = float(np.linalg.norm((a - ref).ravel()))
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return num / den


def errors(out: np.ndarray, ref_out: np.ndarray, state: Optional[np.ndarray], ref_state: Optional[np.ndarray]):
    """Whole-tensor norms plus the worst per-head relative Frobenius errors (a single wrong
    head must not hide inside a 32-head average)."""
    e = dict(out_max_abs=float(np.max(np.abs(out - ref_out))) if out.size else 0.0,
             out_rel_fro=rel_fro(out, ref_out), out_nan=int(np.isnan(out).sum()))
    if out.size:
        num = np.linalg.norm(out - ref_out, axis=(0, 2))
        den = np.linalg.norm(ref_out, axis=(0, 2))
        e["out_rel_fro_worst_head"] = float(np.max(num / np.maximum(den, 1e-300)))
    if state is not None and ref_state is not None and state.size:
        e["state_rel_fro"] = rel_fro(state, ref_state)
        e["state_nan"] = int(np.isnan(state).sum())
        num = np.linalg.norm(state - ref_state, axis=(2, 3))
        den = np.linalg.norm(ref_state, axis=(2, 3))
        e["state_rel_fro_worst_head"] = float(np.max(num / np.maximum(den, 1e-300)))
    return e


def assert_close(out, ref_out, state, ref_state, what: str, worst_head_factor: float = 2.0):
    e = errors(out, ref_out, state, ref_state)
    assert e["out_nan"] == 0, "%s: %d NaN outputs (unwritten elements?)" % (what, e["out_nan"])
    assert e["out_max_abs"] <= OUT_MAX_ABS, "%s: out max-abs %.3e" % (what, e["out_max_abs"])
    assert e["out_rel_fro"] <= OUT_REL_FRO, "%s: out rel-Frobenius %.3e" % (what, e["out_rel_fro"])
    if "out_rel_fro_worst_head" in e:
        assert e["out_rel_fro_worst_head"] <= worst_head_factor * OUT_REL_FRO, \
            "%s: worst head out rel-Frobenius %.3e" % (what, e["out_rel_fro_worst_head"])
    if "state_rel_fro" in e:
        assert e["state_nan"] == 0, "%s: %d NaN state elements" % (what, e["state_nan"])
        assert e["state_rel_fro"] <= STATE_REL_FRO, "%s: state rel-Frobenius %.3e" % (what, e["state_rel_fro"])
        assert e["state_rel_fro_worst_head"] <= worst_head_factor * STATE_REL_FRO, \
            "%s: worst head state rel-Frobenius %.3e" % (what, e["state_rel_fro_worst_head"])
    return e
