"""Sequence-parallel prefill across ranks: one long sequence cut into consecutive pieces, one per rank.

The recurrence is affine in the state, so every rank can walk its piece without knowing the
state that enters it (`gdn_prefill_partial`: from the zero state and from the identity), the
ranks exchange one pair of [128 x 128] matrices per value head (`all_gather` of P and H: the
only collective), fold the pairs of the ranks before them into their entering state
(`gdn_state_scan`) and correct their outputs (`gdn_prefill_apply`).  Every rank does the same
amount of work at the same time; nothing is serial except the fold over at most `world` small
matrices.

This module is plumbing: slicing, the collective and the order of the three library calls.  The
arithmetic lives behind a `backend` with three methods so that the host logic can be exercised on
CPU ranks with a stand-in backend; `CudaBackend` is the product path (the C ABI).
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

CHUNK = 64


def split_tokens(total_tokens: int, world_size: int) -> List[Tuple[int, int]]:
    """Consecutive token ranges [lo, hi) per rank: whole 64-token chunks, as even as possible; only
    the last non-empty piece carries a ragged tail (so chunk boundaries inside every piece are the
    ones the unsplit sequence has)."""
    if total_tokens < 0 or world_size <= 0:
        raise ValueError("bad split arguments")
    nchunks = (total_tokens + CHUNK - 1) // CHUNK
    base, rem = divmod(nchunks, world_size)
    out, c = [], 0
    for r in range(world_size):
        n = base + (1 if r < rem else 0)
        lo, hi = min(c * CHUNK, total_tokens), min((c + n) * CHUNK, total_tokens)
        out.append((lo, hi))
        c += n
    return out


class CudaBackend:
    """The three library calls on CUDA tensors (one sequence per call)."""

    def __init__(self, device="cuda"):
        import torch

        self.torch = torch
        self.device = device

    def partial(self, q, k, v, g, beta):
        """-> out0, qt (bf16 [T,Hv,128]), H, P (fp32 [1,Hv,128,128])"""
        import paper_2607_16831_b200 as gdn
        from paper_2607_16831_b200 import harness

        torch = self.torch
        T, Hqk, _ = q.shape
        Hv = v.shape[1]
        cu = torch.tensor([0, T], dtype=torch.int32, device=q.device)
        out0 = torch.empty((T, Hv, 128), dtype=torch.bfloat16, device=q.device)
        qt = torch.empty((T, Hv, 128), dtype=torch.bfloat16, device=q.device)
        H = torch.empty((1, Hv, 128, 128), dtype=torch.float32, device=q.device)
        P = torch.empty_like(H)
        self._ws = harness.alloc_workspace(T, 1, Hqk, Hv, q.device)
        self._cu, self._T = cu, T
        gdn.gdn_prefill_partial(q, k, v, g, beta, cu, out0, qt, H, P, T, self._ws)
        return out0, qt, H, P

    def scan(self, S0, P_list: Sequence, H_list: Sequence):
        """-> (...((S0 P_0 + H_0) P_1 + H_1)...), fp32 [1,Hv,128,128]"""
        import paper_2607_16831_b200 as gdn

        torch = self.torch
        ref = H_list[0] if len(H_list) else S0
        S_out = torch.empty_like(ref)
        if len(P_list) == 0:
            if S0 is not None:
                S_out.copy_(S0)
            else:
                S_out.zero_()
            return S_out
        gdn.gdn_state_scan(S0, torch.stack(list(P_list)).contiguous(), torch.stack(list(H_list)).contiguous(), S_out)
        return S_out

    def apply(self, S_in, qt, out0):
        """-> out0 + S_in qt, in place"""
        import paper_2607_16831_b200 as gdn

        if self._T > 0:
            gdn.gdn_prefill_apply(S_in, qt, out0, self._cu, self._T, self._ws)
        return out0


def finish_piece(backend, rank: int, initial_state, out0, qt, P_all: Sequence, H_all: Sequence):
    """What a rank does after the exchange: fold the pairs of the ranks before it into the state
    entering its piece, correct its outputs, and fold everything into the final state.
    P_all / H_all: the pairs of all ranks in rank order.  Returns (out, final_state)."""
    if rank == 0 and initial_state is None:
        # the first piece of a sequence that starts from the zero state: nothing enters it
        S_in, out = None, out0
    else:
        S_in = backend.scan(initial_state, list(P_all[:rank]), list(H_all[:rank]))
        out = backend.apply(S_in, qt, out0)
    final = backend.scan(S_in, list(P_all[rank:]), list(H_all[rank:]))
    return out, final


def prefill_sequence_parallel(backend, q, k, v, g, beta, initial_state=None, group=None):
    """Collective over `group`: every rank passes ITS piece of the sequence (see split_tokens) and
    the same `initial_state` (fp32 [1,Hv,128,128] or None); returns (out for the local piece,
    final state of the whole sequence).  One all_gather of (P, H) is the only communication."""
    import torch
    import torch.distributed as dist

    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    out0, qt, H, P = backend.partial(q, k, v, g, beta)
    PH = torch.stack([P, H]).contiguous()
    gathered = [torch.empty_like(PH) for _ in range(world)]
    dist.all_gather(gathered, PH, group=group)
    P_all = [x[0] for x in gathered]
    H_all = [x[1] for x in gathered]
    return finish_piece(backend, rank, initial_state, out0, qt, P_all, H_all)
