"""Sequence-parallel prefill, host logic on CPU: world_size-2 (and 3) gloo ranks each take a piece
of one sequence, exchange (P, H) with one all_gather and finish their piece.  The arithmetic
behind the three backend calls is the fp64 oracle here (zero-state run, identity-state run with
v = 0, plain matrix products), so the gathered result must equal the unsplit oracle run to
rounding: this pins the slicing, the order of the fold and the rank bookkeeping."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2607_16831_b200.sequence_parallel import finish_piece, prefill_sequence_parallel, split_tokens  # noqa: E402


def test_split_tokens_covers_the_sequence_on_chunk_boundaries():
    for T in [0, 1, 63, 64, 65, 1000, 4096]:
        for w in [1, 2, 3, 8]:
            spans = split_tokens(T, w)
            assert spans[0][0] == 0 and spans[-1][1] == T
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            assert all(lo % 64 == 0 for lo, hi in spans if hi > lo)
            chunks = [(hi - lo + 63) // 64 for lo, hi in spans]
            assert max(chunks) - min(chunks) <= 1
    with pytest.raises(ValueError):
        split_tokens(10, 0)


class OracleBackend:
    """fp64 stand-in for the CUDA backend: tensors are CPU float64 / uint16 numpy-backed."""

    def __init__(self, dk, dv):
        import oracle

        self.oracle, self.dk, self.dv = oracle, dk, dv

    def partial(self, q, k, v, g, beta):
        o = self.oracle
        T, Hv = v.shape[0], v.shape[1]
        cu = np.array([0, T], dtype=np.int32)
        out0, H = o.prefill(q, k, v, g, beta, cu, None, threads=1)
        eye = np.broadcast_to(np.eye(self.dk, dtype=np.float32), (1, Hv, self.dk, self.dk)).copy()
        qt, P = o.prefill(q, k, np.zeros_like(v), g, beta, cu, eye, threads=1)
        return torch.from_numpy(out0), torch.from_numpy(qt), torch.from_numpy(H), torch.from_numpy(P)

    def scan(self, S0, P_list, H_list):
        ref = H_list[0] if len(H_list) else S0
        S = torch.zeros_like(ref) if S0 is None else S0.clone().to(torch.float64)
        for P, H in zip(P_list, H_list):
            S = S @ P + H
        return S

    def apply(self, S_in, qt, out0):
        # out[t,h,:] += S_in[h] qt[t,h,:]
        return out0 + torch.einsum("hvk,thk->thv", S_in[0], qt)


def _problem(T=300, Hqk=2, Hv=4, d=8, seed=5):
    from gdn_inputs import make_state, make_tokens

    tok = make_tokens(T, Hqk, Hv, dk=d, dv=d, seed=seed, gate_mean=4.0)
    init = make_state(1, Hv, d, d, seed=seed)
    return tok, init


def _worker(rank, world, port, queue):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    tok, init = _problem()
    lo, hi = split_tokens(tok.T, world)[rank]
    be = OracleBackend(8, 8)
    out, fin = prefill_sequence_parallel(be, tok.q[lo:hi], tok.k[lo:hi], tok.v[lo:hi], tok.g[lo:hi], tok.beta[lo:hi],
                                         torch.from_numpy(init).to(torch.float64))
    got = [None] * world
    dist.all_gather_object(got, (lo, hi, out.numpy(), fin.numpy()))
    if rank == 0:
        queue.put(got)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_ranks_reassemble_the_unsplit_result(world):
    import oracle

    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    queue = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, queue)) for r in range(world)]
    for p in procs:
        p.start()
    got = queue.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    tok, init = _problem()
    ref_o, ref_s = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, np.array([0, tok.T], dtype=np.int32), init, threads=1)
    out = np.zeros_like(ref_o)
    for lo, hi, o, fin in got:
        out[lo:hi] = o
        np.testing.assert_allclose(fin, ref_s, rtol=0, atol=1e-12)  # every rank ends with the same final state
    np.testing.assert_allclose(out, ref_o, rtol=0, atol=1e-12)


def test_finish_piece_uses_only_earlier_ranks_for_the_entering_state():
    """With P = 0 published by an earlier rank, nothing before that rank can leak through."""
    be = OracleBackend(8, 8)
    rng = np.random.default_rng(0)
    H = [torch.from_numpy(rng.standard_normal((1, 2, 8, 8))) for _ in range(3)]
    P = [torch.from_numpy(rng.standard_normal((1, 2, 8, 8))) for _ in range(3)]
    P[1] = torch.zeros_like(P[1])
    qt = torch.from_numpy(rng.standard_normal((5, 2, 8)))
    out0 = torch.zeros((5, 2, 8), dtype=torch.float64)
    S0 = torch.from_numpy(rng.standard_normal((1, 2, 8, 8)))
    out, fin = finish_piece(be, 2, S0, out0, qt, P, H)
    np.testing.assert_allclose(out.numpy(), np.einsum("hvk,thk->thv", H[1][0].numpy(), qt.numpy()), atol=1e-12)
    np.testing.assert_allclose(fin.numpy(), (H[1] @ P[2] + H[2]).numpy(), atol=1e-12)


def test_finish_piece_from_the_zero_state():
    """initial_state = None: the first piece has nothing to correct, later pieces start from the zero state."""
    be = OracleBackend(8, 8)
    rng = np.random.default_rng(1)
    H = [torch.from_numpy(rng.standard_normal((1, 2, 8, 8))) for _ in range(3)]
    P = [torch.from_numpy(rng.standard_normal((1, 2, 8, 8))) for _ in range(3)]
    qt = torch.from_numpy(rng.standard_normal((5, 2, 8)))
    out0 = torch.from_numpy(rng.standard_normal((5, 2, 8)))
    want_final = ((H[0] @ P[1] + H[1]) @ P[2] + H[2]).numpy()
    out, fin = finish_piece(be, 0, None, out0, qt, P, H)
    np.testing.assert_array_equal(out.numpy(), out0.numpy())
    np.testing.assert_allclose(fin.numpy(), want_final, atol=1e-12)
    out, fin = finish_piece(be, 1, None, out0, qt, P, H)
    np.testing.assert_allclose(out.numpy(), out0.numpy() + np.einsum("hvk,thk->thv", H[0][0].numpy(), qt.numpy()), atol=1e-12)
    np.testing.assert_allclose(fin.numpy(), want_final, atol=1e-12)
