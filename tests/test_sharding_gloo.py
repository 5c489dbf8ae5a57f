"""The N > 1 path on CPU: world_size-2 gloo ranks shard a decode batch / a varlen batch with
no data-path collective, each computes its slice (with the CPU oracle standing in for the
device here), and the gathered result equals the unsharded one.  Also the max-over-ranks
timing reduction the benchmark uses."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2607_16831_b200.sharding import shard_range, shard_sequences  # noqa: E402


def test_shard_range_partitions_exactly():
    for n in [0, 1, 7, 64, 129]:
        for w in [1, 2, 3, 8]:
            spans = [shard_range(n, w, r) for r in range(w)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_range(4, 2, 2)


def test_shard_sequences_balances_chunks():
    lens = [2048, 1, 64, 65, 1000, 1000, 3, 700]
    parts = shard_sequences(lens, 2)
    assert sorted(parts[0] + parts[1]) == list(range(len(lens)))
    load = [sum((lens[i] + 63) // 64 for i in p) for p in parts]
    assert max(load) <= (4.0 / 3.0) * sum(load) / 2  # the LPT guarantee


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import oracle
    from gdn_inputs import config, make_cu_seqlens

    # decode: global batch of 6, sharded by batch item
    cfg = config("decode_sweep", B=6, Hqk=2, Hv=4, dk=8, dv=8, seed=3)
    tok, st = cfg["tokens"], cfg["state"]
    lo, hi = shard_range(6, world, rank)
    o, s = oracle.decode(tok.q[lo:hi], tok.k[lo:hi], tok.v[lo:hi], tok.g[lo:hi], tok.beta[lo:hi], st[lo:hi], threads=1)
    gathered = [None] * world
    dist.all_gather_object(gathered, (lo, hi, o, s))  # assembling results is outside the data path
    # timing reduction: max over ranks
    t = torch.tensor([1.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    # prefill: sequences assigned by chunk count
    lens = [70, 5, 130, 64]
    parts = shard_sequences(lens, world)
    from gdn_inputs import make_state, make_tokens
    tokp = make_tokens(sum(lens), 2, 4, dk=8, dv=8, seed=4)
    init = make_state(4, 4, 8, 8, seed=4)
    cu = make_cu_seqlens(lens)
    mine = parts[rank]
    idx = np.concatenate([np.arange(cu[i], cu[i + 1]) for i in mine]) if mine else np.zeros(0, dtype=np.int64)
    po, ps = oracle.prefill(tokp.q[idx], tokp.k[idx], tokp.v[idx], tokp.g[idx], tokp.beta[idx],
                            make_cu_seqlens([lens[i] for i in mine]), init[mine], threads=1)
    pg = [None] * world
    dist.all_gather_object(pg, (mine, idx, po, ps))
    if rank == 0:
        q.put((gathered, float(t.item()), pg))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_sharding_matches_unsharded():
    import socket

    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, tmax, pg = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert tmax == 2.0

    import oracle
    from gdn_inputs import config, make_cu_seqlens, make_state, make_tokens

    cfg = config("decode_sweep", B=6, Hqk=2, Hv=4, dk=8, dv=8, seed=3)
    tok = cfg["tokens"]
    ref_o, ref_s = oracle.decode(tok.q, tok.k, tok.v, tok.g, tok.beta, cfg["state"], threads=1)
    for lo, hi, o, s_ in gathered:
        np.testing.assert_array_equal(o, ref_o[lo:hi])
        np.testing.assert_array_equal(s_, ref_s[lo:hi])

    lens = [70, 5, 130, 64]
    tokp = make_tokens(sum(lens), 2, 4, dk=8, dv=8, seed=4)
    init = make_state(4, 4, 8, 8, seed=4)
    ro, rs = oracle.prefill(tokp.q, tokp.k, tokp.v, tokp.g, tokp.beta, make_cu_seqlens(lens), init, threads=1)
    seen = []
    for mine, idx, po, ps in pg:
        seen += list(mine)
        if len(mine):
            np.testing.assert_array_equal(po, ro[idx])
            np.testing.assert_array_equal(ps, rs[mine])
    assert sorted(seen) == [0, 1, 2, 3]
