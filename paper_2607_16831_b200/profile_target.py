"""Runs a few calls of one entry point on a seeded workload, for `ncu` and for quick timing.

  python -m paper_2607_16831_b200.profile_target --workload decode --B 64 --calls 3
  python -m paper_2607_16831_b200.profile_target --workload prefill_long --T 1024 --calls 2
  python -m paper_2607_16831_b200.profile_target --workload prefill_varlen --calls 2
  python -m paper_2607_16831_b200.profile_target --workload prefill_short --calls 2   (256 x 64 tokens, 4/8 heads)
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="decode", choices=["decode", "prefill_long", "prefill_varlen", "prefill_tiny", "prefill_short"])
    ap.add_argument("--B", type=int, default=64)
    ap.add_argument("--T", type=int, default=4096)
    ap.add_argument("--Hqk", type=int, default=16)
    ap.add_argument("--Hv", type=int, default=32)
    ap.add_argument("--calls", type=int, default=3)
    ap.add_argument("--initial", action="store_true")
    ap.add_argument("--recurrent", action="store_true")
    args = ap.parse_args()

    import torch

    import paper_2607_16831_b200 as gdn
    from gdn_inputs import config
    from paper_2607_16831_b200 import harness

    torch.cuda.set_device(0)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.calls)]
    if args.workload == "decode":
        cfg = config("decode_b64", B=args.B)
        d = harness.to_device(cfg["tokens"])
        s_in = torch.from_numpy(cfg["state"]).cuda()
        bufs = [(s_in.clone(), torch.empty_like(s_in)) for _ in range(max(2, min(args.calls, 4)))]
        out = torch.empty((args.B, 32, 128), dtype=torch.bfloat16, device="cuda")
        for i in range(args.calls):
            a, b = bufs[i % len(bufs)]
            ev[i][0].record()
            gdn.gdn_decode(d["q"], d["k"], d["v"], d["g"], d["beta"], a, b, out)
            ev[i][1].record()
    else:
        if args.workload == "prefill_short":
            # many short sequences at the contest's head counts: 256 sequences of 64 tokens, 4 key / 8 value heads
            from gdn_inputs import make_cu_seqlens, make_state, make_tokens
            lengths = [64] * 256
            cfg = dict(tokens=make_tokens(sum(lengths), 4, 8, seed=0), cu_seqlens=make_cu_seqlens(lengths),
                       initial_state=make_state(len(lengths), 8, seed=0))
        else:
            over = {"T": args.T, "initial": args.initial} if args.workload == "prefill_long" else {}
            cfg = config(args.workload, Hqk=args.Hqk, Hv=args.Hv, **over)
        tok = cfg["tokens"]
        d = harness.to_device(tok)
        cu_np = np.asarray(cfg["cu_seqlens"], dtype=np.int32)
        cu = torch.from_numpy(cu_np).cuda()
        N = len(cu_np) - 1
        init = None if cfg["initial_state"] is None else torch.from_numpy(cfg["initial_state"]).cuda()
        out = torch.empty((tok.T, tok.Hv, 128), dtype=torch.bfloat16, device="cuda")
        fin = torch.empty((N, tok.Hv, 128, 128), dtype=torch.float32, device="cuda")
        ws = harness.alloc_workspace(tok.T, N, tok.Hqk, tok.Hv)
        for i in range(args.calls):
            ev[i][0].record()
            if args.recurrent:
                gdn.gdn_prefill_recurrent(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, init, out, fin,
                                          int(np.max(np.diff(cu_np))))
            else:
                gdn.gdn_prefill(d["q"], d["k"], d["v"], d["g"], d["beta"], cu, init, out, fin,
                                int(np.max(np.diff(cu_np))), ws)
            ev[i][1].record()
        torch.cuda.synchronize()
        if not args.recurrent:
            assert gdn.gdn_last_device_status(ws) == 0
    torch.cuda.synchronize()
    print("call us:", ["%.1f" % (a.elapsed_time(b) * 1e3) for a, b in ev])


if __name__ == "__main__":
    main()
