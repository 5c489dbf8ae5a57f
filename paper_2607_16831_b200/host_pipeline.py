"""Decode from HOST buffers: the batch is cut into slices that move through
host -> device copy, gdn_decode, device -> host copy on a few streams, so that the two copy
engines and the kernel work at the same time.  One step then costs about max(bytes in, bytes
out) / PCIe bandwidth instead of their sum.  Plumbing only: every slice is an ordinary
gdn_decode call on its own rows of the batch (batch items are independent)."""
from __future__ import annotations

from typing import Sequence

import torch

from . import gdn_decode


class HostDecode:
    """Pre-sized device buffers and streams for decode steps whose inputs and outputs live in pinned
    host memory.  `step` enqueues everything and returns; the caller's current stream is made to wait
    for the last copy, so synchronising that stream (or the device) completes the step."""

    def __init__(self, B: int, Hqk: int, Hv: int, slices: int = 8, streams: int = 3, device="cuda"):
        self.B, self.Hqk, self.Hv = B, Hqk, Hv
        slices = max(1, min(slices, B))
        base, rem = divmod(B, slices)
        self.spans, lo = [], 0
        for i in range(slices):
            hi = lo + base + (1 if i < rem else 0)
            self.spans.append((lo, hi))
            lo = hi
        dev = torch.device(device)
        self.q = torch.empty((B, Hqk, 128), dtype=torch.bfloat16, device=dev)
        self.k = torch.empty_like(self.q)
        self.v = torch.empty((B, Hv, 128), dtype=torch.bfloat16, device=dev)
        self.out = torch.empty_like(self.v)
        self.g = torch.empty((B, Hv), dtype=torch.float32, device=dev)
        self.beta = torch.empty_like(self.g)
        self.s_in = torch.empty((B, Hv, 128, 128), dtype=torch.float32, device=dev)
        self.s_out = torch.empty_like(self.s_in)
        self.streams = [torch.cuda.Stream(device=dev) for _ in range(max(1, streams))]
        self.start = torch.cuda.Event()
        self.done = [torch.cuda.Event() for _ in self.streams]

    def step(self, h_q, h_k, h_v, h_g, h_beta, h_state_in, h_state_out, h_out) -> None:
        """All arguments are pinned host tensors shaped like the device tensors (bf16 tensors may be
        passed as int16 views).  h_state_in may be None: the state already on the device (the previous
        step's output, see `swap`) is used and not copied back unless h_state_out is given."""
        main = torch.cuda.current_stream()
        view = lambda h, d: h if h.dtype == d.dtype else h.view(d.dtype)
        # the token inputs are small: whole batch at once on the caller's stream, then the slices start
        for h, d in ((h_q, self.q), (h_k, self.k), (h_v, self.v), (h_g, self.g), (h_beta, self.beta)):
            d.copy_(view(h, d), non_blocking=True)
        self.start.record(main)
        for i, (lo, hi) in enumerate(self.spans):
            st = self.streams[i % len(self.streams)]
            if i < len(self.streams):
                st.wait_event(self.start)
            with torch.cuda.stream(st):
                if h_state_in is not None:
                    self.s_in[lo:hi].copy_(h_state_in[lo:hi], non_blocking=True)
                gdn_decode(self.q[lo:hi], self.k[lo:hi], self.v[lo:hi], self.g[lo:hi], self.beta[lo:hi],
                           self.s_in[lo:hi], self.s_out[lo:hi], self.out[lo:hi], stream=st)
                if h_state_out is not None:
                    h_state_out[lo:hi].copy_(self.s_out[lo:hi], non_blocking=True)
        for st, ev in zip(self.streams, self.done):
            ev.record(st)
            main.wait_event(ev)
        # outputs are small as well: one copy after the last slice
        view(h_out, self.out).copy_(self.out, non_blocking=True)

    def swap(self) -> None:
        """Makes this step's output state the next step's input (state kept on the device)."""
        self.s_in, self.s_out = self.s_out, self.s_in
