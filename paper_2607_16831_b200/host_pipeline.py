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
    host memory.  `step` enqueues everything on internal streams and returns; the caller's current
    stream is made to wait for the step's last copy, so synchronising that stream (or the device)
    completes the step.  Successive steps overlap: the copies back to the host of one step run while the
    next step's inputs come in.  What orders the reuse of the device buffers: a slice keeps to one stream
    (its state buffers); the token buffers are rewritten only after the previous step's kernels; the
    output buffer alternates between two, each rewritten only after its copy to the host."""

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
        self.outs = [torch.empty_like(self.v), torch.empty_like(self.v)]
        self.g = torch.empty((B, Hv), dtype=torch.float32, device=dev)
        self.beta = torch.empty_like(self.g)
        self.s_in = torch.empty((B, Hv, 128, 128), dtype=torch.float32, device=dev)
        self.s_out = torch.empty_like(self.s_in)
        self.streams = [torch.cuda.Stream(device=dev) for _ in range(max(1, streams))]
        self.used = min(len(self.streams), len(self.spans))
        self.aux_in = torch.cuda.Stream(device=dev)   # the small whole-batch copy of the tokens
        self.aux_out = torch.cuda.Stream(device=dev)  # the small whole-batch copy of the outputs
        self.tokens_in = torch.cuda.Event()
        self.kernels = [torch.cuda.Event() for _ in self.streams]
        self.done = [torch.cuda.Event() for _ in self.streams]
        self.out_done = [torch.cuda.Event(), torch.cuda.Event()]
        self.steps = 0

    def step(self, h_q, h_k, h_v, h_g, h_beta, h_state_in, h_state_out, h_out) -> None:
        """All arguments are pinned host tensors shaped like the device tensors (bf16 tensors may be
        passed as int16 views).  h_state_in may be None: the state already on the device (the previous
        step's output, see `swap`) is used and not copied back unless h_state_out is given."""
        main = torch.cuda.current_stream()
        view = lambda h, d: h if h.dtype == d.dtype else h.view(d.dtype)
        b = self.steps & 1
        out = self.outs[b]
        # The inputs are host memory, so nothing has to wait for what the caller's stream holds (which
        # includes the end of the previous step): the internal streams carry on from their own last work.
        if self.steps > 0:
            for j in range(self.used):
                self.aux_in.wait_event(self.kernels[j])  # the previous step's kernels read the token buffers
        with torch.cuda.stream(self.aux_in):
            # the token inputs are small: whole batch at once
            for h, d in ((h_q, self.q), (h_k, self.k), (h_v, self.v), (h_g, self.g), (h_beta, self.beta)):
                d.copy_(view(h, d), non_blocking=True)
            self.tokens_in.record(self.aux_in)
        for i, (lo, hi) in enumerate(self.spans):
            j = i % len(self.streams)
            st = self.streams[j]
            with torch.cuda.stream(st):
                if h_state_in is not None:
                    self.s_in[lo:hi].copy_(h_state_in[lo:hi], non_blocking=True)
                if i < len(self.streams):  # the stream's first kernel of this step (the later ones follow it)
                    st.wait_event(self.tokens_in)
                    if self.steps >= 2:
                        st.wait_event(self.out_done[b])  # this output buffer's last copy to the host
                gdn_decode(self.q[lo:hi], self.k[lo:hi], self.v[lo:hi], self.g[lo:hi], self.beta[lo:hi],
                           self.s_in[lo:hi], self.s_out[lo:hi], out[lo:hi], stream=st)
                self.kernels[j].record(st)  # the last one recorded on a stream stands
                if h_state_out is not None:
                    h_state_out[lo:hi].copy_(self.s_out[lo:hi], non_blocking=True)
        # outputs are small as well: one copy once every kernel of the step is done (not its state copies)
        for j in range(self.used):
            self.aux_out.wait_event(self.kernels[j])
        with torch.cuda.stream(self.aux_out):
            view(h_out, out).copy_(out, non_blocking=True)
            self.out_done[b].record(self.aux_out)
        for j in range(self.used):
            self.done[j].record(self.streams[j])
            main.wait_event(self.done[j])
        main.wait_event(self.out_done[b])
        self.steps += 1

    def swap(self) -> None:
        """Makes this step's output state the next step's input (state kept on the device)."""
        self.s_in, self.s_out = self.s_out, self.s_in
