"""Running the stack on batches that live in pinned host memory.

A step has three legs -- host->device copy of the input, the stack's kernels, device->host copy of the result --
and on a PCIe-attached GPU the two copies together cost more than the kernels.  HostPipeline keeps `depth` steps in
flight on three streams (copy-in, compute, copy-out) so that the legs of neighbouring steps overlap: while step i
computes, step i+1 is being uploaded and step i-1 downloaded.  Every step still moves its own input and its own
result; only the waiting is shared.  Nothing here computes: the kernels are those of GsitStack.forward, replayed
from one CUDA graph per slot."""
from __future__ import annotations

import torch

from . import binding as B
from .stack import GsitStack


class HostPipeline:
    def __init__(self, stack: GsitStack, x_shape, with_valid_len: bool = True, depth: int = 2, device=None):
        """x_shape = (B, L, d) of every batch; with_valid_len: batches come with an int32 [B, 3] array of valid lengths."""
        assert depth >= 1
        self.stack, self.depth = stack, depth
        dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        Bn, L, d = x_shape
        self.x_dev = [torch.empty((Bn, L, d), dtype=torch.float32, device=dev) for _ in range(depth)]
        self.vl_dev = [torch.zeros((Bn, 3), dtype=torch.int32, device=dev) if with_valid_len else None for _ in range(depth)]
        self.y_dev = [None] * depth      # per-slot copy of the stack's output buffer (the stack reuses its own)
        self.graphs = [None] * depth
        self.s_in, self.s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        mk = lambda: [torch.cuda.Event() for _ in range(depth)]
        self.ev_in, self.ev_comp, self.ev_out = mk(), mk(), mk()
        self.n = 0

    def _capture(self, slot):
        # eager once (allocates the stack's buffers, loads modules), then the same calls into a graph
        y = self.stack.forward(self.x_dev[slot], self.vl_dev[slot])
        self.y_dev[slot] = torch.empty_like(y)
        torch.cuda.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):  # the stack delivers straight into the slot's buffer where its last kernel can
            self.stack.forward(self.x_dev[slot], self.vl_dev[slot], out=self.y_dev[slot])
        self.graphs[slot] = gr

    def step(self, x_host, y_host, valid_host=None):
        """Queues one step: x_host (pinned float32 [B, L, d]) -> y_host (pinned float32 [B, L, 2d]).  Returns at once;
        y_host is complete after wait() (or after `depth` further steps)."""
        i, slot = self.n, self.n % self.depth
        if self.graphs[slot] is None:
            if self.vl_dev[slot] is not None:
                assert valid_host is not None
                self.vl_dev[slot].copy_(valid_host)
            self._capture(slot)
        main = torch.cuda.current_stream()
        with torch.cuda.stream(self.s_in):
            if i >= self.depth:
                self.s_in.wait_event(self.ev_comp[slot])      # the kernels of step i - depth have read this slot
            self.x_dev[slot].copy_(x_host, non_blocking=True)
            if self.vl_dev[slot] is not None and valid_host is not None:
                self.vl_dev[slot].copy_(valid_host, non_blocking=True)
            self.ev_in[slot].record(self.s_in)
        main.wait_event(self.ev_in[slot])
        if i >= self.depth:
            main.wait_event(self.ev_out[slot])                # the result of step i - depth has left this slot
        self.graphs[slot].replay()
        self.ev_comp[slot].record(main)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_comp[slot])
            y_host.copy_(self.y_dev[slot], non_blocking=True)
            self.ev_out[slot].record(self.s_out)
        self.n += 1

    def wait(self):
        """Blocks until every queued step has delivered its result, then reads the library's device status word: a
        bounded device-side wait that ran out (the results are then invalid) raises GsitError instead of passing silently."""
        self.s_out.synchronize()
        torch.cuda.current_stream().synchronize()
        code, flags = B.last_device_status()
        if code != 0:
            raise B.GsitError(code, f"HostPipeline: device status flags {flags:#x}")
