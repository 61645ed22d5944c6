"""The GsiT fusion stack as a sequence of library calls (Eq. "All-Modal-In-One fusion"): a forward-ring
encoder and a backward-ring encoder, each with its own weights, both starting from the same input; their
outputs side by side on the feature axis (width 2d); then the intra-modal encoder on that.  Only
sequencing and buffer reuse happen here -- each layer is one gsit_im_layer_fwd call, and the feature
concat costs nothing because the last layer of each ring writes its half of the [B, L, 2d] buffer.

The two rings share nothing but their input, so they are issued on two CUDA streams (fork after the
input is ready, join before the intra encoder): the CTAs of one ring fill the SM slots that the last
wave of the other leaves empty.  Each ring has its own workspace and ping-pong buffers."""
from __future__ import annotations

import torch

from . import binding as B


class GsitStack:
    def __init__(self, fwd_layers, bwd_layers, intra_layers, seg_len, heads, intra_heads, ln_eps=1e-5, head=None,
                 concurrent_rings=True):
        """head: optional (w_f, b_f) of the read-out X_m = f(|| Split(.)[-1]); see read_out().
        concurrent_rings: issue the forward and the backward ring on two streams (False: one after the other)."""
        self.head = head
        self.concurrent_rings = concurrent_rings
        self._side = None  # second stream and fork/join events, created on first use
        self.fwd, self.bwd, self.intra = list(fwd_layers), list(bwd_layers), list(intra_layers)
        self.seg_len, self.heads, self.intra_heads, self.ln_eps = tuple(seg_len), heads, intra_heads, ln_eps
        self._bufs = None

    def _buffers(self, x, valid_len):
        Bn, L, d = x.shape
        key = (Bn, L, d, x.device)
        if self._bufs is None or self._bufs[0] != key:
            code = B._dtype_code(self.fwd[0]["w_qkv"].dtype)
            sh1 = B.make_shape(Bn, self.seg_len, d, self.heads, valid_len, code, B.PHASE_INTER_FWD)
            sh2 = B.make_shape(Bn, self.seg_len, 2 * d, self.intra_heads, valid_len, code, B.PHASE_INTRA)
            need = B.workspace_bytes(sh1, B.CALL_LAYER, self.fwd[0]["w_1"].shape[0])
            if self.intra:
                need = max(need, B.workspace_bytes(sh2, B.CALL_LAYER, self.intra[0]["w_1"].shape[0]))
            f32 = dict(dtype=torch.float32, device=x.device)
            self._bufs = (key, torch.empty(need, dtype=torch.uint8, device=x.device),
                          torch.empty((Bn, L, d), **f32), torch.empty((Bn, L, d), **f32),
                          torch.empty((Bn, L, 2 * d), **f32), torch.empty((Bn, L, 2 * d), **f32),
                          torch.empty(need, dtype=torch.uint8, device=x.device),
                          torch.empty((Bn, L, d), **f32), torch.empty((Bn, L, d), **f32))
        return self._bufs[1:]

    def _ring(self, x, layers, phase, half, c0, ws, ping, valid_len):
        d = x.shape[2]
        cur = x
        for i, w in enumerate(layers):
            dst = c0[:, :, half * d:(half + 1) * d] if i == len(layers) - 1 else ping[i % 2]
            B.im_layer_fwd(cur, w, self.seg_len, self.heads, valid_len, phase, ln_eps=self.ln_eps, out=dst, workspace=ws)
            cur = dst

    def forward(self, x, valid_len=None):
        """x float32 [B, L, d] -> float32 [B, L, 2d].  The result lives in a buffer owned by this object."""
        ws, t0, t1, c0, c1, ws_b, u0, u1 = self._buffers(x, valid_len)
        if self.concurrent_rings and self.fwd and self.bwd:
            if self._side is None:
                self._side = (torch.cuda.Stream(device=x.device), torch.cuda.Event(), torch.cuda.Event())
            side, fork, join = self._side
            main = torch.cuda.current_stream(x.device)
            fork.record(main)
            side.wait_event(fork)
            with torch.cuda.stream(side):
                self._ring(x, self.bwd, B.PHASE_INTER_BWD, 1, c0, ws_b, [u0, u1], valid_len)
                join.record(side)
            x.record_stream(side)
            if valid_len is not None:
                valid_len.record_stream(side)
            self._ring(x, self.fwd, B.PHASE_INTER_FWD, 0, c0, ws, [t0, t1], valid_len)
            main.wait_event(join)
        else:
            self._ring(x, self.fwd, B.PHASE_INTER_FWD, 0, c0, ws, [t0, t1], valid_len)
            self._ring(x, self.bwd, B.PHASE_INTER_BWD, 1, c0, ws, [t0, t1], valid_len)
        cur, ping = c0, [c1, c0]
        for i, w in enumerate(self.intra):
            dst = ping[i % 2]
            B.im_layer_fwd(cur, w, self.seg_len, self.intra_heads, valid_len, B.PHASE_INTRA, ln_eps=self.ln_eps,
                           out=dst, workspace=ws)
            cur = dst
        return cur

    def read_out(self, c, valid_len=None):
        """X_m = f(|| Split(c)[-1]): last real step of each modality of the stack output c [B, L, 2d], through the linear
        map given as `head` -> float32 [B, out_features] (one gsit_stack_head_fwd call)."""
        assert self.head is not None, "no read-out weights were given"
        w_f, b_f = self.head
        return B.stack_head_fwd(c, w_f, b_f, self.seg_len, valid_len)
