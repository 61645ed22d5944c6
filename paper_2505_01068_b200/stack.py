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
                 concurrent_rings=True, batch_chunks=1, intra_halves=True,
                 packed=True, paired_rings=True):
        """head: optional (w_f, b_f) of the read-out X_m = f(|| Split(.)[-1]); see read_out().
        concurrent_rings: issue independent work on several streams (False: every launch on the caller's stream, whole
        batch per launch).  batch_chunks: with concurrent issue, the batch is cut into this many groups of samples, each
        with its own pair of streams; samples never interact, so the result does not depend on it.  (At B = 64, L = 1050
        one chunk is fastest: the persistent fused kernels pay their per-CTA set-up once per launch.)
        intra_halves: with concurrent issue, the intra encoder runs on the two halves of the batch on the two streams, so
        that the attention of one half overlaps the fused layer halves of the other (0.794 -> 0.784 ms at that shape
        with paired rings; three or four parts are slower again).
        packed: when valid lengths are given (and the layers are bf16 at widths the tcgen05 fused kernels cover), the
        stack works on the packed row layout: the real rows are gathered once, every layer runs on them only, and the
        result is scattered back with +0 in the padded positions.  The row-wise parts of the layers then do no work
        for padding (24 % of the rows at the benchmark's lengths).  The plan of where each segment starts is made on the
        device, so a captured forward stays valid when the lengths change.
        paired_rings: (packed layout, rings of equal depth) the forward-ring and backward-ring layers of equal depth go
        through one gsit_im_layer_pair_fwd call each -- three launches per depth for both rings, on one stream, each
        starting under the tail of the one before it -- instead of two streams of three launches (0.784 against
        0.789 ms at that shape).  False: one stream per ring."""
        self.head = head
        self.concurrent_rings = concurrent_rings
        self.batch_chunks = max(1, int(batch_chunks))
        self.intra_halves = bool(intra_halves)
        self.packed = bool(packed)
        self.paired_rings = bool(paired_rings)
        self.fwd, self.bwd, self.intra = list(fwd_layers), list(bwd_layers), list(intra_layers)
        self.seg_len, self.heads, self.intra_heads, self.ln_eps = tuple(seg_len), heads, intra_heads, ln_eps
        self._bufs = None
        self._lanes = None  # streams and events of the concurrent issue, created on first use
        self._ring_done = None

    def _chunks(self, Bn):
        nch = min(self.batch_chunks, Bn) if (self.concurrent_rings and self.fwd and self.bwd) else 1
        q, r = divmod(Bn, nch)
        out, lo = [], 0
        for c in range(nch):
            hi = lo + q + (1 if c < r else 0)
            out.append(slice(lo, hi))
            lo = hi
        return out

    def _buffers(self, x, valid_len):
        Bn, L, d = x.shape
        chunks = self._chunks(Bn)
        key = (Bn, L, d, x.device, len(chunks))
        if self._bufs is None:
            self._bufs = {}
        if key not in self._bufs:
            code = B._dtype_code(self.fwd[0]["w_qkv"].dtype)
            ws = []
            for sl in chunks:  # two workspaces per chunk of the batch: one per ring (the intra encoder reuses the first)
                n = sl.stop - sl.start
                vl = None if valid_len is None else valid_len[sl]
                sh1 = B.make_shape(n, self.seg_len, d, self.heads, vl, code, B.PHASE_INTER_FWD)
                need = B.workspace_bytes(sh1, B.CALL_LAYER, self.fwd[0]["w_1"].shape[0])
                if self.intra:
                    sh2 = B.make_shape(n, self.seg_len, 2 * d, self.intra_heads, vl, code, B.PHASE_INTRA)
                    need = max(need, B.workspace_bytes(sh2, B.CALL_LAYER, self.intra[0]["w_1"].shape[0]))
                ws.append([torch.empty(need, dtype=torch.uint8, device=x.device) for _ in range(2)])
            f32 = dict(dtype=torch.float32, device=x.device)
            self._bufs[key] = (ws, [torch.empty((Bn, L, d), **f32) for _ in range(4)],
                               torch.empty((Bn, L, 2 * d), **f32), torch.empty((Bn, L, 2 * d), **f32))
        return (chunks,) + self._bufs[key]

    def _ring(self, x, layers, phase, half, c0, ws, ping, valid_len):
        d = x.shape[2]
        cur = x
        for i, w in enumerate(layers):
            dst = c0[:, :, half * d:(half + 1) * d] if i == len(layers) - 1 else ping[i % 2]
            B.im_layer_fwd(cur, w, self.seg_len, self.heads, valid_len, phase, ln_eps=self.ln_eps, out=dst, workspace=ws)
            cur = dst

    def _intra(self, c0, c1, ws, valid_len):
        cur, ping = c0, [c1, c0]
        for i, w in enumerate(self.intra):
            dst = ping[i % 2]
            B.im_layer_fwd(cur, w, self.seg_len, self.intra_heads, valid_len, B.PHASE_INTRA, ln_eps=self.ln_eps,
                           out=dst, workspace=ws)
            cur = dst
        return len(self.intra) % 2  # 1: the result is in c1, 0: in c0

    def _packed_buffers(self, x, valid_len):
        Bn, L, d = x.shape
        key = ("packed", Bn, L, d, x.device)
        if self._bufs is None:
            self._bufs = {}
        if key not in self._bufs:
            cap = Bn * L + 128  # always enough: the real rows plus the alignment of the second half's first row
            code = B._dtype_code(self.fwd[0]["w_qkv"].dtype)
            plan = torch.zeros(3 * Bn + 1, dtype=torch.int32, device=x.device)
            sh1 = B.make_shape(Bn, self.seg_len, d, self.heads, valid_len, code, B.PHASE_INTER_FWD, row_start=plan, capacity=cap)
            need = B.workspace_bytes(sh1, B.CALL_LAYER, self.fwd[0]["w_1"].shape[0])
            if self.intra:
                sh2 = B.make_shape(Bn, self.seg_len, 2 * d, self.intra_heads, valid_len, code, B.PHASE_INTRA, row_start=plan,
                                   capacity=cap)
                need = max(need, B.workspace_bytes(sh2, B.CALL_LAYER, self.intra[0]["w_1"].shape[0]))
            f32 = dict(dtype=torch.float32, device=x.device)
            ws_all = torch.empty(2 * need, dtype=torch.uint8, device=x.device)   # one per ring, or both for a paired call
            self._ws_pair = ws_all
            self._bufs[key] = (cap, plan, [ws_all[:need], ws_all[need:]],
                               [torch.zeros((cap, d), **f32) for _ in range(5)],
                               torch.zeros((cap, 2 * d), **f32), torch.zeros((cap, 2 * d), **f32),
                               torch.empty((Bn, L, 2 * d), **f32))
        return self._bufs[key]

    def _forward_packed(self, x, valid_len, out=None):
        cap, plan, ws, t, c0, c1, y = self._packed_buffers(x, valid_len)
        if out is not None:
            y = out
        Bn, L, d = x.shape
        conc = self.concurrent_rings and self.fwd and self.bwd
        halves = conc and self.intra_halves and self.intra and Bn >= 2
        mid = Bn // 2
        B.plan_rows(valid_len, self.seg_len, mid if halves else 0, out=plan)
        xp = B.pack_rows(x, t[4], self.seg_len, valid_len, plan)

        def ring(layers, phase, half, w_s, ping):
            cur = xp
            for i, w in enumerate(layers):
                dst = c0[:, half * d:(half + 1) * d] if i == len(layers) - 1 else ping[i % 2]
                B.im_layer_fwd(cur, w, self.seg_len, self.heads, valid_len, phase, ln_eps=self.ln_eps, out=dst, workspace=w_s,
                               row_start=plan)
                cur = dst

        def intra(lo, hi, w_s):  # samples lo .. hi - 1: their rows of the packed matrices are addressed through the plan
            cur, ping = c0, [c1, c0]
            for i, w in enumerate(self.intra):
                dst = ping[i % 2]
                B.im_layer_fwd(cur, w, self.seg_len, self.intra_heads, valid_len[lo:hi], B.PHASE_INTRA, ln_eps=self.ln_eps,
                               out=dst, workspace=w_s, row_start=plan[3 * lo:])
                cur = dst
            return cur

        paired = self.paired_rings and len(self.fwd) == len(self.bwd) and len(self.fwd) > 0

        def rings_paired():
            cur_a = cur_b = xp
            n = len(self.fwd)
            for i in range(n):
                last = i == n - 1
                dst_a = c0[:, 0:d] if last else t[i % 2]
                dst_b = c0[:, d:2 * d] if last else t[2 + i % 2]
                B.im_layer_pair_fwd(cur_a, cur_b, self.fwd[i], self.bwd[i], self.seg_len, self.heads, valid_len, B.PHASE_INTER_FWD,
                                    B.PHASE_INTER_BWD, ln_eps=self.ln_eps, out_a=dst_a, out_b=dst_b, workspace=self._ws_pair,
                                    row_start=plan)
                cur_a, cur_b = dst_a, dst_b

        if paired and not (halves and self.intra):
            rings_paired()
            res = intra(0, Bn, ws[0]) if self.intra else c0
        elif paired:
            # both rings on the caller's stream, then the intra encoder on the two halves of the batch on two streams
            rings_paired()
            if self._lanes is None:
                dev = x.device
                self._lanes = ([torch.cuda.Stream(device=dev) for _ in range(2)], torch.cuda.Event(),
                               [torch.cuda.Event() for _ in range(2)])
                self._ring_done = [torch.cuda.Event()]
            streams, fork, done = self._lanes
            main = torch.cuda.current_stream(x.device)
            fork.record(main)
            for si, (lo, hi) in enumerate(((0, mid), (mid, Bn))):
                streams[si].wait_event(fork)
                with torch.cuda.stream(streams[si]):
                    r_ = intra(lo, hi, ws[si])
                    done[si].record(streams[si])
                if si == 0:
                    res = r_
            for si in range(2):
                main.wait_event(done[si])
                x.record_stream(streams[si])
                valid_len.record_stream(streams[si])
        elif not conc:
            ring(self.fwd, B.PHASE_INTER_FWD, 0, ws[0], t[0:2])
            ring(self.bwd, B.PHASE_INTER_BWD, 1, ws[0], t[0:2])
            res = intra(0, Bn, ws[0]) if self.intra else c0
        else:
            if self._lanes is None:
                dev = x.device
                self._lanes = ([torch.cuda.Stream(device=dev) for _ in range(2)], torch.cuda.Event(),
                               [torch.cuda.Event() for _ in range(2)])
                self._ring_done = [torch.cuda.Event()]
            streams, fork, done = self._lanes
            s_f, s_b = streams[0], streams[1]
            main = torch.cuda.current_stream(x.device)
            fork.record(main)
            s_f.wait_event(fork)
            s_b.wait_event(fork)
            with torch.cuda.stream(s_b):
                ring(self.bwd, B.PHASE_INTER_BWD, 1, ws[1], t[2:4])
                done[1].record(s_b)
            with torch.cuda.stream(s_f):
                ring(self.fwd, B.PHASE_INTER_FWD, 0, ws[0], t[0:2])
                res = c0
                if halves:
                    ring_f = self._ring_done[0]
                    ring_f.record(s_f)
                    s_f.wait_event(done[1])
                    res = intra(0, mid, ws[0])
                    with torch.cuda.stream(s_b):
                        s_b.wait_event(ring_f)
                        intra(mid, Bn, ws[1])
                        done[1].record(s_b)
                    s_f.wait_event(done[1])
                else:
                    s_f.wait_event(done[1])
                    if self.intra:
                        res = intra(0, Bn, ws[0])
                done[0].record(s_f)
            main.wait_event(done[0])
            for st in streams:
                x.record_stream(st)
                valid_len.record_stream(st)
        B.unpack_rows(res, y, self.seg_len, valid_len, plan)
        return y

    def forward(self, x, valid_len=None, out=None, check=False):
        """x float32 [B, L, d] -> float32 [B, L, 2d].  The result lives in a buffer owned by this object, or in `out`
        (float32 [B, L, 2d], contiguous) when one is given.  check=True synchronises the stream afterwards and raises
        GsitError if a kernel reported a timed-out device-side wait (not for use under stream capture)."""
        if out is not None:
            assert out.shape == (x.shape[0], x.shape[1], 2 * x.shape[2]) and out.dtype == torch.float32 and out.is_contiguous()
        res = self._forward(x, valid_len, out)
        if out is not None and res.data_ptr() != out.data_ptr():
            out.copy_(res)
            res = out
        if check:
            code, flags = B.last_device_status()
            if code != 0:
                raise B.GsitError(code, f"GsitStack.forward: device status flags {flags:#x}")
        return res

    def _forward(self, x, valid_len, out):
        if self.packed and valid_len is not None and self.batch_chunks == 1:
            try:
                return self._forward_packed(x, valid_len, out)
            except B.GsitError as e:
                if e.code != 2:  # anything but "this shape is not covered": a real error
                    raise
                self.packed = False
        chunks, ws, t, c0, c1 = self._buffers(x, valid_len)
        if len(chunks) == 1 and not (self.concurrent_rings and self.fwd and self.bwd):
            self._ring(x, self.fwd, B.PHASE_INTER_FWD, 0, c0, ws[0][0], t[0:2], valid_len)
            self._ring(x, self.bwd, B.PHASE_INTER_BWD, 1, c0, ws[0][0], t[0:2], valid_len)
            return c1 if self._intra(c0, c1, ws[0][0], valid_len) else c0
        nch = len(chunks)
        if self._lanes is None or len(self._lanes[0]) != 2 * nch:
            dev = x.device
            self._lanes = ([torch.cuda.Stream(device=dev) for _ in range(2 * nch)], torch.cuda.Event(),
                           [torch.cuda.Event() for _ in range(2 * nch)])
            self._ring_done = [torch.cuda.Event() for _ in range(nch)]
        streams, fork, done = self._lanes
        main = torch.cuda.current_stream(x.device)
        fork.record(main)
        for c, sl in enumerate(chunks):
            vl = None if valid_len is None else valid_len[sl]
            s_f, s_b = streams[2 * c], streams[2 * c + 1]
            s_f.wait_event(fork)
            s_b.wait_event(fork)
            with torch.cuda.stream(s_b):
                self._ring(x[sl], self.bwd, B.PHASE_INTER_BWD, 1, c0[sl], ws[c][1], [t[2][sl], t[3][sl]], vl)
                done[2 * c + 1].record(s_b)
            with torch.cuda.stream(s_f):
                self._ring(x[sl], self.fwd, B.PHASE_INTER_FWD, 0, c0[sl], ws[c][0], [t[0][sl], t[1][sl]], vl)
                n = sl.stop - sl.start
                if self.intra_halves and self.intra and n >= 2:
                    # both streams wait for both rings, then each runs the intra encoder on one half of the samples
                    # (the ring workspaces are free by then: one per half)
                    lo, hi = slice(sl.start, sl.start + n // 2), slice(sl.start + n // 2, sl.stop)
                    ring_f = self._ring_done[c]
                    ring_f.record(s_f)
                    s_f.wait_event(done[2 * c + 1])
                    which = self._intra(c0[lo], c1[lo], ws[c][0], None if valid_len is None else valid_len[lo])
                    with torch.cuda.stream(s_b):
                        s_b.wait_event(ring_f)
                        self._intra(c0[hi], c1[hi], ws[c][1], None if valid_len is None else valid_len[hi])
                        done[2 * c + 1].record(s_b)
                    s_f.wait_event(done[2 * c + 1])
                else:
                    s_f.wait_event(done[2 * c + 1])  # both rings of this chunk are complete
                    which = self._intra(c0[sl], c1[sl], ws[c][0], vl)
                done[2 * c].record(s_f)
        for c in range(nch):
            main.wait_event(done[2 * c])
        for st in streams:
            x.record_stream(st)
            if valid_len is not None:
                valid_len.record_stream(st)
        return c1 if which else c0

    def read_out(self, c, valid_len=None):
        """X_m = f(|| Split(c)[-1]): last real step of each modality of the stack output c [B, L, 2d], through the linear
        map given as `head` -> float32 [B, out_features] (one gsit_stack_head_fwd call)."""
        assert self.head is not None, "no read-out weights were given"
        w_f, b_f = self.head
        return B.stack_head_fwd(c, w_f, b_f, self.seg_len, valid_len)
