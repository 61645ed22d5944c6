"""Small command-line driver: launches one library call a few times on synthetic workload-shaped inputs.

Meant for profilers and quick timing (the benchmark proper is bench.py at the repository root):

    python -m paper_2505_01068_b200.drive attention <workload 2..5> <batch> <phase 0|1|2> [--time]
    python -m paper_2505_01068_b200.drive layer <workload 2..5> <batch> <phase 0|1|2> [--d D --heads H] [--time]

`attention` fills a fused qkv buffer with N(0,1) values and calls gsit_im_attention_fwd; `layer` draws Xavier weights
and calls gsit_im_layer_fwd.  Valid lengths follow the workload's padding recipe.  With --time the call is repeated
over buffer sets larger than L2 and the mean device time per call is printed.
"""
from __future__ import annotations

import argparse
import sys
from pathlib import Path

import numpy as np
import torch

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

import workloads as wk  # noqa: E402

from . import binding as g  # noqa: E402


def main(argv=None):
    ap = argparse.ArgumentParser(prog="python -m paper_2505_01068_b200.drive")
    ap.add_argument("call", choices=["attention", "layer"])
    ap.add_argument("workload", type=int)
    ap.add_argument("batch", type=int)
    ap.add_argument("phase", type=int)
    ap.add_argument("--d", type=int, default=0, help="layer: d_model override (e.g. 128 for the intra encoder)")
    ap.add_argument("--heads", type=int, default=0)
    ap.add_argument("--time", action="store_true")
    ap.add_argument("--calls", type=int, default=3)
    a = ap.parse_args(argv)
    g.load()
    wl = wk.WORKLOADS[a.workload]
    rng = np.random.default_rng(wl.seed)
    valid = wk.draw_valid_len(rng, wl, a.batch)
    vl = None if valid is None else torch.from_numpy(valid).cuda()
    d = a.d or wl.d_model
    heads = a.heads or wl.heads
    B, L = a.batch, wl.L
    set_bytes = B * L * d * (8 if a.call == "attention" else 8)
    nsets = max(2, int(np.ceil(1.5 * 126e6 / set_bytes))) if a.time else 1
    gen = torch.Generator(device="cuda").manual_seed(1)
    if a.call == "attention":
        bufs = [torch.randn((B, L, 3, heads, d // heads), device="cuda", generator=gen).bfloat16() for _ in range(nsets)]
        outs = [torch.empty((B, L, d), device="cuda", dtype=torch.bfloat16) for _ in range(nsets)]
        run = lambda i: g.im_attention_fwd(bufs[i][:, :, 0], bufs[i][:, :, 1], bufs[i][:, :, 2], wl.seg_len, vl, a.phase,
                                           out=outs[i])
    else:
        w = wk.draw_layer_weights(rng, d, wl.d_ff_mult * d, wl.dtype)
        wd = {k: (None if v is None else (torch.from_numpy(v).cuda().bfloat16() if (k.startswith("w_") and wl.dtype == "bf16")
                                          else torch.from_numpy(v).cuda())) for k, v in w.items()}
        bufs = [torch.randn((B, L, d), device="cuda", generator=gen) for _ in range(nsets)]
        outs = [torch.empty((B, L, d), device="cuda") for _ in range(nsets)]
        sh = g.make_shape(B, wl.seg_len, d, heads, vl, g._dtype_code(wd["w_qkv"].dtype), a.phase)
        ws = torch.empty(g.workspace_bytes(sh, g.CALL_LAYER, wd["w_1"].shape[0]), dtype=torch.uint8, device="cuda")
        run = lambda i: g.im_layer_fwd(bufs[i], wd, wl.seg_len, heads, vl, a.phase, out=outs[i], workspace=ws)
    for _ in range(a.calls):
        for i in range(nsets):
            run(i)
    torch.cuda.synchronize()
    if a.time:
        beg, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        beg.record()
        for _ in range(5):
            for i in range(nsets):
                run(i)
        end.record()
        torch.cuda.synchronize()
        print(f"{a.call} workload {a.workload} batch {B} phase {a.phase} d {d}: "
              f"{beg.elapsed_time(end) * 1e3 / (5 * nsets):.1f} us per call over {nsets} buffer sets")
    print("device status", g.last_device_status())


if __name__ == "__main__":
    main()
