"""Parity at the workloads' full sizes, in the launch configuration bench.py times, on sampled outputs: samples are
independent, so the oracle is run on a few whole samples of the full batch (bit-for-bit the same inputs) and compared
element by element; padded rows are checked on the whole batch."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wk
from gpu_util import STACK_TOL, check_close, pad_mask, to_dev, to_np64, weights_to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def g():
    import paper_2505_01068_b200 as lib
    lib.load()
    return lib


def test_cfg4_full_batch_stack_sampled_samples(g):
    """The MOSEI-shaped stack at B = 64 exactly as the benchmark runs it (GsitStack, fused kernels, one workspace)."""
    inp = wk.make_inputs(4)
    wl = inp["workload"]
    n_f, n_b, n_i, ih = wl.stack
    valid = inp["valid_len"]
    vl = torch.from_numpy(valid).cuda()
    stack = g.GsitStack([weights_to_dev(w, "bf16") for w in inp["fwd_layers"]],
                        [weights_to_dev(w, "bf16") for w in inp["bwd_layers"]],
                        [weights_to_dev(w, "bf16") for w in inp["intra_layers"]], wl.seg_len, wl.heads, ih)
    x_dev = to_dev(wk.fill_padding(inp["x"], wl.seg_len, valid, np.nan))
    y = to_np64(stack.forward(x_dev, vl))
    pm = pad_mask(wl.seg_len, valid, wl.batch)
    assert np.isfinite(y).all() and np.all(y[pm] == 0.0) and not np.signbit(y[pm]).any()
    for b in (0, 37, 63):
        ref = oracle.gsit_stack_fwd(inp["x"][b:b + 1], inp["fwd_layers"], inp["bwd_layers"], inp["intra_layers"], wl.seg_len,
                                    wl.heads, ih, valid[b:b + 1])
        err = np.abs(y[b:b + 1] - ref)
        # ten layers in sequence: the measured compounding of the storage rounding times 1.5 (see STACK_TOL)
        assert err.max() <= STACK_TOL["max_abs"] and err.mean() <= STACK_TOL["mean_abs"], (b, err.max(), err.mean())
    # one layer of the same batch, held to the per-call tolerance
    w = inp["fwd_layers"][0]
    y1 = to_np64(g.im_layer_fwd(x_dev, weights_to_dev(w, "bf16"), wl.seg_len, wl.heads, vl, oracle.PHASE_INTER_FWD))
    assert np.all(y1[pm] == 0.0)
    for b in (5, 62):
        ref = oracle.im_layer_fwd(inp["x"][b:b + 1], w, wl.seg_len, wl.heads, valid[b:b + 1], oracle.PHASE_INTER_FWD)
        check_close(y1[b:b + 1], ref, "bf16", pm[b:b + 1], f"full-batch layer, sample {b}")
    code, flags = g.last_device_status()
    assert code == 0 and flags == 0


@pytest.mark.parametrize("which", ["cross_d64", "intra_d128"])
def test_full_batch_layer_repeats_bit_for_bit(g, which):
    """The same layer call on the same inputs, many times, at the full batch (several tiles per persistent CTA, every
    prefetch and hand-over of the fused kernels in play): every run must give the bits of the first.  A buffer that is
    refilled or an accumulator that is overwritten a moment too early shows up here as a handful of changed rows in a
    few runs out of a hundred, which a single comparison with the oracle would mostly miss."""
    inp = wk.make_inputs(4)
    wl = inp["workload"]
    n_f, n_b, n_i, ih = wl.stack
    valid = inp["valid_len"]
    vl = torch.from_numpy(valid).cuda()
    d, heads, w, phase = ((wl.d_model, wl.heads, inp["fwd_layers"][0], oracle.PHASE_INTER_FWD) if which == "cross_d64"
                          else (2 * wl.d_model, ih, inp["intra_layers"][0], oracle.PHASE_INTRA))
    rng = np.random.default_rng(31)
    x = to_dev(wk.fill_padding(rng.standard_normal((wl.batch, wl.L, d)).astype(np.float32), wl.seg_len, valid, np.nan))
    wd = weights_to_dev(w, "bf16")
    first = g.im_layer_fwd(x, wd, wl.seg_len, heads, vl, phase).clone()
    torch.cuda.synchronize()
    assert torch.isfinite(first).all()
    for run in range(120):
        y = g.im_layer_fwd(x, wd, wl.seg_len, heads, vl, phase)
        torch.cuda.synchronize()
        assert torch.equal(y, first), (which, run)
    # the packed row layout through the same kernels
    cap = wl.batch * wl.L + 128
    plan = g.plan_rows(vl, wl.seg_len)
    xp = torch.zeros((cap, d), device="cuda")
    g.pack_rows(x, xp, wl.seg_len, vl, plan)
    used = int(plan[-1])
    firstp = None
    for run in range(60):
        yp = torch.zeros((cap, d), device="cuda")
        g.im_layer_fwd(xp, wd, wl.seg_len, heads, vl, phase, out=yp, row_start=plan)
        torch.cuda.synchronize()
        if firstp is None:
            firstp = yp.clone()
        assert torch.equal(yp[:used], firstp[:used]), (which, "packed", run)
    assert g.last_device_status() == (0, 0)


def test_cfg4_stack_repeats_bit_for_bit(g):
    """The whole stack, eager, repeated on NaN-padded input in each way of issuing it."""
    inp = wk.make_inputs(4)
    wl = inp["workload"]
    n_f, n_b, n_i, ih = wl.stack
    valid = inp["valid_len"]
    vl = torch.from_numpy(valid).cuda()
    x_dev = to_dev(wk.fill_padding(inp["x"], wl.seg_len, valid, np.nan))
    for kw in (dict(), dict(paired_rings=False), dict(packed=False)):
        stack = g.GsitStack([weights_to_dev(w, "bf16") for w in inp["fwd_layers"]],
                            [weights_to_dev(w, "bf16") for w in inp["bwd_layers"]],
                            [weights_to_dev(w, "bf16") for w in inp["intra_layers"]], wl.seg_len, wl.heads, ih, **kw)
        first = stack.forward(x_dev, vl).clone()
        torch.cuda.synchronize()
        for run in range(12):
            y = stack.forward(x_dev, vl)
            torch.cuda.synchronize()
            assert torch.equal(y, first), (kw, run)
    assert g.last_device_status() == (0, 0)


def test_cfg5_full_batch_attention_and_projection_sampled_samples(g):
    """The scaled shape at B = 128: tcgen05 attention (all three patterns) and the tcgen05 QKV projection."""
    wl = wk.WORKLOADS[5]
    B = wl.batch
    rng = np.random.default_rng(wl.seed)
    valid = wk.draw_valid_len(rng, wl, B)
    vl = torch.from_numpy(valid).cuda()
    gen = torch.Generator(device="cuda").manual_seed(wl.seed)
    x = torch.randn((B, wl.L, wl.d_model), device="cuda", generator=gen).bfloat16()
    w = (torch.randn((3 * wl.d_model, wl.d_model), device="cuda", generator=gen) * wl.d_model ** -0.5).bfloat16()
    qkv = g.im_qkv_proj(x, w, None, wl.seg_len, wl.heads, vl)
    pm = pad_mask(wl.seg_len, valid, B)
    pm_dev = torch.from_numpy(pm).cuda()
    assert bool((qkv[pm_dev] == 0).all())
    samples = (0, 3, 127)   # 3 is one of the half-length samples
    w_np = to_np64(w).astype(np.float32)
    for b in samples:
        xb = to_np64(x[b:b + 1]).astype(np.float32)
        ref = oracle.qkv_proj(xb, w_np, None, wl.seg_len, wl.heads, valid[b:b + 1])
        check_close(to_np64(qkv[b:b + 1]).reshape(1, wl.L, -1), ref.reshape(1, wl.L, -1), "bf16", pm[b:b + 1],
                    f"full-batch projection, sample {b}")
    for ph in (oracle.PHASE_INTER_FWD, oracle.PHASE_INTER_BWD, oracle.PHASE_INTRA):
        out = g.im_attention_fwd(qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2], wl.seg_len, vl, ph)
        assert bool((out[pm_dev] == 0).all()) and bool(torch.isfinite(out.float()).all())
        for b in samples:
            q64 = to_np64(qkv[b:b + 1])
            ref = oracle.im_attention_dense(q64[:, :, 0], q64[:, :, 1], q64[:, :, 2], wl.seg_len, valid[b:b + 1], ph)
            check_close(to_np64(out[b:b + 1]), ref, "bf16", pm[b:b + 1], f"full-batch attention phase {ph}, sample {b}")
        for run in range(10):  # the same launch again: the same bits, whichever CTA takes which work item
            again = g.im_attention_fwd(qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2], wl.seg_len, vl, ph)
            assert torch.equal(again, out), (ph, run)
    for run in range(10):
        assert torch.equal(g.im_qkv_proj(x, w, None, wl.seg_len, wl.heads, vl), qkv), run
    code, flags = g.last_device_status()
    assert code == 0 and flags == 0
