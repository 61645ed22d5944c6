"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element, on the same
seeded inputs, at the five workload shapes (batch reduced where the oracle would take minutes)."""
import numpy as np
import pytest
import torch

import oracle
import workloads as wk
from gpu_util import STACK_TOL, check_close, pad_mask, to_dev, to_np64, weights_to_dev

pytestmark = pytest.mark.gpu
PHASES = [oracle.PHASE_INTER_FWD, oracle.PHASE_INTER_BWD, oracle.PHASE_INTRA]


@pytest.fixture(scope="module")
def g():
    import paper_2505_01068_b200 as lib
    lib.load()
    return lib


def _attention_case(g, x, w_qkv, seg, heads, valid, dtype, phases=PHASES, nan_padding=False, check_lse=True):
    """qkv projection + attention per phase, each compared with the oracle fed the same (rounded) arrays."""
    B = x.shape[0]
    pm = pad_mask(seg, valid, B)
    x_dev_np = wk.fill_padding(x, seg, valid, np.nan) if nan_padding else x
    vl = None if valid is None else torch.from_numpy(valid).cuda()
    xd, wd = to_dev(x_dev_np, dtype), to_dev(w_qkv, dtype)
    qkv = g.im_qkv_proj(xd, wd, None, seg, heads, vl)
    ref_qkv = oracle.qkv_proj(x, w_qkv, None, seg, heads, valid)
    check_close(to_np64(qkv).reshape(B, -1, 3 * x.shape[2]), ref_qkv.reshape(B, -1, 3 * x.shape[2]), dtype, pm, "qkv_proj")
    # the oracle attends over exactly the q, k, v the GPU attention reads (the GPU's own rounded projection)
    qkv64 = to_np64(qkv)
    res = {}
    for ph in phases:
        out, lse = g.im_attention_fwd(qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2], seg, vl, ph, want_lse=True)
        ref, ref_lse = oracle.im_attention_dense(qkv64[:, :, 0], qkv64[:, :, 1], qkv64[:, :, 2], seg, valid, ph, want_lse=True)
        res[ph] = check_close(to_np64(out), ref, dtype, pm, f"attention phase {ph}")
        if check_lse:
            gl = to_np64(lse)
            fin = np.isfinite(ref_lse)
            assert np.array_equal(np.isneginf(gl), np.isneginf(ref_lse))
            assert np.abs(gl[fin] - ref_lse[fin]).max() <= (1e-4 if dtype == "f32" else 2e-2)
    code, flags = g.last_device_status()
    assert code == 0 and flags == 0
    return res


def test_cfg1_tiny_f32_attention_and_layers(g):
    inp = wk.make_inputs(1)
    wl = inp["workload"]
    _attention_case(g, inp["x"], inp["layer"]["w_qkv"], wl.seg_len, wl.heads, None, "f32")
    wd = weights_to_dev(inp["layer"], "f32")
    xd = to_dev(inp["x"])
    for ph in PHASES:
        y = g.im_layer_fwd(xd, wd, wl.seg_len, wl.heads, None, ph)
        ref = oracle.im_layer_fwd(inp["x"], inp["layer"], wl.seg_len, wl.heads, None, ph)
        check_close(to_np64(y), ref, "f32", None, f"layer phase {ph}")


def test_cfg1_f32_wo_projected_attention(g):
    """Attention followed by the shared W_o (the layer with the MLP switched off and x = 0 residual removed)."""
    inp = wk.make_inputs(1)
    wl = inp["workload"]
    w = dict(inp["layer"], w_2=np.zeros_like(inp["layer"]["w_2"]))
    wd = weights_to_dev(w, "f32")
    for ph in PHASES:
        y = g.im_layer_fwd(to_dev(inp["x"]), wd, wl.seg_len, wl.heads, None, ph)
        ref = oracle.im_layer_fwd(inp["x"], w, wl.seg_len, wl.heads, None, ph)
        check_close(to_np64(y), ref, "f32", None, f"x + O W_o phase {ph}")


def test_cfg2_aligned_bf16(g):
    inp = wk.make_inputs(2)
    wl = inp["workload"]
    _attention_case(g, inp["x"], inp["layer"]["w_qkv"], wl.seg_len, wl.heads, None, "bf16")


def test_cfg3_mosi_unaligned_bf16_nan_padding(g):
    inp = wk.make_inputs(3)
    wl = inp["workload"]
    _attention_case(g, inp["x"], inp["layer"]["w_qkv"], wl.seg_len, wl.heads, inp["valid_len"], "bf16", nan_padding=True)


def test_cfg4_mosei_attention_and_layer_bf16(g):
    inp = wk.make_inputs(4, batch=8)
    wl = inp["workload"]
    _attention_case(g, inp["x"], inp["layer"]["w_qkv"], wl.seg_len, wl.heads, inp["valid_len"], "bf16", nan_padding=True)
    vl = torch.from_numpy(inp["valid_len"]).cuda()
    pm = pad_mask(wl.seg_len, inp["valid_len"], 8)
    xd = to_dev(wk.fill_padding(inp["x"], wl.seg_len, inp["valid_len"], np.nan))
    for ph, w in ((oracle.PHASE_INTER_FWD, inp["fwd_layers"][0]), (oracle.PHASE_INTER_BWD, inp["bwd_layers"][0])):
        y = g.im_layer_fwd(xd, weights_to_dev(w, "bf16"), wl.seg_len, wl.heads, vl, ph)
        ref = oracle.im_layer_fwd(inp["x"], w, wl.seg_len, wl.heads, inp["valid_len"], ph)
        check_close(to_np64(y), ref, "bf16", pm, f"layer d=64 phase {ph}")
    # intra layer at width 2d with 8 heads of 16
    rng = np.random.default_rng(77)
    x2 = rng.standard_normal((8, wl.L, 2 * wl.d_model), dtype=np.float32)
    w = inp["intra_layers"][0]
    y = g.im_layer_fwd(to_dev(x2), weights_to_dev(w, "bf16"), wl.seg_len, 8, vl, oracle.PHASE_INTRA)
    ref = oracle.im_layer_fwd(x2, w, wl.seg_len, 8, inp["valid_len"], oracle.PHASE_INTRA)
    check_close(to_np64(y), ref, "bf16", pm, "intra layer d=128")


def test_cfg4_full_stack_bf16(g):
    inp = wk.make_inputs(4, batch=4)
    wl = inp["workload"]
    n_f, n_b, n_i, ih = wl.stack
    vl = torch.from_numpy(inp["valid_len"]).cuda()
    stack = g.GsitStack([weights_to_dev(w, "bf16") for w in inp["fwd_layers"]],
                        [weights_to_dev(w, "bf16") for w in inp["bwd_layers"]],
                        [weights_to_dev(w, "bf16") for w in inp["intra_layers"]], wl.seg_len, wl.heads, ih)
    y = stack.forward(to_dev(inp["x"]), vl)
    ref = oracle.gsit_stack_fwd(inp["x"], inp["fwd_layers"], inp["bwd_layers"], inp["intra_layers"], wl.seg_len,
                                wl.heads, ih, inp["valid_len"])
    pm = pad_mask(wl.seg_len, inp["valid_len"], 4)
    got = to_np64(y)
    assert np.isfinite(got).all() and np.all(got[pm] == 0.0)
    err = np.abs(got - ref)
    # ten layers in sequence: the measured compounding of the storage rounding times 1.5 (see STACK_TOL)
    assert err.max() <= STACK_TOL["max_abs"] and err.mean() <= STACK_TOL["mean_abs"], (err.max(), err.mean())


def test_cfg4_every_stack_layer_teacher_forced(g):
    """Each of the ten layers of the MOSEI-shaped stack on its own, fed the ORACLE's previous activation (rounded to the
    float32 residual stream the library stores), against the oracle's output of that layer at the per-call tolerance:
    an error of one layer cannot hide behind, or be blamed on, the layers before it."""
    inp = wk.make_inputs(4, batch=2)
    wl = inp["workload"]
    n_f, n_b, n_i, ih = wl.stack
    valid = inp["valid_len"]
    vl = torch.from_numpy(valid).cuda()
    pm = pad_mask(wl.seg_len, valid, 2)

    def ring(layers, phase, heads, a, name):
        for i, w in enumerate(layers):
            a32 = a.astype(np.float32)
            ref = oracle.im_layer_fwd(a32, w, wl.seg_len, heads, valid, phase)
            xd = to_dev(wk.fill_padding(a32, wl.seg_len, valid, np.nan))
            y = g.im_layer_fwd(xd, weights_to_dev(w, "bf16"), wl.seg_len, heads, vl, phase)
            check_close(to_np64(y), ref, "bf16", pm, f"{name} layer {i}, teacher-forced")
            a = ref
        return a

    a = ring(inp["fwd_layers"], oracle.PHASE_INTER_FWD, wl.heads, inp["x"].astype(np.float64), "forward-ring")
    b = ring(inp["bwd_layers"], oracle.PHASE_INTER_BWD, wl.heads, inp["x"].astype(np.float64), "backward-ring")
    ring(inp["intra_layers"], oracle.PHASE_INTRA, ih, np.concatenate([a, b], axis=-1), "intra")
    assert g.last_device_status() == (0, 0)


def test_cfg5_scaled_hd64_bf16(g):
    """Scaled shape (L=2176, d=512, 8 heads of 64) on two samples, one of them padded to half length."""
    wl = wk.WORKLOADS[5]
    B = 2
    rng = np.random.default_rng(wl.seed)
    q, k, v = wk.draw_qkv(rng, B, wl.L, wl.heads, wl.d_model // wl.heads, "bf16")
    valid = np.array([wl.seg_len, [s // 2 for s in wl.seg_len]], dtype=np.int32)
    vl = torch.from_numpy(valid).cuda()
    pm = pad_mask(wl.seg_len, valid, B)
    qd, kd, vd = (to_dev(a, "bf16") for a in (q, k, v))
    for ph in PHASES:
        out = g.im_attention_fwd(qd, kd, vd, wl.seg_len, vl, ph)
        ref = oracle.im_attention_dense(q, k, v, wl.seg_len, valid, ph)
        check_close(to_np64(out), ref, "bf16", pm, f"cfg5 attention phase {ph}")
    # the shared projection at d=512
    x = wk.storage_round(rng.standard_normal((2, wl.L, wl.d_model), dtype=np.float32), "bf16")
    w = wk.draw_layer_weights(rng, wl.d_model, 4 * wl.d_model, "bf16")["w_qkv"]
    qkv = g.im_qkv_proj(to_dev(x, "bf16"), to_dev(w, "bf16"), None, wl.seg_len, wl.heads, vl[:2].contiguous())
    ref = oracle.qkv_proj(x, w, None, wl.seg_len, wl.heads, valid[:2])
    check_close(to_np64(qkv).reshape(2, wl.L, -1), ref.reshape(2, wl.L, -1), "bf16", pad_mask(wl.seg_len, valid[:2], 2),
                "qkv_proj d=512")


@pytest.mark.parametrize("d,heads,d_ff,seg,B", [(64, 8, 256, (50, 170, 93), 3), (128, 8, 512, (37, 150, 64), 2),
                                                (64, 4, 64, (50, 30, 90), 2), (64, 8, 128, (5, 0, 9), 3),
                                                (32, 4, 128, (40, 33, 20), 2), (192, 3, 768, (70, 129, 33), 2), (128, 4, 64, (5, 0, 9), 3),
                                                (128, 8, 320, (50, 201, 93), 2), (64, 8, 192, (300, 20, 333), 2)])
def test_layer_bf16_affine_biases_ragged(g, d, heads, d_ff, seg, B):
    """One IM layer with LayerNorm affine parameters and every bias set, ragged valid lengths, NaN in the padded input
    rows and a row count that is not a multiple of any tile: d = 64 / 128 take the fused tcgen05 kernels, d = 32 the separate
    LayerNorm / mma.sync linear kernels, d = 192 the separate kernels with every linear layer on the tcgen05 GEMM (bias,
    ReLU, float output with residual, TMA-stored bf16 output)."""
    rng = np.random.default_rng(d * 1000 + d_ff)
    x = rng.standard_normal((B, sum(seg), d), dtype=np.float32)
    w = wk.draw_layer_weights(rng, d, d_ff, "bf16", affine=True)
    valid = np.stack([rng.integers(0, s + 1, size=B) for s in seg], axis=1).astype(np.int32)
    valid[0] = seg
    pm = pad_mask(seg, valid, B)
    xd = to_dev(wk.fill_padding(x, seg, valid, np.nan))
    vl = torch.from_numpy(valid).cuda()
    for ph in PHASES:
        y = g.im_layer_fwd(xd, weights_to_dev(w, "bf16"), seg, heads, vl, ph)
        ref = oracle.im_layer_fwd(x, w, seg, heads, valid, ph)
        check_close(to_np64(y), ref, "bf16", pm, f"affine layer d={d} phase {ph}")
    code, flags = g.last_device_status()
    assert code == 0 and flags == 0


def test_qkv_proj_tcgen05_matches_mma_sync_kernel(g):
    """The shared projection through the tcgen05 GEMM and through the mma.sync kernel (kernel choice ATTN_LEGACY) on the same inputs:
    both within the bf16 tolerance of the oracle, and within rounding of each other."""
    rng = np.random.default_rng(31)
    seg, B, d, H = (37, 300, 129), 3, 256, 4
    x = wk.storage_round(rng.standard_normal((B, sum(seg), d), dtype=np.float32), "bf16")
    w = wk.draw_layer_weights(rng, d, 4 * d, "bf16", affine=True)
    valid = np.array([[37, 300, 129], [1, 150, 0], [20, 299, 64]], dtype=np.int32)
    vl = torch.from_numpy(valid).cuda()
    xd = to_dev(wk.fill_padding(x, seg, valid, np.nan), "bf16")
    wd, bd = to_dev(w["w_qkv"], "bf16"), to_dev(w["b_qkv"])
    new = to_np64(g.im_qkv_proj(xd, wd, bd, seg, H, vl)).reshape(B, sum(seg), -1)
    g.tune_attention(g.ATTN_LEGACY)
    try:
        old = to_np64(g.im_qkv_proj(xd, wd, bd, seg, H, vl)).reshape(B, sum(seg), -1)
    finally:
        g.tune_attention(0)
    ref = oracle.qkv_proj(x, w["w_qkv"], w["b_qkv"], seg, H, valid).reshape(B, sum(seg), -1)
    pm = pad_mask(seg, valid, B)
    check_close(new, ref, "bf16", pm, "tcgen05 projection")
    check_close(old, ref, "bf16", pm, "mma.sync projection")
    assert np.abs(new - old).max() <= 2.0 ** -6
    code, flags = g.last_device_status()
    assert code == 0 and flags == 0


@pytest.mark.parametrize("d,heads,d_ff", [(64, 8, 256), (128, 8, 512)])
def test_fused_layer_tcgen05_matches_mma_sync_fused_kernels(g, d, heads, d_ff):
    """The tcgen05 fused halves and the mma.sync fused halves (kernel choice ATTN_LEGACY) compute the same layer."""
    rng = np.random.default_rng(d)
    seg, B = (50, 333, 190), 2
    x = rng.standard_normal((B, sum(seg), d), dtype=np.float32)
    w = weights_to_dev(wk.draw_layer_weights(rng, d, d_ff, "bf16", affine=True), "bf16")
    valid = np.array([[50, 333, 190], [25, 170, 1]], dtype=np.int32)
    vl = torch.from_numpy(valid).cuda()
    xd = to_dev(wk.fill_padding(x, seg, valid, np.nan))
    new = to_np64(g.im_layer_fwd(xd, w, seg, heads, vl, oracle.PHASE_INTER_BWD))
    g.tune_attention(g.ATTN_LEGACY)
    try:
        old = to_np64(g.im_layer_fwd(xd, w, seg, heads, vl, oracle.PHASE_INTER_BWD))
    finally:
        g.tune_attention(0)
    assert np.isfinite(new).all() and np.abs(new - old).max() <= 2e-2 and np.abs(new - old).mean() <= 1e-3
    pm = pad_mask(seg, valid, B)
    assert np.all(new[pm] == 0.0)
    code, flags = g.last_device_status()
    assert code == 0 and flags == 0


@pytest.mark.parametrize("d,heads,d_ff", [(64, 8, 256), (64, 4, 128), (128, 8, 512), (32, 4, 128)])
def test_layer_pair_call_equals_two_layer_calls(g, d, heads, d_ff):
    """gsit_im_layer_pair_fwd (both ring encoders' layers of one depth in one call; one launch per kernel at d_model 64,
    the two layers in sequence elsewhere) gives the bits of two gsit_im_layer_fwd calls, padded and packed layout, and the
    forward-ring member is held to the oracle."""
    rng = np.random.default_rng(d + d_ff)
    seg, B = (50, 300, 170), 3
    xa = rng.standard_normal((B, sum(seg), d), dtype=np.float32)
    xb = rng.standard_normal((B, sum(seg), d), dtype=np.float32)
    wa_np = wk.draw_layer_weights(rng, d, d_ff, "bf16", affine=True)
    wa, wb = weights_to_dev(wa_np, "bf16"), weights_to_dev(wk.draw_layer_weights(rng, d, d_ff, "bf16", affine=True), "bf16")
    valid = np.array([[50, 300, 170], [25, 151, 0], [1, 299, 100]], dtype=np.int32)
    vl = torch.from_numpy(valid).cuda()
    xad, xbd = to_dev(wk.fill_padding(xa, seg, valid, np.nan)), to_dev(wk.fill_padding(xb, seg, valid, np.nan))
    want_a = g.im_layer_fwd(xad, wa, seg, heads, vl, g.PHASE_INTER_FWD)
    want_b = g.im_layer_fwd(xbd, wb, seg, heads, vl, g.PHASE_INTER_BWD)
    got_a, got_b = g.im_layer_pair_fwd(xad, xbd, wa, wb, seg, heads, vl)
    torch.cuda.synchronize()
    assert torch.equal(got_a, want_a) and torch.equal(got_b, want_b)
    ref = oracle.im_layer_fwd(xa, wa_np, seg, heads, valid, oracle.PHASE_INTER_FWD)
    check_close(to_np64(got_a), ref, "bf16", pad_mask(seg, valid, B), "pair call, forward-ring member")
    # the same input for both members (the first layer of the stack), and a custom pattern for the second
    got_a2, got_c = g.im_layer_pair_fwd(xad, xad, wa, wb, seg, heads, vl, g.PHASE_INTER_FWD, g.PHASE_INTRA)
    assert torch.equal(got_a2, want_a) and torch.equal(got_c, g.im_layer_fwd(xad, wb, seg, heads, vl, g.PHASE_INTRA))
    if d in (64, 128):  # packed layout
        L = sum(seg)
        cap = B * L + 128
        plan = g.plan_rows(vl, seg)
        xp = [torch.zeros((cap, d), device="cuda") for _ in range(2)]
        g.pack_rows(xad, xp[0], seg, vl, plan)
        g.pack_rows(xbd, xp[1], seg, vl, plan)
        yp = [torch.full((cap, d), float("nan"), device="cuda") for _ in range(2)]
        g.im_layer_pair_fwd(xp[0], xp[1], wa, wb, seg, heads, vl, out_a=yp[0], out_b=yp[1], row_start=plan)
        for ypk, want in ((yp[0], want_a), (yp[1], want_b)):
            back = torch.full_like(want, 3.0)
            g.unpack_rows(ypk, back, seg, vl, plan)
            torch.cuda.synchronize()
            assert torch.equal(back, want)
    assert g.last_device_status() == (0, 0)


@pytest.mark.parametrize("index", [6, 7, 8])
def test_second_workload_family_attention_and_layer(g, index):
    """Dataset-statistics lengths (MOSEI averages) and the CH-SIMS / MIntRec segment shapes: projection, all three
    block patterns and one layer, NaN in the padded rows."""
    inp = wk.make_inputs(index, batch=6)
    wl = inp["workload"]
    _attention_case(g, inp["x"], inp["layer"]["w_qkv"], wl.seg_len, wl.heads, inp["valid_len"], "bf16", nan_padding=True)
    vl = torch.from_numpy(inp["valid_len"]).cuda()
    pm = pad_mask(wl.seg_len, inp["valid_len"], 6)
    xd = to_dev(wk.fill_padding(inp["x"], wl.seg_len, inp["valid_len"], np.nan))
    y = g.im_layer_fwd(xd, weights_to_dev(inp["layer"], "bf16"), wl.seg_len, wl.heads, vl, oracle.PHASE_INTER_BWD)
    ref = oracle.im_layer_fwd(inp["x"], inp["layer"], wl.seg_len, wl.heads, inp["valid_len"], oracle.PHASE_INTER_BWD)
    check_close(to_np64(y), ref, "bf16", pm, f"workload {index} layer")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_stack_head_readout(g, dtype):
    """Last real step of each modality, concatenated, through the linear map f -- against the oracle."""
    rng = np.random.default_rng(77)
    seg, B, dc, n_out = (50, 300, 270), 5, 128, 192
    c = rng.standard_normal((B, sum(seg), dc), dtype=np.float32)
    w = wk.storage_round(wk.xavier_uniform(rng, n_out, 3 * dc), dtype)
    bias = (0.1 * rng.standard_normal(n_out)).astype(np.float32)
    valid = np.array([[50, 300, 270], [1, 150, 270], [25, 0, 1], [50, 1, 135], [13, 299, 200]], dtype=np.int32)
    vl = torch.from_numpy(valid).cuda()
    cd = to_dev(wk.fill_padding(c, seg, valid, np.nan))
    for v_np, v_dev in ((valid, vl), (None, None)):
        src = cd if v_np is not None else to_dev(c)
        got = to_np64(g.stack_head_fwd(src, to_dev(w, dtype), to_dev(bias), seg, v_dev))
        ref = oracle.stack_head_fwd(c, w, bias, seg, v_np)
        assert np.isfinite(got).all() and np.abs(got - ref).max() <= (1e-4 if dtype == "f32" else 2e-2)
    # a strided view (the right half of a wider buffer) gives the same result as its contiguous copy
    wide = torch.zeros((B, sum(seg), 2 * dc), device="cuda")
    wide[:, :, dc:] = to_dev(c)
    a = g.stack_head_fwd(wide[:, :, dc:], to_dev(w, dtype), None, seg, vl)
    b2 = g.stack_head_fwd(to_dev(c), to_dev(w, dtype), None, seg, vl)
    assert torch.equal(a, b2)


def test_stack_rings_on_two_streams_match_serial_issue(g):
    """Issuing the forward and backward rings on two streams changes the order of launches, not a single bit."""
    inp = wk.make_inputs(4, batch=6)
    wl = inp["workload"]
    n_f, n_b, n_i, ih = wl.stack
    vl = torch.from_numpy(inp["valid_len"]).cuda()
    mk = lambda conc, chunks=1: g.GsitStack([weights_to_dev(w, "bf16") for w in inp["fwd_layers"]],
                                            [weights_to_dev(w, "bf16") for w in inp["bwd_layers"]],
                                            [weights_to_dev(w, "bf16") for w in inp["intra_layers"]], wl.seg_len, wl.heads,
                                            ih, concurrent_rings=conc, batch_chunks=chunks, paired_rings=False)
    x = to_dev(inp["x"])
    a = mk(True).forward(x, vl).clone()
    b = mk(False).forward(x, vl).clone()
    c = mk(True, 4).forward(x, vl).clone()  # the batch cut into groups of samples (6 -> 2, 2, 1, 1), each on its own streams
    st = mk(True)
    st.intra_halves = False                 # intra encoder on the whole batch instead of one half per stream
    d = st.forward(x, vl).clone()
    st = mk(True)
    st.paired_rings = True                  # both rings through the pair call on one stream (the default)
    e = st.forward(x, vl).clone()
    torch.cuda.synchronize()
    assert torch.equal(a, b) and torch.equal(a, c) and torch.equal(a, d) and torch.equal(a, e)
    assert g.last_device_status() == (0, 0)


def test_host_pipeline_delivers_every_step(g):
    """Overlapped host->device / kernels / device->host legs: each step's result equals the plain forward of its own
    input (bit for bit), for more steps than the pipeline is deep, and one of them is held to the oracle."""
    from paper_2505_01068_b200.hostio import HostPipeline
    inp = wk.make_inputs(4, batch=3)
    wl = inp["workload"]
    n_f, n_b, n_i, ih = wl.stack
    stack = g.GsitStack([weights_to_dev(w, "bf16") for w in inp["fwd_layers"]],
                        [weights_to_dev(w, "bf16") for w in inp["bwd_layers"]],
                        [weights_to_dev(w, "bf16") for w in inp["intra_layers"]], wl.seg_len, wl.heads, ih)
    rng = np.random.default_rng(5)
    steps = 5
    xs = [inp["x"]] + [rng.standard_normal(inp["x"].shape).astype(np.float32) for _ in range(steps - 1)]
    vs = [inp["valid_len"]] + [wk.draw_valid_len(rng, wl, 3) for _ in range(steps - 1)]
    x_host = [torch.from_numpy(x).pin_memory() for x in xs]
    v_host = [torch.from_numpy(v).pin_memory() for v in vs]
    y_host = [torch.empty((3, wl.L, 2 * wl.d_model), dtype=torch.float32).pin_memory() for _ in range(steps)]
    pipe = HostPipeline(stack, inp["x"].shape, depth=2)
    for i in range(steps):
        pipe.step(x_host[i], y_host[i], v_host[i])
    pipe.wait()
    for i in range(steps):
        want = stack.forward(x_host[i].cuda(), v_host[i].cuda())
        torch.cuda.synchronize()
        assert torch.equal(want.cpu(), y_host[i]), i
    ref = oracle.gsit_stack_fwd(xs[0], inp["fwd_layers"], inp["bwd_layers"], inp["intra_layers"], wl.seg_len, wl.heads, ih, vs[0])
    err = np.abs(y_host[0].numpy().astype(np.float64) - ref)
    assert err.max() <= STACK_TOL["max_abs"] and err.mean() <= STACK_TOL["mean_abs"], (err.max(), err.mean())
    assert g.last_device_status() == (0, 0)


def test_stack_replayed_back_to_back_gives_the_same_bits(g):
    """Kernels of a stream start under the tail of the one before them (programmatic dependent launch), inside one forward
    and from one forward to the next.  Many captured forwards replayed back to back over alternating inputs must each
    give exactly what a lone eager forward of that input gives: a kernel that touched its predecessor's data before the
    predecessor had finished would show up as a changed bit."""
    inp = wk.make_inputs(4, batch=8)
    wl = inp["workload"]
    n_f, n_b, n_i, ih = wl.stack
    vl = torch.from_numpy(inp["valid_len"]).cuda()
    rng = np.random.default_rng(77)
    xs = [to_dev(inp["x"]), to_dev(rng.standard_normal(inp["x"].shape).astype(np.float32))]
    for kw in (dict(), dict(paired_rings=False)):
        stack = g.GsitStack([weights_to_dev(w, "bf16") for w in inp["fwd_layers"]],
                            [weights_to_dev(w, "bf16") for w in inp["bwd_layers"]],
                            [weights_to_dev(w, "bf16") for w in inp["intra_layers"]], wl.seg_len, wl.heads, ih, **kw)
        want = []
        for x in xs:
            want.append(stack.forward(x, vl).clone())
            torch.cuda.synchronize()
        outs = [torch.empty_like(want[0]) for _ in xs]
        graphs = []
        for x, o in zip(xs, outs):
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr):
                stack.forward(x, vl, out=o)
            graphs.append(gr)
        for rep in range(10):
            for o in outs:
                o.fill_(float("nan"))
            for k in range(6):
                graphs[k % 2].replay()
            torch.cuda.synchronize()
            for k in range(2):
                assert torch.equal(outs[k], want[k]), (kw, rep, k)
    assert g.last_device_status() == (0, 0)


def _real_mask(seg_len, valid, B):
    L = sum(seg_len)
    off = np.cumsum([0] + list(seg_len))
    real = np.zeros((B, L), dtype=bool)
    for b in range(B):
        for s in range(3):
            real[b, off[s]:off[s] + valid[b, s]] = True
    return real


def test_packed_rows_plan_pack_unpack(g):
    """Packed row layout: the device-made plan is the running sum of the valid lengths (with the requested sample
    starting on a multiple of 128 rows), packing gathers exactly the real rows, unpacking restores them and writes +0
    in the padded positions."""
    seg = (50, 300, 270)
    valid = np.array([[50, 300, 270], [25, 0, 200], [0, 0, 0], [1, 151, 7], [50, 299, 1]], dtype=np.int32)
    B, L, cols = valid.shape[0], sum(seg), 64
    vl = torch.from_numpy(valid).cuda()
    rng = np.random.default_rng(3)
    x = rng.standard_normal((B, L, cols), dtype=np.float32)
    real = _real_mask(seg, valid, B)
    for split in (0, 2, 4):
        plan = g.plan_rows(vl, seg, split).cpu().numpy()
        run, want = 0, []
        for b in range(B):
            if split and b == split:
                run = (run + 127) // 128 * 128
            for s in range(3):
                want.append(run)
                run += int(valid[b, s])
        want.append(run)
        assert np.array_equal(plan, np.array(want, dtype=np.int32)), split
        plan_d = torch.from_numpy(plan).cuda()
        xp = torch.full((B * L + 128, cols), float("nan"), device="cuda")
        g.pack_rows(to_dev(x), xp, seg, vl, plan_d)
        xp_h = xp.cpu().numpy()
        for b in range(B):
            off = 0
            for s in range(3):
                n = valid[b, s]
                assert np.array_equal(xp_h[plan[3 * b + s]:plan[3 * b + s] + n], x[b, off:off + n])
                off += seg[s]
        back = torch.full((B, L, cols), 7.0, device="cuda")
        g.unpack_rows(xp, back, seg, vl, plan_d)
        bk = back.cpu().numpy()
        assert np.array_equal(bk[real], x[real]) and np.all(bk[~real] == 0.0) and not np.signbit(bk[~real]).any()
    assert g.last_device_status() == (0, 0)


def test_packed_layout_gives_the_same_bits_as_the_padded_one(g):
    """Layers and the whole stack on the packed rows against the same calls on the padded layout: samples and rows are
    independent and the arithmetic per row is the same, so the results are equal bit for bit (and the padded layout is
    held to the oracle above)."""
    inp = wk.make_inputs(4, batch=5)
    wl = inp["workload"]
    n_f, n_b, n_i, ih = wl.stack
    valid = inp["valid_len"].copy()
    valid[1] = [0, valid[1, 1], 0]          # a sample with two empty modalities
    valid[3] = [0, 0, 0]                     # and an empty sample
    vl = torch.from_numpy(valid).cuda()
    B, L, d = inp["x"].shape
    cap = B * L + 128
    x = to_dev(wk.fill_padding(inp["x"], wl.seg_len, valid, np.nan))
    plan = g.plan_rows(vl, wl.seg_len)
    for w, heads, ph, width in ((inp["fwd_layers"][0], wl.heads, g.PHASE_INTER_FWD, d), (inp["bwd_layers"][1], wl.heads, g.PHASE_INTER_BWD, d),
                                (inp["intra_layers"][0], ih, g.PHASE_INTRA, 2 * d)):
        xin = x if width == d else torch.cat([x, x.flip(2)], dim=2).contiguous()
        wd = weights_to_dev(w, "bf16")
        want = g.im_layer_fwd(xin, wd, wl.seg_len, heads, vl, ph)
        xp = torch.zeros((cap, width), device="cuda")
        g.pack_rows(xin, xp, wl.seg_len, vl, plan)
        yp = torch.full((cap, width), float("nan"), device="cuda")
        g.im_layer_fwd(xp, wd, wl.seg_len, heads, vl, ph, out=yp, row_start=plan)
        got = torch.full_like(want, 3.0)
        g.unpack_rows(yp, got, wl.seg_len, vl, plan)
        torch.cuda.synchronize()
        assert torch.equal(got, want), (ph, width)
    mk = lambda **kw: g.GsitStack([weights_to_dev(w, "bf16") for w in inp["fwd_layers"]],
                                  [weights_to_dev(w, "bf16") for w in inp["bwd_layers"]],
                                  [weights_to_dev(w, "bf16") for w in inp["intra_layers"]], wl.seg_len, wl.heads, ih, **kw)
    a = mk(packed=False).forward(x, vl).clone()
    for kw in (dict(), dict(intra_halves=False), dict(concurrent_rings=False), dict(paired_rings=False),
               dict(paired_rings=False, intra_halves=False), dict(paired_rings=False, concurrent_rings=False)):
        st = mk(**kw)
        b = st.forward(x, vl).clone()
        torch.cuda.synchronize()
        assert st.packed and torch.equal(a, b), kw
    assert g.last_device_status() == (0, 0)
