"""GPU edge cases and properties: ragged / empty segments, every supported head width and slice width,
custom block patterns (union softmax), separate vs fused q/k/v, explicit scale, bit-exact padding,
run-to-run determinism, device status flags and host-side argument rejection."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import workloads as wk
from gpu_util import check_close, pad_mask, to_dev, to_np64

pytestmark = pytest.mark.gpu
PHASES = [oracle.PHASE_INTER_FWD, oracle.PHASE_INTER_BWD, oracle.PHASE_INTRA]


@pytest.fixture(scope="module")
def g():
    import paper_2505_01068_b200 as lib
    lib.load()
    return lib


def _run(g, q, k, v, seg, valid, phase, dtype, custom=0, scale=0.0, nan_pad=True):
    B = q.shape[0]
    pm = pad_mask(seg, valid, B)
    qd, kd, vd = (to_dev(wk.fill_padding(a, seg, valid, np.nan) if (nan_pad and valid is not None) else a, dtype)
                  for a in (q, k, v))
    vl = None if valid is None else torch.from_numpy(valid).cuda()
    out, lse = g.im_attention_fwd(qd, kd, vd, seg, vl, phase, custom, scale, want_lse=True)
    ref, ref_lse = oracle.im_attention_dense(q, k, v, seg, valid, phase, custom, scale, want_lse=True)
    check_close(to_np64(out), ref, dtype, pm, f"seg={seg} phase={phase} custom={custom:#x}")
    gl = to_np64(lse)
    assert np.array_equal(np.isneginf(gl), np.isneginf(ref_lse))
    fin = np.isfinite(ref_lse)
    if fin.any():
        assert np.abs(gl[fin] - ref_lse[fin]).max() <= (1e-4 if dtype == "f32" else 2e-2)
    return out


@pytest.mark.parametrize("H,hd", [(8, 8), (4, 16), (2, 32), (1, 64), (4, 8), (2, 16), (1, 32), (2, 8), (1, 16),
                                  (16, 8), (8, 16), (4, 64), (12, 8), (6, 16), (3, 32), (10, 8)])
def test_bf16_every_head_and_slice_width(g, H, hd):
    """d = H*hd covers slice widths 64, 32 and 16 and every supported head_dim; ragged lengths, several key
    tiles, a ragged last tile, a one-row segment."""
    rng = np.random.default_rng(100 + H * 64 + hd)
    seg, B = (37, 150, 1), 3
    q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, "bf16")
    valid = np.array([[37, 150, 1], [20, 65, 1], [1, 129, 0]], dtype=np.int32)
    for ph in PHASES:
        _run(g, q, k, v, seg, valid, ph, "bf16")


@pytest.mark.parametrize("seg", [(0, 70, 33), (64, 0, 128), (5, 5, 0), (130, 1, 1), (1, 1, 1), (200, 0, 0)])
def test_bf16_empty_and_tiny_segments(g, seg):
    rng = np.random.default_rng(sum(seg))
    B, H, hd = 2, 8, 8
    q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, "bf16")
    valid = np.stack([rng.integers(0, s + 1, size=B) for s in seg], axis=1).astype(np.int32)
    for ph in PHASES:
        _run(g, q, k, v, seg, None, ph, "bf16")
        _run(g, q, k, v, seg, valid, ph, "bf16")


def test_random_shapes_property(g):
    rng = np.random.default_rng(2024)
    for it in range(12):
        H, hd = [(8, 8), (4, 16), (2, 32), (2, 64), (4, 8)][it % 5]
        seg = tuple(int(s) for s in rng.integers(0, 180, size=3))
        if sum(seg) == 0:
            seg = (3, 0, 0)
        B = int(rng.integers(1, 4))
        q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, "bf16")
        valid = np.stack([rng.integers(0, s + 1, size=B) for s in seg], axis=1).astype(np.int32)
        ph = PHASES[it % 3]
        _run(g, q, k, v, seg, valid, ph, "bf16")
        qf, kf, vf = (a[:, :, : max(1, H // 2)].copy() for a in (q, k, v))
        _run(g, qf, kf, vf, seg, valid, ph, "f32")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_custom_block_patterns_union_softmax(g, dtype):
    rng = np.random.default_rng(31)
    seg, B, H, hd = (40, 90, 70), 2, 4, 8
    q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, dtype)
    valid = np.array([[40, 50, 70], [13, 90, 33]], dtype=np.int32)
    # naive unmasked graph, "disorder" pattern with two open blocks in row 0, a closed row, ablation-like pattern
    for bits in (0x1FF, 0b001100110, 0b110000000, 0b100100100, 0):
        _run(g, q, k, v, seg, valid, oracle.PHASE_CUSTOM, dtype, custom=bits)


@pytest.mark.parametrize("H,hd", [(4, 16), (2, 32), (2, 64), (8, 16), (1, 64)])
def test_custom_block_patterns_every_head_width(g, H, hd):
    """The union walk (two and three open blocks in a block row, a closed row, the empty mask) in every bf16 kernel
    family: head_dim 16 and 32, and head_dim 64 (the tensor-memory kernel), over several key tiles per open block,
    ragged last tiles and an empty key segment."""
    rng = np.random.default_rng(500 + H * 64 + hd)
    seg, B = (70, 200, 150), 3
    q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, "bf16")
    valid = np.array([[70, 200, 150], [33, 129, 65], [70, 0, 1]], dtype=np.int32)
    # unmasked naive graph; two open blocks in rows 0 and 1 with row 2 closed; three in row 2 only; a permutation-like
    # ablation pattern; one block; nothing open
    for bits in (0x1FF, 0b000101011, 0b111000000, 0b010001100, 0b000010000, 0):
        _run(g, q, k, v, seg, valid, oracle.PHASE_CUSTOM, "bf16", custom=bits)
        _run(g, q, k, v, seg, None, oracle.PHASE_CUSTOM, "bf16", custom=bits, nan_pad=False)


@pytest.mark.parametrize("choice", ["ATTN_TMEM", "ATTN_LEGACY"])
def test_bf16_both_kernel_families_at_every_head_width(g, choice):
    """The tensor-memory attention at head_dim 8 (not its default there) and the mma.sync attention at head_dim 16 / 32 / 64
    (not the default there): every kernel that can be selected meets the oracle on ragged inputs with custom patterns."""
    rng = np.random.default_rng(77)
    seg, B = (50, 170, 129), 3
    valid = np.array([[50, 170, 129], [25, 65, 33], [1, 0, 128]], dtype=np.int32)
    g.tune_attention(getattr(g, choice))
    try:
        for H, hd in ((8, 8), (4, 8), (4, 16), (2, 32), (2, 64)):
            q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, "bf16")
            for ph, bits in ((oracle.PHASE_INTER_FWD, 0), (oracle.PHASE_INTRA, 0), (oracle.PHASE_CUSTOM, 0b000101011)):
                _run(g, q, k, v, seg, valid, ph, "bf16", custom=bits)
    finally:
        g.tune_attention(g.ATTN_DEFAULT)


def test_attention_with_and_without_scratch_gives_the_same_bits(g):
    """The optional scratch of gsit_im_attention_fwd only changes which SM takes which work item."""
    rng = np.random.default_rng(78)
    seg, B, H, hd = (50, 300, 270), 4, 8, 16
    q, k, v = (to_dev(a, "bf16") for a in wk.draw_qkv(rng, B, sum(seg), H, hd, "bf16"))
    vl = torch.from_numpy(np.array([[50, 300, 270], [25, 151, 200], [50, 1, 135], [13, 299, 64]], dtype=np.int32)).cuda()
    lib = g.load()
    sh = g.make_shape(B, seg, H * hd, H, vl, g.DTYPE_BF16, g.PHASE_INTER_BWD)
    outs = []
    for ws in (None, torch.full((256,), 0xAB, dtype=torch.uint8, device="cuda")):
        out = torch.empty((B, sum(seg), H * hd), dtype=torch.bfloat16, device="cuda")
        code = lib.gsit_im_attention_fwd(ctypes.byref(sh), q.data_ptr(), k.data_ptr(), v.data_ptr(), H * hd, out.data_ptr(), None,
                                         None if ws is None else ws.data_ptr(), 0 if ws is None else ws.numel(), None)
        assert code == 0
        torch.cuda.synchronize()
        outs.append(out)
    assert torch.equal(outs[0], outs[1])
    assert g.last_device_status() == (0, 0)


@pytest.mark.parametrize("H,hd", [(2, 64), (4, 16), (8, 8), (2, 32)])
def test_attention_on_packed_rows_equals_padded_layout(g, H, hd):
    """gsit_im_attention_fwd on the packed row layout (q, k, v and out hold real rows only) against the padded layout, for
    every bf16 kernel family: the same bits in every real row, and nothing written outside them."""
    rng = np.random.default_rng(900 + hd)
    seg, B = (70, 200, 150), 4
    d = H * hd
    valid = np.array([[70, 200, 150], [33, 129, 65], [70, 0, 1], [0, 0, 0]], dtype=np.int32)
    vl = torch.from_numpy(valid).cuda()
    q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, "bf16")
    qkv = torch.stack([to_dev(a, "bf16") for a in (q, k, v)], dim=2).contiguous()          # [B, L, 3, H, hd]
    want = g.im_attention_fwd(qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2], seg, vl, oracle.PHASE_INTER_FWD)
    L, cap = sum(seg), B * sum(seg) + 128
    plan = g.plan_rows(vl, seg)
    plan_h = plan.cpu().numpy()
    packed = torch.full((cap, 3 * d), float("nan"), dtype=torch.bfloat16, device="cuda")
    off = np.cumsum([0] + list(seg))
    flat = qkv.reshape(B, L, 3 * d)
    for b in range(B):
        for s_ in range(3):
            n = int(valid[b, s_])
            packed[plan_h[3 * b + s_]:plan_h[3 * b + s_] + n] = flat[b, off[s_]:off[s_] + n]
    out = torch.full((cap, d), 7.0, dtype=torch.bfloat16, device="cuda")
    sh = g.make_shape(B, seg, d, H, vl, g.DTYPE_BF16, g.PHASE_INTER_FWD, row_start=plan, capacity=cap)
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    lib = g.load()
    es = 2
    code = lib.gsit_im_attention_fwd(ctypes.byref(sh), packed.data_ptr(), packed.data_ptr() + d * es, packed.data_ptr() + 2 * d * es, 3 * d,
                                     out.data_ptr(), None, ws.data_ptr(), ws.numel(), None)
    assert code == 0
    torch.cuda.synchronize()
    used = int(plan_h[-1])
    for b in range(B):
        for s_ in range(3):
            n = int(valid[b, s_])
            assert torch.equal(out[plan_h[3 * b + s_]:plan_h[3 * b + s_] + n], want[b, off[s_]:off[s_] + n]), (b, s_)
    assert bool((out[used:] == 7.0).all())
    assert g.last_device_status() == (0, 0)


def test_projection_on_packed_rows_equals_padded_layout_and_leaves_other_rows_alone(g):
    """gsit_im_qkv_proj on the packed row layout: the real rows get the bits of the padded layout; a call on a sub-range
    of the samples writes their rows only (tiles at the edges of the range are shared with the neighbours)."""
    rng = np.random.default_rng(77)
    seg, B, d, H = (70, 200, 150), 5, 128, 8
    L = sum(seg)
    valid = np.array([[70, 200, 150], [33, 129, 65], [70, 0, 1], [0, 0, 0], [61, 77, 150]], dtype=np.int32)
    vl = torch.from_numpy(valid).cuda()
    x = to_dev(rng.standard_normal((B, L, d)).astype(np.float32), "bf16")
    w = to_dev((rng.standard_normal((3 * d, d)) * d ** -0.5).astype(np.float32), "bf16")
    bias = to_dev(rng.standard_normal(3 * d).astype(np.float32))
    want = g.im_qkv_proj(x, w, bias, seg, H, vl).reshape(B, L, 3 * d)
    cap = B * L + 128
    plan = g.plan_rows(vl, seg)
    plan_h = plan.cpu().numpy()
    off = np.cumsum([0] + list(seg))
    xp = torch.full((cap, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    for b in range(B):
        for s_ in range(3):
            n = int(valid[b, s_])
            xp[plan_h[3 * b + s_]:plan_h[3 * b + s_] + n] = x[b, off[s_]:off[s_] + n]
    for lo, hi in ((0, B), (1, 3), (4, 5)):
        out = torch.full((cap, 3, H, d // H), 7.0, dtype=torch.bfloat16, device="cuda")
        g.im_qkv_proj(xp, w, bias, seg, H, vl[lo:hi], out=out, row_start=plan[3 * lo:])
        torch.cuda.synchronize()
        flat = out.reshape(cap, 3 * d)
        begin, end = int(plan_h[3 * lo]), int(plan_h[3 * hi])
        for b in range(lo, hi):
            for s_ in range(3):
                n = int(valid[b, s_])
                assert torch.equal(flat[plan_h[3 * b + s_]:plan_h[3 * b + s_] + n], want[b, off[s_]:off[s_] + n]), (lo, hi, b, s_)
        assert bool((flat[:begin] == 7.0).all()) and bool((flat[end:] == 7.0).all()), (lo, hi)
    assert g.last_device_status() == (0, 0)


def test_bounded_wait_runs_out_and_is_reported(g):
    """A device-side wait that nothing will ever satisfy gives up after its poll limit: the kernel returns, the status
    word carries the timeout flag exactly once, and the next ordinary call is clean."""
    assert g.last_device_status() == (0, 0)
    g.expire_wait_selftest()
    code, flags = g.last_device_status()
    assert code == 5 and flags & g.DEVFLAG_TIMEOUT and g.status_string(code) == "device-side wait timed out"
    assert g.last_device_status() == (0, 0)
    rng = np.random.default_rng(79)
    seg = (20, 70, 33)
    q, k, v = wk.draw_qkv(rng, 2, sum(seg), 4, 16, "bf16")
    _run(g, q, k, v, seg, None, oracle.PHASE_INTRA, "bf16")
    assert g.last_device_status() == (0, 0)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_explicit_scale_and_fused_vs_separate(g, dtype):
    rng = np.random.default_rng(32)
    seg, B, H, hd = (30, 75, 66), 2, 4, 16
    q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, dtype)
    out_sep = _run(g, q, k, v, seg, None, oracle.PHASE_INTER_BWD, dtype, scale=0.4)
    fused = torch.stack([to_dev(a, dtype) for a in (q, k, v)], dim=2).contiguous()   # [B, L, 3, H, hd]
    out_fused = g.im_attention_fwd(fused[:, :, 0], fused[:, :, 1], fused[:, :, 2], seg, None, oracle.PHASE_INTER_BWD,
                                   scale=0.4)
    assert torch.equal(out_sep, out_fused)


def test_f32_large_head_dim_and_masking(g):
    rng = np.random.default_rng(33)
    seg, B, H, hd = (9, 20, 14), 2, 2, 40
    q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, "f32")
    valid = np.array([[9, 0, 14], [4, 20, 1]], dtype=np.int32)
    for ph in PHASES:
        _run(g, q, k, v, seg, valid, ph, "f32")


def test_masked_blocks_do_not_influence_gpu_output(g):
    """Information-disorder invariant on the GPU: keys/values of closed blocks and padded rows may hold anything."""
    rng = np.random.default_rng(34)
    seg, B, H, hd = (50, 100, 80), 2, 8, 8
    q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, "bf16")
    valid = np.array([[50, 70, 80], [25, 100, 41]], dtype=np.int32)
    vl = torch.from_numpy(valid).cuda()
    off = [0, 50, 150]
    base = g.im_attention_fwd(*(to_dev(a, "bf16") for a in (q, k, v)), seg, vl, oracle.PHASE_INTER_FWD)
    al = oracle.allowed_blocks(oracle.PHASE_INTER_FWD)
    for s in range(3):
        k2, v2 = k.copy(), v.copy()
        for r in range(3):
            if not al[s, r]:
                k2[:, off[r]:off[r] + seg[r]] = np.inf
                v2[:, off[r]:off[r] + seg[r]] = np.nan
        k2, v2 = (wk.fill_padding(a, seg, valid, np.nan) for a in (k2, v2))
        out = g.im_attention_fwd(*(to_dev(a, "bf16") for a in (q, k2, v2)), seg, vl, oracle.PHASE_INTER_FWD)
        assert torch.equal(out[:, off[s]:off[s] + seg[s]], base[:, off[s]:off[s] + seg[s]])


def test_run_to_run_bit_identical(g):
    inp = wk.make_inputs(3, batch=4)
    wl = inp["workload"]
    vl = torch.from_numpy(inp["valid_len"]).cuda()
    qkv = g.im_qkv_proj(to_dev(inp["x"], "bf16"), to_dev(inp["layer"]["w_qkv"], "bf16"), None, wl.seg_len, wl.heads, vl)
    outs = [g.im_attention_fwd(qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2], wl.seg_len, vl, oracle.PHASE_INTRA).clone()
            for _ in range(3)]
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


def test_out_of_range_valid_len_is_clamped_and_flagged(g):
    rng = np.random.default_rng(35)
    seg, B, H, hd = (20, 30, 25), 2, 4, 8
    q, k, v = wk.draw_qkv(rng, B, sum(seg), H, hd, "bf16")
    bad = np.array([[25, 30, -3], [20, 99, 25]], dtype=np.int32)
    clamped = np.clip(bad, 0, np.array(seg)[None]).astype(np.int32)
    g.last_device_status()
    out = g.im_attention_fwd(*(to_dev(a, "bf16") for a in (q, k, v)), seg, torch.from_numpy(bad).cuda(),
                             oracle.PHASE_INTER_FWD)
    code, flags = g.last_device_status()
    assert code == 0 and flags == g.DEVFLAG_CLAMPED
    ref = oracle.im_attention_dense(q, k, v, seg, clamped, oracle.PHASE_INTER_FWD)
    check_close(to_np64(out), ref, "bf16", pad_mask(seg, clamped, B), "clamped")
    assert g.last_device_status() == (0, 0)


def test_host_side_rejection(g):
    lib = g.load()
    dev = torch.device("cuda")
    t = torch.zeros((1, 16, 64), dtype=torch.bfloat16, device=dev)
    ok = g.make_shape(1, (4, 8, 4), 64, 8, None, g.DTYPE_BF16, g.PHASE_INTRA)
    p = t.data_ptr()
    o_buf = torch.zeros_like(t)
    call = lambda sh, q=p, k=p, v=p, rs=64, o=o_buf.data_ptr(): lib.gsit_im_attention_fwd(ctypes.byref(sh), q, k, v, rs, o, None, None, 0, None)
    assert call(ok) == 0
    assert call(ok, q=None) == 1 and call(ok, rs=32) == 1 and call(ok, q=p + 2) == 1 and call(ok, rs=68) == 1
    assert call(g.make_shape(1, (4, 8, 4), 64, 7, None, g.DTYPE_BF16, g.PHASE_INTRA)) == 1      # d % heads
    assert call(g.make_shape(0, (4, 8, 4), 64, 8, None, g.DTYPE_BF16, g.PHASE_INTRA)) == 1      # batch
    assert call(g.make_shape(1, (4, -8, 4), 64, 8, None, g.DTYPE_BF16, g.PHASE_INTRA)) == 1     # negative length
    assert call(g.make_shape(1, (0, 0, 0), 64, 8, None, g.DTYPE_BF16, g.PHASE_INTRA)) == 1      # empty sequence
    assert call(g.make_shape(1, (4, 8, 4), 64, 8, None, g.DTYPE_BF16, 7)) == 1                  # bad phase
    assert call(g.make_shape(1, (4, 8, 4), 64, 8, None, g.DTYPE_BF16, g.PHASE_CUSTOM, 0x400)) == 1
    assert call(g.make_shape(1, (4, 8, 4), 64, 8, None, 5, g.PHASE_INTRA)) == 1                 # bad dtype
    assert call(g.make_shape(1, (4, 8, 4), 64, 16, None, g.DTYPE_BF16, g.PHASE_INTRA)) == 2     # head_dim 4 unsupported
    assert call(g.make_shape(1, (4, 8, 4), 24, 3, None, g.DTYPE_BF16, g.PHASE_INTRA)) == 2      # d % 16
    # layer: workspace too small / missing
    w = {k_: torch.zeros(s, dtype=torch.bfloat16, device=dev) for k_, s in
         (("w_qkv", (192, 64)), ("w_o", (64, 64)), ("w_1", (256, 64)), ("w_2", (64, 256)))}
    x = torch.zeros((1, 16, 64), dtype=torch.float32, device=dev)
    with pytest.raises(g.GsitError) as e:
        g.im_layer_fwd(x, w, (4, 8, 4), 8, workspace=torch.empty(256, dtype=torch.uint8, device=dev))
    assert e.value.code == 3
    assert g.workspace_bytes(ok, g.CALL_ATTENTION) <= 4096 and g.workspace_bytes(ok, g.CALL_LAYER, 256) > 0
    torch.cuda.synchronize()
