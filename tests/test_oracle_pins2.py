"""More oracle pins (no GPU): closed forms, the textbook special case against torch's attention,
symmetries, the pair count, the log-sum-exp output, the shared projection and the layer wrapper."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
import workloads as wk

PHASES = [oracle.PHASE_INTER_FWD, oracle.PHASE_INTER_BWD, oracle.PHASE_INTRA]


def _rand_qkv(rng, B, L, H, hd, scale=1.0):
    return tuple(scale * rng.standard_normal((B, L, H, hd)) for _ in range(3))


def _offsets(seg):
    return [0, seg[0], seg[0] + seg[1]]


# ---------------------------------------------------------------- P5: closed forms
@pytest.mark.parametrize("phase", PHASES)
def test_constant_values_give_constant_output(phase):
    rng = np.random.default_rng(1)
    seg, B, H, hd = (5, 6, 4), 2, 2, 3
    q, k, _ = _rand_qkv(rng, B, sum(seg), H, hd)
    c = rng.standard_normal(H * hd)
    v = np.broadcast_to(c.reshape(1, 1, H, hd), q.shape).copy()
    out = oracle.im_attention_dense(q, k, v, seg, None, phase)
    assert np.abs(out - c).max() <= 1e-14


@pytest.mark.parametrize("phase", PHASES)
def test_zero_queries_give_mean_of_allowed_valid_values(phase):
    rng = np.random.default_rng(2)
    seg, B, H, hd = (5, 6, 4), 2, 2, 3
    _, k, v = _rand_qkv(rng, B, sum(seg), H, hd)
    q = np.zeros_like(k)
    vl = np.array([[5, 3, 4], [2, 6, 1]], dtype=np.int32)
    out = oracle.im_attention_dense(q, k, v, seg, vl, phase)
    al = oracle.allowed_blocks(phase)
    off = _offsets(seg)
    for b in range(B):
        for s in range(3):
            r = int(np.argmax(al[s]))
            mean = v[b, off[r]:off[r] + vl[b, r]].reshape(vl[b, r], -1).mean(0)
            rows = out[b, off[s]:off[s] + vl[b, s]]
            assert np.abs(rows - mean).max() <= 1e-14


def test_single_valid_key_and_dominant_key():
    rng = np.random.default_rng(3)
    seg, H, hd = (4, 5, 3), 1, 4
    q, k, v = _rand_qkv(rng, 1, sum(seg), H, hd)
    off = _offsets(seg)
    vl = np.array([[4, 1, 3]], dtype=np.int32)          # segment 1 has one real key
    out = oracle.im_attention_dense(q, k, v, seg, vl, oracle.PHASE_INTER_FWD)  # seg 0 attends seg 1
    assert np.abs(out[0, :4] - v[0, off[1]].reshape(-1)).max() <= 1e-15
    # planted dominant key: key j* of segment 2 equals a multiple of the query direction
    q[0, off[1]:off[1] + 5] = np.array([1.0, 0, 0, 0])
    k[0, off[2]:off[2] + 3] = 0.0
    k[0, off[2] + 1] = np.array([1.0, 0, 0, 0])
    out = oracle.im_attention_dense(q, k, v, seg, None, oracle.PHASE_INTER_FWD, scale=1e3)
    assert np.abs(out[0, off[1]:off[1] + 5] - v[0, off[2] + 1].reshape(-1)).max() <= 1e-12


def test_empty_key_set_gives_zero_row_not_nan():
    rng = np.random.default_rng(4)
    seg, H, hd = (3, 4, 2), 2, 2
    q, k, v = _rand_qkv(rng, 2, sum(seg), H, hd)
    vl = np.array([[3, 0, 2], [3, 4, 2]], dtype=np.int32)   # sample 0: segment 1 fully padded
    out, lse = oracle.im_attention_dense(q, k, v, seg, vl, oracle.PHASE_INTER_FWD, want_lse=True)
    assert np.all(out[0, :3] == 0.0) and np.all(lse[0, :, :3] == -np.inf)
    assert np.isfinite(out).all()
    out = oracle.im_attention_dense(q, k, v, seg, None, oracle.PHASE_CUSTOM, 0b000000111)  # rows of seg 1, 2 closed
    assert np.all(out[:, 3:] == 0.0) and np.abs(out[:, :3]).min() > 0


# ---------------------------------------------------------------- P6: textbook special case vs library
@pytest.mark.parametrize("seg", [(17, 0, 0), (0, 9, 0), (0, 0, 13)])
def test_single_segment_intra_is_plain_self_attention(seg):
    rng = np.random.default_rng(6)
    B, H, hd, L = 2, 3, 5, sum(seg)
    q, k, v = _rand_qkv(rng, B, L, H, hd)
    out, lse = oracle.im_attention_dense(q, k, v, seg, None, oracle.PHASE_INTRA, want_lse=True)
    tq, tk, tv = (torch.from_numpy(a).transpose(1, 2) for a in (q, k, v))
    ref = F.scaled_dot_product_attention(tq, tk, tv).transpose(1, 2).reshape(B, L, H * hd).numpy()
    assert np.abs(out - ref).max() <= 1e-12
    ref_lse = torch.logsumexp(tq @ tk.transpose(-1, -2) / math.sqrt(hd), dim=-1).numpy()
    assert np.abs(lse - ref_lse).max() <= 1e-12


@pytest.mark.parametrize("phase", PHASES)
def test_against_library_attention_with_boolean_mask(phase):
    """Whole-sequence library attention with an independently built boolean mask."""
    rng = np.random.default_rng(7)
    seg, B, H, hd = (6, 8, 5), 2, 2, 4
    L = sum(seg)
    q, k, v = _rand_qkv(rng, B, L, H, hd)
    vl = np.array([[6, 4, 5], [3, 8, 2]], dtype=np.int32)
    seg_id = np.repeat(np.arange(3), seg)
    ring = {oracle.PHASE_INTER_FWD: 1, oracle.PHASE_INTER_BWD: 2, oracle.PHASE_INTRA: 0}[phase]
    block_open = (seg_id[None, :] == (seg_id[:, None] + ring) % 3)
    pad = wk.padded_row_mask(seg, vl, B)
    mask = torch.from_numpy(block_open[None, None] & ~pad[:, None, None, :])
    tq, tk, tv = (torch.from_numpy(a).transpose(1, 2) for a in (q, k, v))
    ref = F.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask).transpose(1, 2).reshape(B, L, H * hd).numpy()
    out = oracle.im_attention_dense(q, k, v, seg, vl, phase)
    assert np.abs(out[~pad] - ref[~pad]).max() <= 1e-12


# ---------------------------------------------------------------- P7: symmetries
def test_key_permutation_and_query_permutation():
    rng = np.random.default_rng(9)
    seg, H, hd = (5, 7, 6), 2, 3
    q, k, v = _rand_qkv(rng, 1, sum(seg), H, hd)
    off = _offsets(seg)
    base = oracle.im_attention_dense(q, k, v, seg, None, oracle.PHASE_INTER_FWD)
    perm = rng.permutation(seg[1])
    k2, v2 = k.copy(), v.copy()
    k2[:, off[1]:off[1] + seg[1]] = k[:, off[1] + perm]
    v2[:, off[1]:off[1] + seg[1]] = v[:, off[1] + perm]
    out = oracle.im_attention_dense(q, k2, v2, seg, None, oracle.PHASE_INTER_FWD)
    assert np.abs(out[:, :seg[0]] - base[:, :seg[0]]).max() <= 1e-14        # seg 0 attends seg 1
    qp = rng.permutation(seg[0])
    q2 = q.copy()
    q2[:, :seg[0]] = q[:, qp]
    out = oracle.im_attention_dense(q2, k, v, seg, None, oracle.PHASE_INTER_FWD)
    assert np.array_equal(out[:, :seg[0]], base[:, qp])


def test_ring_symmetries():
    rng = np.random.default_rng(10)
    n, H, hd = 5, 2, 3
    seg = (n, n, n)
    q, k, v = _rand_qkv(rng, 2, 3 * n, H, hd)
    fwd = oracle.im_attention_dense(q, k, v, seg, None, oracle.PHASE_INTER_FWD)
    rot = lambda a: np.concatenate([a[:, n:], a[:, :n]], axis=1)     # (0,1,2) -> (1,2,0)
    fwd_rot = oracle.im_attention_dense(rot(q), rot(k), rot(v), seg, None, oracle.PHASE_INTER_FWD)
    assert np.abs(fwd_rot - rot(fwd)).max() <= 1e-14
    # forward ring on order (0,1,2) == backward ring on order (0,2,1) after undoing the swap
    seg2 = (4, 6, 3)
    q, k, v = _rand_qkv(rng, 2, sum(seg2), H, hd)
    o = _offsets(seg2)
    swap = lambda a: np.concatenate([a[:, :o[1]], a[:, o[2]:], a[:, o[1]:o[2]]], axis=1)
    fwd = oracle.im_attention_dense(q, k, v, seg2, None, oracle.PHASE_INTER_FWD)
    bwd_sw = oracle.im_attention_dense(swap(q), swap(k), swap(v), (4, 3, 6), None, oracle.PHASE_INTER_BWD)
    assert np.abs(bwd_sw - swap(fwd)).max() <= 1e-14


# ---------------------------------------------------------------- P8: pair count
@pytest.mark.parametrize("phase", PHASES)
def test_pair_count_closed_form(phase):
    rng = np.random.default_rng(12)
    seg, B, H, hd = (7, 11, 9), 3, 2, 2
    q, k, v = _rand_qkv(rng, B, sum(seg), H, hd)
    _, pairs = oracle.im_attention_dense(q, k, v, seg, None, phase, want_pairs=True)
    Tt, Tv, Ta = seg
    expect = (Tt * Tv + Tt * Ta + Tv * Ta) if phase != oracle.PHASE_INTRA else (Tt * Tt + Tv * Tv + Ta * Ta)
    assert pairs == B * expect
    vl = np.stack([rng.integers(0, s + 1, size=B) for s in seg], axis=1).astype(np.int32)
    _, pairs = oracle.im_attention_dense(q, k, v, seg, vl, phase, want_pairs=True)
    assert pairs == wk.useful_pairs(seg, vl, oracle.allowed_blocks(phase), B)
    assert pairs == sum(int(vl[b, s]) * int(vl[b, r]) for b in range(B) for s in range(3) for r in range(3)
                        if oracle.allowed_blocks(phase)[s, r])


# ---------------------------------------------------------------- shared projection
def test_qkv_proj_against_matmul_and_sharing():
    rng = np.random.default_rng(13)
    seg, B, d, H = (4, 6, 5), 2, 8, 2
    x = rng.standard_normal((B, sum(seg), d))
    w = rng.standard_normal((3 * d, d))
    bias = rng.standard_normal(3 * d)
    vl = np.array([[4, 3, 5], [2, 6, 0]], dtype=np.int32)
    got = oracle.qkv_proj(x, w, bias, seg, H, vl)
    ref = (torch.from_numpy(x) @ torch.from_numpy(w).T + torch.from_numpy(bias)).numpy()
    pad = wk.padded_row_mask(seg, vl, B)
    flat = got.reshape(B, sum(seg), 3 * d)
    assert np.abs(flat[~pad] - ref[~pad]).max() <= 1e-13
    assert np.all(flat[pad] == 0.0)
    # layout [B, L, 3, H, hd]: index 0/1/2 are W_q / W_k / W_v rows
    assert np.abs(got[:, :, 1].reshape(B, -1, d)[~pad] - (x @ w[d:2 * d].T + bias[d:2 * d])[~pad]).max() <= 1e-13
    # NaN in padded input rows does not leak
    x2 = wk.fill_padding(x, seg, vl, np.nan)
    assert np.array_equal(oracle.qkv_proj(x2, w, bias, seg, H, vl), got)


# ---------------------------------------------------------------- P9: layer wrapper (textbook identities)
def _layer_weights(rng, d, d_ff, affine=True):
    w = wk.draw_layer_weights(rng, d, d_ff, "f32", affine=affine)
    return {k: (None if a is None else a.astype(np.float64)) for k, a in w.items()}


def test_layernorm_against_library():
    rng = np.random.default_rng(14)
    x = rng.standard_normal((5, 7, 16)) * 3 + 1
    g, b = rng.standard_normal(16), rng.standard_normal(16)
    ref = F.layer_norm(torch.from_numpy(x), (16,), torch.from_numpy(g), torch.from_numpy(b), 1e-5).numpy()
    assert np.abs(oracle.layernorm(x, g, b, 1e-5) - ref).max() <= 1e-13
    y = oracle.layernorm(x)
    assert np.abs(y.mean(-1)).max() <= 1e-14 and np.abs(y.var(-1) - 1).max() <= 1e-4


def test_layer_identity_and_ffn_only():
    rng = np.random.default_rng(15)
    seg, B, d, H, d_ff = (4, 6, 5), 2, 8, 2, 32
    x = rng.standard_normal((B, sum(seg), d))
    w = _layer_weights(rng, d, d_ff)
    vl = np.array([[4, 3, 5], [2, 6, 1]], dtype=np.int32)
    pad = wk.padded_row_mask(seg, vl, B)
    w0 = dict(w, w_o=np.zeros((d, d)), b_o=None, w_2=np.zeros((d, d_ff)), b_2=None)
    y = oracle.im_layer_fwd(x, w0, seg, H, vl, oracle.PHASE_INTRA)
    assert np.array_equal(y[~pad], x[~pad]) and np.all(y[pad] == 0.0)
    # attention disabled (all blocks closed) and no out-proj bias: y = x + FFN(LN2(x)) via library routines
    w1 = dict(w, b_o=None)
    y = oracle.im_layer_fwd(x, w1, seg, H, vl, oracle.PHASE_CUSTOM, 0)
    tx = torch.from_numpy(x)
    h = F.layer_norm(tx, (d,), torch.from_numpy(w["ln2_g"]), torch.from_numpy(w["ln2_b"]), 1e-5)
    ref = tx + F.linear(F.relu(F.linear(h, torch.from_numpy(w["w_1"]), torch.from_numpy(w["b_1"]))),
                        torch.from_numpy(w["w_2"]), torch.from_numpy(w["b_2"]))
    assert np.abs(y[~pad] - ref.numpy()[~pad]).max() <= 1e-12


@pytest.mark.parametrize("phase", PHASES)
def test_layer_against_library_composition(phase):
    rng = np.random.default_rng(16)
    seg, B, d, H, d_ff = (5, 7, 6), 2, 8, 2, 32
    L = sum(seg)
    x = rng.standard_normal((B, L, d))
    w = _layer_weights(rng, d, d_ff)
    vl = np.array([[5, 4, 6], [3, 7, 2]], dtype=np.int32)
    pad = wk.padded_row_mask(seg, vl, B)
    y = oracle.im_layer_fwd(x, w, seg, H, vl, phase)
    t = {k: (None if a is None else torch.from_numpy(a)) for k, a in w.items()}
    tx = torch.from_numpy(x)
    h = F.layer_norm(tx, (d,), t["ln1_g"], t["ln1_b"], 1e-5)
    qkv = F.linear(h, t["w_qkv"], t["b_qkv"]).view(B, L, 3, H, d // H)
    seg_id = np.repeat(np.arange(3), seg)
    ring = {oracle.PHASE_INTER_FWD: 1, oracle.PHASE_INTER_BWD: 2, oracle.PHASE_INTRA: 0}[phase]
    mask = torch.from_numpy((seg_id[None, :] == (seg_id[:, None] + ring) % 3)[None, None] & ~pad[:, None, None, :])
    att = F.scaled_dot_product_attention(qkv[:, :, 0].transpose(1, 2), qkv[:, :, 1].transpose(1, 2),
                                         qkv[:, :, 2].transpose(1, 2), attn_mask=mask)
    att = att.transpose(1, 2).reshape(B, L, d)
    y1 = tx + F.linear(att, t["w_o"], t["b_o"])
    h2 = F.layer_norm(y1, (d,), t["ln2_g"], t["ln2_b"], 1e-5)
    ref = y1 + F.linear(F.relu(F.linear(h2, t["w_1"], t["b_1"])), t["w_2"], t["b_2"])
    assert np.abs(y[~pad] - ref.numpy()[~pad]).max() <= 1e-11
    assert np.all(y[pad] == 0.0)
    # NaN in padded rows of x does not leak into real rows
    y_nan = oracle.im_layer_fwd(wk.fill_padding(x, seg, vl, np.nan), w, seg, H, vl, phase)
    assert np.array_equal(y_nan, y)


def test_stack_composition_shapes_and_concat():
    rng = np.random.default_rng(17)
    seg, B, d, H = (3, 4, 5), 1, 8, 2
    x = rng.standard_normal((B, sum(seg), d))
    fw = [_layer_weights(rng, d, 4 * d, False) for _ in range(2)]
    bw = [_layer_weights(rng, d, 4 * d, False) for _ in range(2)]
    iw = [_layer_weights(rng, 2 * d, 8 * d, False)]
    y = oracle.gsit_stack_fwd(x, fw, bw, iw, seg, H, H)
    assert y.shape == (B, sum(seg), 2 * d)
    # with the intra layer made an identity, the output is the feature concat of the two encoders
    iw0 = [dict(iw[0], w_o=np.zeros((2 * d, 2 * d)), w_2=np.zeros((2 * d, 8 * d)))]
    y = oracle.gsit_stack_fwd(x, fw, bw, iw0, seg, H, H)
    a = x
    for w in fw:
        a = oracle.im_layer_fwd(a, w, seg, H, None, oracle.PHASE_INTER_FWD)
    b = x
    for w in bw:
        b = oracle.im_layer_fwd(b, w, seg, H, None, oracle.PHASE_INTER_BWD)
    assert np.array_equal(y[..., :d], a) and np.array_equal(y[..., d:], b)


def _torch_layer(tx, t, seg, pad, H, ring):
    """One IM layer out of torch library routines (LayerNorm, linear, SDPA with a boolean mask built here from segment
    ids); `ring` is the key-segment shift of the block pattern: 1 forward, 2 backward, 0 intra."""
    B, L, d = tx.shape
    h = F.layer_norm(tx, (d,), t["ln1_g"], t["ln1_b"], 1e-5)
    qkv = F.linear(h, t["w_qkv"], t["b_qkv"]).view(B, L, 3, H, d // H)
    seg_id = np.repeat(np.arange(3), seg)
    mask = torch.from_numpy((seg_id[None, :] == (seg_id[:, None] + ring) % 3)[None, None] & ~pad[:, None, None, :])
    att = F.scaled_dot_product_attention(qkv[:, :, 0].transpose(1, 2), qkv[:, :, 1].transpose(1, 2),
                                         qkv[:, :, 2].transpose(1, 2), attn_mask=mask)
    att = att.transpose(1, 2).reshape(B, L, d)
    y1 = tx + F.linear(att, t["w_o"], t["b_o"])
    h2 = F.layer_norm(y1, (d,), t["ln2_g"], t["ln2_b"], 1e-5)
    y = y1 + F.linear(F.relu(F.linear(h2, t["w_1"], t["b_1"])), t["w_2"], t["b_2"])
    return torch.where(torch.from_numpy(pad)[:, :, None], torch.zeros_like(y), y)


def test_stack_against_library_composition_with_distinct_intra_heads():
    """Eq. "All-Modal-In-One fusion": G_inter^{forward} and G_inter^{backward} encoders from the same input with their own
    weights, feature concat, then the G_intra encoder -- here with a head count different from the ring encoders', two
    layers per encoder, affine LayerNorms, biases and ragged lengths, composed independently from torch routines.  A wrong
    block pattern, head count or operand order in any leg of oracle.gsit_stack_fwd moves the result far beyond 1e-10."""
    rng = np.random.default_rng(18)
    seg, B, d, H, IH = (5, 7, 6), 2, 8, 2, 4
    x = rng.standard_normal((B, sum(seg), d))
    vl = np.array([[5, 4, 6], [3, 7, 2]], dtype=np.int32)
    pad = wk.padded_row_mask(seg, vl, B)
    fw = [_layer_weights(rng, d, 4 * d) for _ in range(2)]
    bw = [_layer_weights(rng, d, 4 * d) for _ in range(2)]
    iw = [_layer_weights(rng, 2 * d, 8 * d) for _ in range(2)]
    got = oracle.gsit_stack_fwd(x, fw, bw, iw, seg, H, IH, vl)
    tt = lambda w: {k: (None if a is None else torch.from_numpy(a)) for k, a in w.items()}
    a = b = torch.from_numpy(x)
    for w in fw:
        a = _torch_layer(a, tt(w), seg, pad, H, 1)
    for w in bw:
        b = _torch_layer(b, tt(w), seg, pad, H, 2)
    c = torch.cat([a, b], dim=-1)
    for w in iw:
        c = _torch_layer(c, tt(w), seg, pad, IH, 0)
    ref = c.numpy()
    assert np.abs(got[~pad] - ref[~pad]).max() <= 1e-10
    assert np.all(got[pad] == 0.0)
    # the pins bite: the ring head count in the intra leg, or the rings swapped, is far outside the bound
    wrong_heads = oracle.gsit_stack_fwd(x, fw, bw, iw, seg, H, H, vl)
    swapped = oracle.gsit_stack_fwd(x, bw, fw, iw, seg, H, IH, vl)
    assert np.abs(wrong_heads[~pad] - ref[~pad]).max() > 1e-4 and np.abs(swapped[~pad] - ref[~pad]).max() > 1e-4


def test_workload_generators_are_seeded_and_shaped():
    a, b = wk.make_inputs(3, batch=2), wk.make_inputs(3, batch=2)
    assert np.array_equal(a["x"], b["x"]) and np.array_equal(a["valid_len"], b["valid_len"])
    wl = wk.WORKLOADS[3]
    assert a["x"].shape == (2, wl.L, wl.d_model)
    assert (a["valid_len"] >= (np.asarray(wl.seg_len) + 1) // 2).all() and (a["valid_len"] <= wl.seg_len).all()
    assert np.array_equal(wk.round_to_bf16(a["x"]), a["x"])          # already bf16-representable
    v5 = wk.draw_valid_len(np.random.default_rng(0), wk.WORKLOADS[5], 8)
    assert (v5[3] == (64, 512, 512)).all() and (v5[0] == (128, 1024, 1024)).all()
    r = wk.round_to_bf16(np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.00390625], np.float32))
    assert r[0] == 1.0 and r[1] == 1.015625 and r[2] == 1.0
    # second family: lengths around the dataset averages stay inside [1, max]; the other shapes keep the half-length floor
    v6 = wk.draw_valid_len(np.random.default_rng(1), wk.WORKLOADS[6], 4000)
    assert (v6 >= 1).all() and (v6 <= (50, 500, 500)).all()
    assert abs(v6[:, 0].mean() - 24) < 2 and abs(v6[:, 2].mean() - 94) < 6 and v6[:, 1].mean() < 190
    for idx in (7, 8):
        w = wk.WORKLOADS[idx]
        v = wk.draw_valid_len(np.random.default_rng(2), w, 64)
        assert (v >= (np.asarray(w.seg_len) + 1) // 2).all() and (v <= w.seg_len).all()
        assert wk.make_inputs(idx, batch=2)["x"].shape == (2, w.L, 64)


def test_stack_head_picks_last_real_step_of_each_modality():
    """Eq. "All-Modal-In-One fusion", X_m = f(|| Split(.)[-1]): with a selection matrix for f the read-out must return
    exactly the last real row of each segment; without padding that is the last row of the segment; an empty segment
    gives zeros; a general f agrees with a matrix product on the gathered rows."""
    rng = np.random.default_rng(12)
    seg, B, dc = (4, 7, 5), 3, 6
    c = rng.standard_normal((B, sum(seg), dc))
    ident = np.eye(3 * dc)
    out = oracle.stack_head_fwd(c, ident, None, seg, None)
    assert np.array_equal(out, np.concatenate([c[:, 3], c[:, 10], c[:, 15]], axis=1))
    valid = np.array([[4, 7, 5], [1, 3, 2], [2, 0, 5]], dtype=np.int32)
    out = oracle.stack_head_fwd(c, ident, None, seg, valid)
    assert np.array_equal(out[1], np.concatenate([c[1, 0], c[1, 4 + 2], c[1, 11 + 1]]))
    assert np.array_equal(out[2], np.concatenate([c[2, 1], np.zeros(dc), c[2, 15]]))
    w, bias = rng.standard_normal((9, 3 * dc)), rng.standard_normal(9)
    got = oracle.stack_head_fwd(c, w, bias, seg, valid)
    assert np.allclose(got, oracle.stack_head_fwd(c, ident, None, seg, valid) @ w.T + bias, rtol=0, atol=1e-12)
