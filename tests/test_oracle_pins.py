"""Pins for the CPU oracle (no GPU): each test checks the oracle against something other than itself --
the block patterns the paper prints, the paper's equivalence between masked and decomposed attention,
a per-vertex brute force written from the GAT equations, closed forms, a library routine, symmetries
and the closed-form pair count."""
import math
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
import workloads as wk

PHASES = [oracle.PHASE_INTER_FWD, oracle.PHASE_INTER_BWD, oracle.PHASE_INTRA]
GOLDEN = Path(__file__).resolve().parent / "golden"


def _rand_qkv(rng, B, L, H, hd, scale=1.0):
    return tuple(scale * rng.standard_normal((B, L, H, hd)) for _ in range(3))


def _offsets(seg):
    return [0, seg[0], seg[0] + seg[1]]


# ---------------------------------------------------------------- printed block patterns (Eq. IFM / IEM)
def _read_golden_masks():
    blocks, name = {}, None
    for line in (GOLDEN / "im_masks.txt").read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("["):
            name = line.strip("[]")
            blocks[name] = []
        else:
            blocks[name].append([1 if c == "O" else 0 for c in line.split()])
    return {k: np.array(v) for k, v in blocks.items()}


def test_block_patterns_match_printed_masks():
    g = _read_golden_masks()
    assert (oracle.allowed_blocks(oracle.PHASE_INTER_FWD) == g["inter_forward"]).all()
    assert (oracle.allowed_blocks(oracle.PHASE_INTER_BWD) == g["inter_backward"]).all()
    assert (oracle.allowed_blocks(oracle.PHASE_INTRA) == g["intra"]).all()
    # two opposing unidirectional rings: each is a permutation, together with intra they tile the 3x3 grid
    total = sum(oracle.allowed_blocks(p) for p in PHASES)
    assert (total == 1).all()
    assert (oracle.allowed_blocks(oracle.PHASE_INTER_FWD).T == oracle.allowed_blocks(oracle.PHASE_INTER_BWD)).all()


def test_custom_mask_bits():
    for bits in (0, 0b111111111, 0b000010001, 0b100000110):
        a = oracle.allowed_blocks(oracle.PHASE_CUSTOM, bits)
        for s in range(3):
            for r in range(3):
                assert a[s, r] == (bits >> (3 * s + r)) & 1


def test_dense_mask_expands_blocks_and_padding():
    seg = (3, 4, 2)
    g = _read_golden_masks()["inter_forward"]
    n = [2, 4, 1]
    M = oracle.dense_mask(seg, n, g)
    off = _offsets(seg)
    for p in range(9):
        sp = max(s for s in range(3) if p >= off[s])
        for q in range(9):
            sq = max(s for s in range(3) if q >= off[s])
            open_ = g[sp, sq] == 1 and (q - off[sq]) < n[sq]
            assert M[p, q] == (0.0 if open_ else -math.inf)


# ---------------------------------------------------------------- P1: masked-dense == decomposed
@pytest.mark.parametrize("phase", PHASES)
@pytest.mark.parametrize("seg,H,hd", [((8, 12, 10), 4, 8), ((5, 1, 7), 2, 3), ((6, 0, 9), 1, 4)])
def test_dense_equals_decomposed(phase, seg, H, hd):
    rng = np.random.default_rng(11 + phase)
    B, L = 3, sum(seg)
    q, k, v = _rand_qkv(rng, B, L, H, hd)
    vl = np.stack([rng.integers(0, s + 1, size=B) for s in seg], axis=1).astype(np.int32)
    for valid in (None, vl):
        a = oracle.im_attention_dense(q, k, v, seg, valid, phase)
        b = oracle.im_attention_decomposed(q, k, v, seg, valid, phase)
        assert np.abs(a - b).max() <= 1e-12


def test_dense_equals_decomposed_custom_union():
    rng = np.random.default_rng(5)
    seg, B, H, hd = (4, 6, 5), 2, 2, 4
    q, k, v = _rand_qkv(rng, B, sum(seg), H, hd)
    vl = np.array([[4, 3, 5], [2, 6, 0]], dtype=np.int32)
    for bits in (0b111111111, 0b000000110, 0b010101010, 0b001000000, 0):
        a = oracle.im_attention_dense(q, k, v, seg, vl, oracle.PHASE_CUSTOM, bits)
        b = oracle.im_attention_decomposed(q, k, v, seg, vl, oracle.PHASE_CUSTOM, bits)
        assert np.abs(a - b).max() <= 1e-12


def test_equals_separately_computed_cross_modal_attention_with_shared_weights():
    """The IM-masked attention over [V_0;V_1;V_2] with shared W equals the three bi-modal cross-modal
    attentions computed one by one with torch's library attention (Section "Motivation")."""
    rng = np.random.default_rng(3)
    seg, B, H, d = (5, 7, 6), 2, 2, 8
    x = rng.standard_normal((B, sum(seg), d))
    w = rng.standard_normal((3 * d, d)) / math.sqrt(d)
    qkv = oracle.qkv_proj(x, w, None, seg, H)
    q, k, v = qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2]
    off = _offsets(seg)
    for phase in PHASES:
        out = oracle.im_attention_dense(q, k, v, seg, None, phase)
        al = oracle.allowed_blocks(phase)
        for i in range(3):
            j = int(np.argmax(al[i]))
            xi = torch.from_numpy(x[:, off[i]:off[i] + seg[i]])
            xj = torch.from_numpy(x[:, off[j]:off[j] + seg[j]])
            W = torch.from_numpy(w)
            qi = (xi @ W[:d].T).view(B, seg[i], H, d // H).transpose(1, 2)
            kj = (xj @ W[d:2 * d].T).view(B, seg[j], H, d // H).transpose(1, 2)
            vj = (xj @ W[2 * d:].T).view(B, seg[j], H, d // H).transpose(1, 2)
            ref = torch.nn.functional.scaled_dot_product_attention(qi, kj, vj).transpose(1, 2).reshape(B, seg[i], d)
            assert np.abs(out[:, off[i]:off[i] + seg[i]] - ref.numpy()).max() <= 1e-12


# ---------------------------------------------------------------- P2: masked-block invariance
@pytest.mark.parametrize("phase", PHASES)
def test_masked_blocks_and_padding_do_not_influence_output(phase):
    rng = np.random.default_rng(21)
    seg, B, H, hd = (6, 9, 7), 2, 2, 4
    L = sum(seg)
    q, k, v = _rand_qkv(rng, B, L, H, hd)
    vl = np.array([[6, 5, 7], [3, 9, 4]], dtype=np.int32)
    base = oracle.im_attention_dense(q, k, v, seg, vl, phase)
    al = oracle.allowed_blocks(phase)
    off = _offsets(seg)
    pad = wk.padded_row_mask(seg, vl, B)
    # padded rows of q, k, v become NaN
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[pad] = np.nan
    k2[pad] = np.nan
    v2[pad] = np.nan
    assert np.array_equal(oracle.im_attention_dense(q2, k2, v2, seg, vl, phase), base)
    # per query segment: keys/values of every closed segment replaced by huge values
    for s in range(3):
        k3, v3 = k.copy(), v.copy()
        for r in range(3):
            if not al[s, r]:
                k3[:, off[r]:off[r] + seg[r]] = 1e30
                v3[:, off[r]:off[r] + seg[r]] = -1e30
        o3 = oracle.im_attention_dense(q, k3, v3, seg, vl, phase)
        assert np.array_equal(o3[:, off[s]:off[s] + seg[s]], base[:, off[s]:off[s] + seg[s]])
    # padded output rows are exactly +0
    assert np.all(base[pad] == 0.0) and not np.signbit(base[pad]).any()


# ---------------------------------------------------------------- P3: zero structure, row-stochastic
@pytest.mark.parametrize("phase", PHASES)
def test_adjacency_zero_blocks_and_row_sums(phase):
    rng = np.random.default_rng(8)
    seg, B, H, hd = (4, 5, 6), 2, 3, 2
    q, k, v = _rand_qkv(rng, B, sum(seg), H, hd)
    vl = np.array([[4, 2, 6], [1, 5, 3]], dtype=np.int32)
    out, P = oracle.im_attention_dense(q, k, v, seg, vl, phase, want_P=True)
    al = oracle.allowed_blocks(phase)
    off = _offsets(seg)
    pad = wk.padded_row_mask(seg, vl, B)
    for s in range(3):
        for r in range(3):
            blk = P[:, :, off[s]:off[s] + seg[s], off[r]:off[r] + seg[r]]
            if not al[s, r]:
                assert np.all(blk == 0.0)
            else:
                assert np.all(blk[:, :, :, :][np.broadcast_to(pad[:, None, None, off[r]:off[r] + seg[r]], blk.shape)] == 0.0)
    sums = P.sum(-1)
    for b in range(B):
        assert np.allclose(sums[b][:, ~pad[b]], 1.0, atol=1e-14)
        assert np.all(sums[b][:, pad[b]] == 0.0)


# ---------------------------------------------------------------- P4: per-vertex brute force (GAT equations)
def _gat_brute_force(q, k, v, seg, valid, allowed, scale):
    """Per vertex i: neighbourhood N_i = real vertices of the open key segment(s);
    alpha_ij = exp(e_ij) / sum_{k in N_i} exp(e_ik); out_i = sum_j alpha_ij v_j; heads concatenated."""
    B, L, H, hd = q.shape
    off = _offsets(seg)
    out = np.zeros((B, L, H * hd))
    for b in range(B):
        n = list(seg) if valid is None else [int(t) for t in valid[b]]
        for s in range(3):
            N_i = [off[r] + t for r in range(3) if allowed[s][r] for t in range(n[r])]
            for i in range(off[s], off[s] + n[s]):
                for l in range(H):
                    e = {j: scale * sum(q[b, i, l, c] * k[b, j, l, c] for c in range(hd)) for j in N_i}
                    denom = sum(math.exp(e[j]) for j in N_i)
                    for c in range(hd):
                        out[b, i, l * hd + c] = sum(math.exp(e[j]) / denom * v[b, j, l, c] for j in N_i) if N_i else 0.0
    return out


@pytest.mark.parametrize("phase", PHASES)
@pytest.mark.parametrize("seg,H,hd", [((2, 3, 1), 1, 2), ((8, 12, 10), 4, 8)])
def test_brute_force_per_vertex(phase, seg, H, hd):
    rng = np.random.default_rng(99)
    B, L = 2, sum(seg)
    q, k, v = _rand_qkv(rng, B, L, H, hd, scale=0.7)
    vl = np.stack([rng.integers(1, s + 1, size=B) for s in seg], axis=1).astype(np.int32)
    al = oracle.allowed_blocks(phase)
    for valid in (None, vl):
        ref = _gat_brute_force(q, k, v, seg, valid, al, 1.0 / math.sqrt(hd))
        got = oracle.im_attention_dense(q, k, v, seg, valid, phase)
        assert np.abs(got - ref).max() <= 1e-12
        got2 = oracle.im_attention_decomposed(q, k, v, seg, valid, phase)
        assert np.abs(got2 - ref).max() <= 1e-12


def test_explicit_scale_is_used():
    rng = np.random.default_rng(4)
    seg, H, hd = (3, 2, 4), 2, 3
    q, k, v = _rand_qkv(rng, 1, sum(seg), H, hd)
    al = oracle.allowed_blocks(oracle.PHASE_INTER_BWD)
    ref = _gat_brute_force(q, k, v, seg, None, al, 0.37)
    got = oracle.im_attention_dense(q, k, v, seg, None, oracle.PHASE_INTER_BWD, scale=0.37)
    assert np.abs(got - ref).max() <= 1e-12
