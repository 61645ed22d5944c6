"""Seeded synthetic workloads shaped like the multimodal sentiment-analysis data the paper uses.

This module only *draws inputs* (random features, Xavier weights, valid lengths) and rounds them to
the storage type.  It contains none of the method's arithmetic and is the one module that both the
CPU oracle's tests and the GPU path's tests/benchmark read, so both sides see identical arrays.

The public datasets (CMU-MOSI, CMU-MOSEI, ...) are not available offline; these generators stand in
for them with the sequence lengths and feature widths of the paper's dataset table (Appendix
"Datasets": max lengths 50/375/500 and 50/500/500, raw feature widths 768/5/20 and 768/74/35).
Segment order is text, audio, video.  Raw features are N(0,1); each modality is brought to the common
width d_model by its own Xavier-uniform linear map (input synthesis, never timed, not a library call).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 20250501


@dataclass(frozen=True)
class Workload:
    index: int
    name: str
    dtype: str                 # "f32" or "bf16": storage type of activations and weights
    batch: int
    seg_len: tuple             # (text, audio, video)
    d_model: int
    heads: int
    raw_dims: tuple | None     # raw feature widths per modality, None = draw X ~ N(0,1) directly
    padding: str               # "none" | "uniform_half" | "quarter_half" | "stats"
    d_ff_mult: int = 4
    stack: tuple | None = None  # (n_fwd, n_bwd, n_intra, intra_heads) for the full-stack workload
    len_mean: tuple | None = None  # "stats" padding: mean and variance of the valid length per segment
    len_var: tuple | None = None

    @property
    def L(self) -> int:
        return int(sum(self.seg_len))

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index


WORKLOADS = {
    1: Workload(1, "tiny_f32", "f32", 2, (8, 12, 10), 32, 4, None, "none"),
    2: Workload(2, "aligned_msa", "bf16", 32, (50, 50, 50), 32, 4, (768, 5, 20), "none"),
    3: Workload(3, "mosi_unaligned", "bf16", 32, (50, 375, 500), 64, 8, (768, 5, 20), "uniform_half"),
    4: Workload(4, "mosei_unaligned_stack", "bf16", 64, (50, 500, 500), 64, 8, (768, 74, 35), "uniform_half",
                stack=(4, 4, 2, 8)),
    5: Workload(5, "scaled_stress", "bf16", 128, (128, 1024, 1024), 512, 8, None, "quarter_half"),
    # Second workload family: realistic sparsity and other segment-size ratios (paper, Appendix "Datasets").
    # 6: MOSEI maxima with valid lengths drawn around the train-split averages 24 / 94 / 149 (text / vision / audio;
    #    variances 148 / 5115 / 8105) -- far shorter than the maxima, so most key tiles are skipped.
    6: Workload(6, "mosei_length_stats", "bf16", 32, (50, 500, 500), 64, 8, (768, 74, 35), "stats",
                len_mean=(24.0, 149.0, 94.0), len_var=(148.0, 8105.0, 5115.0)),
    # 7: CH-SIMS-shaped maxima 39 / 400 / 55 (text / vision / audio), raw widths 768 / 709 / 33
    7: Workload(7, "chsims_shaped", "bf16", 32, (39, 55, 400), 64, 8, (768, 33, 709), "uniform_half"),
    # 8: MIntRec-shaped maxima 30 / 230 / 480 (text / vision / audio), raw widths 768 / 256 / 768
    8: Workload(8, "mintrec_shaped", "bf16", 32, (30, 480, 230), 64, 8, (768, 768, 256), "uniform_half"),
}


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    out = rounded.view(np.float32).copy()
    nan = np.isnan(a)
    if nan.any():
        out[nan] = np.nan
    return out


def storage_round(a: np.ndarray, dtype: str) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return round_to_bf16(a) if dtype == "bf16" else a


def xavier_uniform(rng: np.random.Generator, fan_out: int, fan_in: int) -> np.ndarray:
    a = np.sqrt(6.0 / (fan_in + fan_out))
    return rng.uniform(-a, a, size=(fan_out, fan_in)).astype(np.float32)


def draw_valid_len(rng: np.random.Generator, wl: Workload, batch: int | None = None) -> np.ndarray | None:
    """Per-sample valid lengths [B, 3] (int32) or None when the workload has no padding."""
    B = wl.batch if batch is None else batch
    if wl.padding == "none":
        return None
    seg = np.asarray(wl.seg_len)
    if wl.padding == "uniform_half":
        lo = (seg + 1) // 2
        return np.stack([rng.integers(lo[m], seg[m] + 1, size=B) for m in range(3)], axis=1).astype(np.int32)
    if wl.padding == "stats":
        mean, std = np.asarray(wl.len_mean), np.sqrt(np.asarray(wl.len_var))
        n = np.rint(rng.normal(mean[None, :], std[None, :], size=(B, 3)))
        return np.clip(n, 1, seg[None, :]).astype(np.int32)
    if wl.padding == "quarter_half":
        n = np.tile(seg[None, :], (B, 1))
        n[np.arange(B) % 4 == 3] = seg // 2
        return n.astype(np.int32)
    raise ValueError(wl.padding)


def draw_x(rng: np.random.Generator, wl: Workload, batch: int | None = None) -> np.ndarray:
    """Concatenated sequence X [B, L, d_model] (float32, rounded to the storage type)."""
    B = wl.batch if batch is None else batch
    if wl.raw_dims is None:
        x = rng.standard_normal((B, wl.L, wl.d_model), dtype=np.float32)
    else:
        parts = []
        for m in range(3):
            raw = rng.standard_normal((B, wl.seg_len[m], wl.raw_dims[m]), dtype=np.float32)
            p = xavier_uniform(rng, wl.d_model, wl.raw_dims[m])
            parts.append(raw @ p.T)
        x = np.concatenate(parts, axis=1)
    return storage_round(x, wl.dtype)


def padded_row_mask(wl_seg_len, valid_len: np.ndarray | None, batch: int) -> np.ndarray:
    """Boolean [B, L]: True at padded positions."""
    L = int(sum(wl_seg_len))
    mask = np.zeros((batch, L), dtype=bool)
    if valid_len is None:
        return mask
    off = 0
    for s in range(3):
        pos = np.arange(wl_seg_len[s])[None, :]
        mask[:, off:off + wl_seg_len[s]] = pos >= valid_len[:, s:s + 1]
        off += wl_seg_len[s]
    return mask


def fill_padding(a: np.ndarray, seg_len, valid_len, value) -> np.ndarray:
    """Return a copy of a [B, L, ...] with every padded row overwritten by ``value`` (e.g. NaN)."""
    out = a.copy()
    m = padded_row_mask(seg_len, valid_len, a.shape[0])
    out[m] = value
    return out


def draw_layer_weights(rng: np.random.Generator, d: int, d_ff: int, dtype: str, affine: bool = False) -> dict:
    """Xavier-uniform weights of one IM layer, no biases, LayerNorm gamma=1 / beta=0 unless ``affine``."""
    w = {
        "w_qkv": np.concatenate([xavier_uniform(rng, d, d) for _ in range(3)], axis=0),
        "w_o": xavier_uniform(rng, d, d),
        "w_1": xavier_uniform(rng, d_ff, d),
        "w_2": xavier_uniform(rng, d, d_ff),
        "b_qkv": None, "b_o": None, "b_1": None, "b_2": None,
        "ln1_g": np.ones(d, np.float32), "ln1_b": np.zeros(d, np.float32),
        "ln2_g": np.ones(d, np.float32), "ln2_b": np.zeros(d, np.float32),
    }
    if affine:
        for kk, n in (("b_qkv", 3 * d), ("b_o", d), ("b_1", d_ff), ("b_2", d)):
            w[kk] = (0.1 * rng.standard_normal(n)).astype(np.float32)
        for kk in ("ln1_g", "ln2_g"):
            w[kk] = (1.0 + 0.1 * rng.standard_normal(d)).astype(np.float32)
        for kk in ("ln1_b", "ln2_b"):
            w[kk] = (0.1 * rng.standard_normal(d)).astype(np.float32)
    for kk in ("w_qkv", "w_o", "w_1", "w_2", "b_qkv", "b_o", "b_1", "b_2"):
        if w[kk] is not None:
            w[kk] = storage_round(w[kk], dtype)
    return w


def make_inputs(index: int, batch: int | None = None, seed: int | None = None) -> dict:
    """All arrays of workload ``index``: x, valid_len, one layer's weights (and the stack's, if any).

    ``batch`` overrides the batch size (used to bound the CPU oracle's share of the work); the draws
    for the first samples are not guaranteed to equal those of the full batch.
    """
    wl = WORKLOADS[index]
    rng = np.random.default_rng(wl.seed if seed is None else seed)
    B = wl.batch if batch is None else batch
    out = {"workload": wl, "batch": B}
    out["valid_len"] = draw_valid_len(rng, wl, B)
    out["x"] = draw_x(rng, wl, B)
    d = wl.d_model
    out["layer"] = draw_layer_weights(rng, d, wl.d_ff_mult * d, wl.dtype)
    if wl.stack is not None:
        n_fwd, n_bwd, n_intra, _ = wl.stack
        out["fwd_layers"] = [draw_layer_weights(rng, d, wl.d_ff_mult * d, wl.dtype) for _ in range(n_fwd)]
        out["bwd_layers"] = [draw_layer_weights(rng, d, wl.d_ff_mult * d, wl.dtype) for _ in range(n_bwd)]
        out["intra_layers"] = [draw_layer_weights(rng, 2 * d, wl.d_ff_mult * 2 * d, wl.dtype)
                               for _ in range(n_intra)]
    return out


def draw_qkv(rng: np.random.Generator, batch: int, L: int, heads: int, head_dim: int, dtype: str):
    """Q, K, V ~ N(0,1), each [B, L, H, hd], for attention-only cases."""
    return tuple(storage_round(rng.standard_normal((batch, L, heads, head_dim), dtype=np.float32), dtype)
                 for _ in range(3))


def useful_pairs(seg_len, valid_len: np.ndarray | None, allowed: np.ndarray, batch: int) -> int:
    """Closed-form count of (query, key) pairs in open blocks over real positions, per head."""
    n = np.tile(np.asarray(seg_len)[None, :], (batch, 1)) if valid_len is None else np.asarray(valid_len)
    n = np.clip(n, 0, np.asarray(seg_len)[None, :]).astype(np.int64)
    total = 0
    for s in range(3):
        for r in range(3):
            if allowed[s][r]:
                total += int((n[:, s] * n[:, r]).sum())
    return total
