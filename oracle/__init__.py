"""CPU oracle for GsiT Interlaced-Mask attention -- TEST INFRASTRUCTURE ONLY.

Thin ctypes/numpy access to ``gsit_oracle.c`` (plain C, fp64) plus the stack composition of
Eq. "All-Modal-In-One fusion".  Nothing here is used by, or shares code with, the CUDA path; only
tests, the smoke check and the benchmark's CPU-baseline leg may import this package.

All arrays are numpy float64, C-contiguous.  ``valid_len`` is an int32 array [B, 3] or None.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

PHASE_INTER_FWD, PHASE_INTER_BWD, PHASE_INTRA, PHASE_CUSTOM = 0, 1, 2, 3

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "gsit_oracle.c"
_LIB_PATH = _HERE / "libgsit_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (OpenMP, no fast-math).  Building the checker is not using it."""
    if force or not _LIB_PATH.exists() or _LIB_PATH.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB_PATH.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.run(["gcc", "-O2", "-std=c11", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC",
                        "-o", str(tmp), str(_SRC), "-lm"], check=True)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int32)


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB_PATH))
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_im_dense_mask.restype = None
        _lib.oracle_layernorm.restype = None
        for name in ("oracle_allowed_blocks", "oracle_im_attention_dense", "oracle_im_attention_decomposed",
                     "oracle_qkv_proj", "oracle_im_layer_fwd"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def _d(a):
    return None if a is None else a.ctypes.data_as(_D)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _seg(seg_len):
    s = (ctypes.c_int * 3)(*[int(v) for v in seg_len])
    return s


def _vl(valid_len, batch):
    if valid_len is None:
        return None, None
    a = np.ascontiguousarray(valid_len, dtype=np.int32)
    assert a.shape == (batch, 3), a.shape
    return a, a.ctypes.data_as(_I)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def allowed_blocks(phase: int, custom_mask: int = 0) -> np.ndarray:
    out = (ctypes.c_int * 9)()
    rc = _load().oracle_allowed_blocks(ctypes.c_int(phase), ctypes.c_uint32(custom_mask), out)
    if rc:
        raise ValueError("bad phase")
    return np.array(list(out), dtype=np.int32).reshape(3, 3)


def dense_mask(seg_len, valid_len_row, allowed) -> np.ndarray:
    """Dense additive mask [L, L] of one sample (0 / -inf).  ``valid_len_row`` is [3] or None."""
    L = int(sum(seg_len))
    M = np.empty((L, L), dtype=np.float64)
    al = (ctypes.c_int * 9)(*[int(v) for v in np.asarray(allowed).reshape(-1)])
    vl, vlp = _vl(None if valid_len_row is None else np.asarray(valid_len_row).reshape(1, 3), 1)
    _load().oracle_im_dense_mask(_seg(seg_len), vlp, ctypes.c_int(0), al, _d(M))
    return M


def _split_qkv_args(q, k, v):
    """q, k, v: separate [B, L, H, hd] arrays.  They are packed into one [B, L, 3, H, hd] buffer so the
    three views share a row stride, as the C entry point expects."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    assert q.shape == k.shape == v.shape and q.ndim == 4
    B, L, H, hd = q.shape
    buf = np.stack([q, k, v], axis=2)  # [B, L, 3, H, hd]
    d = H * hd
    flat = buf.reshape(-1)
    return buf, flat, B, L, H, hd, d


def im_attention_dense(q, k, v, seg_len, valid_len=None, phase=PHASE_INTER_FWD, custom_mask=0, scale=0.0,
                       want_lse=False, want_P=False, want_pairs=False):
    """Dense-mask IM attention.  Returns out [B, L, d] (and lse [B,H,L], P [B,H,L,L], pair count)."""
    buf, flat, B, L, H, hd, d = _split_qkv_args(q, k, v)
    assert L == sum(seg_len)
    out = np.empty((B, L, d), dtype=np.float64)
    lse = np.empty((B, H, L), dtype=np.float64) if want_lse else None
    P = np.empty((B, H, L, L), dtype=np.float64) if want_P else None
    pairs = ctypes.c_int64(0)
    vl, vlp = _vl(valid_len, B)
    base = flat.ctypes.data
    ptr = lambda off: ctypes.cast(base + 8 * off, _D)
    rc = _load().oracle_im_attention_dense(
        ctypes.c_int(B), _seg(seg_len), ctypes.c_int(d), ctypes.c_int(H), vlp, ctypes.c_int(phase),
        ctypes.c_uint32(custom_mask), ctypes.c_double(scale), ptr(0), ptr(d), ptr(2 * d),
        ctypes.c_int64(3 * d), _d(out), _d(lse), _d(P), ctypes.byref(pairs))
    if rc:
        raise RuntimeError(f"oracle_im_attention_dense failed ({rc})")
    res = [out]
    if want_lse:
        res.append(lse)
    if want_P:
        res.append(P)
    if want_pairs:
        res.append(int(pairs.value))
    return res[0] if len(res) == 1 else tuple(res)


def im_attention_decomposed(q, k, v, seg_len, valid_len=None, phase=PHASE_INTER_FWD, custom_mask=0, scale=0.0):
    """Block-by-block (decomposed) IM attention.  Returns out [B, L, d]."""
    buf, flat, B, L, H, hd, d = _split_qkv_args(q, k, v)
    assert L == sum(seg_len)
    out = np.empty((B, L, d), dtype=np.float64)
    vl, vlp = _vl(valid_len, B)
    base = flat.ctypes.data
    ptr = lambda off: ctypes.cast(base + 8 * off, _D)
    rc = _load().oracle_im_attention_decomposed(
        ctypes.c_int(B), _seg(seg_len), ctypes.c_int(d), ctypes.c_int(H), vlp, ctypes.c_int(phase),
        ctypes.c_uint32(custom_mask), ctypes.c_double(scale), ptr(0), ptr(d), ptr(2 * d),
        ctypes.c_int64(3 * d), _d(out))
    if rc:
        raise RuntimeError(f"oracle_im_attention_decomposed failed ({rc})")
    return out


def qkv_proj(x, w_qkv, b_qkv, seg_len, heads, valid_len=None) -> np.ndarray:
    """x [B, L, d], w_qkv [3d, d] -> qkv [B, L, 3, H, hd]."""
    x, w_qkv, b_qkv = _f64(x), _f64(w_qkv), _f64(b_qkv)
    B, L, d = x.shape
    assert L == sum(seg_len) and w_qkv.shape == (3 * d, d) and d % heads == 0
    qkv = np.empty((B, L, 3 * d), dtype=np.float64)
    vl, vlp = _vl(valid_len, B)
    rc = _load().oracle_qkv_proj(ctypes.c_int(B), _seg(seg_len), ctypes.c_int(d), vlp, _d(x), ctypes.c_int64(d),
                                 _d(w_qkv), _d(b_qkv), _d(qkv))
    if rc:
        raise RuntimeError("oracle_qkv_proj failed")
    return qkv.reshape(B, L, 3, heads, d // heads)


def layernorm(x, gamma=None, beta=None, eps=1e-5) -> np.ndarray:
    x = _f64(x)
    d = x.shape[-1]
    rows = x.size // d
    y = np.empty_like(x)
    _load().oracle_layernorm(ctypes.c_int64(rows), ctypes.c_int(d), _d(x), ctypes.c_int64(d), _d(_f64(gamma)),
                             _d(_f64(beta)), ctypes.c_double(eps), _d(y))
    return y


LAYER_KEYS = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o", "ln2_g", "ln2_b", "w_1", "b_1", "w_2", "b_2")


def im_layer_fwd(x, weights: dict, seg_len, heads, valid_len=None, phase=PHASE_INTER_FWD, custom_mask=0,
                 scale=0.0, ln_eps=1e-5) -> np.ndarray:
    """One IM encoder layer.  ``weights`` maps LAYER_KEYS to arrays (biases / LN affine may be None)."""
    x = _f64(x)
    B, L, d = x.shape
    w = {kk: _f64(weights.get(kk)) for kk in LAYER_KEYS}
    d_ff = w["w_1"].shape[0]
    assert w["w_qkv"].shape == (3 * d, d) and w["w_o"].shape == (d, d)
    assert w["w_1"].shape == (d_ff, d) and w["w_2"].shape == (d, d_ff)
    y = np.empty((B, L, d), dtype=np.float64)
    vl, vlp = _vl(valid_len, B)
    rc = _load().oracle_im_layer_fwd(
        ctypes.c_int(B), _seg(seg_len), ctypes.c_int(d), ctypes.c_int(heads), ctypes.c_int(d_ff), vlp,
        ctypes.c_int(phase), ctypes.c_uint32(custom_mask), ctypes.c_double(scale), ctypes.c_double(ln_eps),
        *[_d(w[kk]) for kk in LAYER_KEYS], _d(x), ctypes.c_int64(d), _d(y), ctypes.c_int64(d))
    if rc:
        raise RuntimeError("oracle_im_layer_fwd failed")
    return y


def gsit_stack_fwd(x, fwd_layers, bwd_layers, intra_layers, seg_len, heads, intra_heads, valid_len=None,
                   ln_eps=1e-5) -> np.ndarray:
    """Fusion encoder pair followed by the intra-enhancement encoder (Eq. "All-Modal-In-One fusion"):
    the forward-ring layers and the backward-ring layers each start from x with their own weights, their
    outputs are concatenated on the feature axis (width 2d), and the intra layers run on that."""
    a = _f64(x)
    for w in fwd_layers:
        a = im_layer_fwd(a, w, seg_len, heads, valid_len, PHASE_INTER_FWD, ln_eps=ln_eps)
    b = _f64(x)
    for w in bwd_layers:
        b = im_layer_fwd(b, w, seg_len, heads, valid_len, PHASE_INTER_BWD, ln_eps=ln_eps)
    c = np.concatenate([a, b], axis=-1)
    for w in intra_layers:
        c = im_layer_fwd(c, w, seg_len, intra_heads, valid_len, PHASE_INTRA, ln_eps=ln_eps)
    return c


def stack_head_fwd(c, w_f, b_f, seg_len, valid_len=None) -> np.ndarray:
    """Read-out of the fusion stack (Eq. "All-Modal-In-One fusion": X_m = f(|| Split(a(G_intra))[-1])): split the
    encoder output by the original modality lengths, take the last time step of each modality (with right padding inside
    a segment: its last real step; an empty segment contributes zeros), concatenate the three vectors and apply the
    linear map f.  c [B, L, dc] -> [B, out_features], w_f [out_features, 3*dc]."""
    c = _f64(c)
    w = _f64(w_f)
    B, L, dc = c.shape
    assert L == sum(seg_len) and w.shape[1] == 3 * dc
    out = np.zeros((B, w.shape[0]), dtype=np.float64)
    for b in range(B):
        z = np.zeros(3 * dc, dtype=np.float64)
        off = 0
        for s in range(3):
            n = seg_len[s] if valid_len is None else int(min(max(int(valid_len[b][s]), 0), seg_len[s]))
            if n > 0:
                z[s * dc:(s + 1) * dc] = c[b, off + n - 1]
            off += seg_len[s]
        for o in range(w.shape[0]):
            acc = 0.0 if b_f is None else float(b_f[o])
            for i in range(3 * dc):
                acc += w[o, i] * z[i]
            out[b, o] = acc
    return out
