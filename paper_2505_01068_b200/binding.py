"""ctypes binding of libgsit.so: argument marshalling only.

Every step of the hot path runs in the CUDA kernels of the library; PyTorch is used here for device
memory (output and workspace allocation) and for the current stream.  There is no CPU fallback: if the
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

PHASE_INTER_FWD, PHASE_INTER_BWD, PHASE_INTRA, PHASE_CUSTOM = 0, 1, 2, 3
DTYPE_F32, DTYPE_BF16 = 0, 1
CALL_QKV_PROJ, CALL_ATTENTION, CALL_LAYER = 0, 1, 2
DEVFLAG_CLAMPED, DEVFLAG_TIMEOUT = 1, 2

_LIB_PATH = Path(__file__).resolve().parent / "libgsit.so"
_lib = None


class GsitError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: gsit status {code} ({status_string(code)})")
        self.code = code


class Shape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("seg_len", ctypes.c_int32 * 3), ("d_model", ctypes.c_int32),
                ("heads", ctypes.c_int32), ("valid_len", ctypes.c_void_p), ("dtype", ctypes.c_int32),
                ("phase", ctypes.c_int32), ("custom_mask", ctypes.c_uint32), ("scale", ctypes.c_float),
                ("row_start", ctypes.c_void_p), ("packed_capacity", ctypes.c_int32)]


class LayerWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("ln1_gamma", "ln1_beta", "w_qkv", "b_qkv", "w_o", "b_o", "ln2_gamma", "ln2_beta",
                 "w_1", "b_1", "w_2", "b_2")] + [("d_ff", ctypes.c_int32), ("ln_eps", ctypes.c_float)]


EXPORTS = ("gsit_im_qkv_proj", "gsit_im_attention_fwd", "gsit_im_layer_fwd", "gsit_workspace_bytes",
           "gsit_last_device_status", "gsit_status_string", "gsit_version", "gsit_trace_enable", "gsit_trace_read",
           "gsit_trace_launches", "gsit_trace_reset", "gsit_tune_attention", "gsit_test_expire_wait", "gsit_im_layer_fwd_static",
           "gsit_stack_head_fwd", "gsit_im_layer_pair_fwd",
           "gsit_plan_rows", "gsit_pack_rows", "gsit_unpack_rows")
STATIC_SCRATCH_BYTES = 4 << 20
KERNEL_ATTENTION, KERNEL_LINEAR, KERNEL_LAYERNORM = 0, 1, 2
ATTN_DEFAULT, ATTN_UNFUSED, ATTN_LEGACY, ATTN_TMEM = 0, 8, 9, 10   # gsit_kernel_choice of include/gsit_test.h


def load():
    """Loads libgsit.so (built in-tree by paper_2505_01068_b200.build); fails loudly when it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise FileNotFoundError(f"{_LIB_PATH} is missing: run `python -m paper_2505_01068_b200.build` "
                                "(there is no fallback path)")
    lib = ctypes.CDLL(str(_LIB_PATH))
    vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
    sp = ctypes.POINTER(Shape)
    lib.gsit_im_qkv_proj.argtypes = [sp, vp, i64, vp, vp, vp, vp]
    lib.gsit_im_qkv_proj.restype = ctypes.c_int
    lib.gsit_im_attention_fwd.argtypes = [sp, vp, vp, vp, i64, vp, vp, vp, sz, vp]
    lib.gsit_im_attention_fwd.restype = ctypes.c_int
    lib.gsit_im_layer_fwd.argtypes = [sp, ctypes.POINTER(LayerWeights), vp, i64, vp, i64, vp, sz, vp]
    lib.gsit_im_layer_fwd.restype = ctypes.c_int
    lib.gsit_im_layer_pair_fwd.argtypes = [sp, sp, ctypes.POINTER(LayerWeights), ctypes.POINTER(LayerWeights), vp, i64, vp, i64, vp, i64,
                                           vp, i64, vp, sz, vp]
    lib.gsit_im_layer_pair_fwd.restype = ctypes.c_int
    lib.gsit_im_layer_fwd_static.argtypes = [sp, ctypes.POINTER(LayerWeights), vp, i64, vp, i64, vp]
    lib.gsit_im_layer_fwd_static.restype = ctypes.c_int
    lib.gsit_stack_head_fwd.argtypes = [sp, vp, i64, ctypes.c_int32, vp, vp, vp, ctypes.c_int32, vp]
    lib.gsit_stack_head_fwd.restype = ctypes.c_int
    lib.gsit_plan_rows.argtypes = [sp, ctypes.c_int32, vp, vp]
    lib.gsit_plan_rows.restype = ctypes.c_int
    for fn in (lib.gsit_pack_rows, lib.gsit_unpack_rows):
        fn.argtypes = [sp, vp, i64, vp, i64, ctypes.c_int32, vp]
        fn.restype = ctypes.c_int
    lib.gsit_workspace_bytes.argtypes = [sp, ctypes.c_int, ctypes.c_int32]
    lib.gsit_workspace_bytes.restype = sz
    lib.gsit_last_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.gsit_last_device_status.restype = ctypes.c_int
    lib.gsit_status_string.argtypes = [ctypes.c_int]
    lib.gsit_status_string.restype = ctypes.c_char_p
    lib.gsit_version.restype = ctypes.c_int
    lib.gsit_trace_enable.argtypes = [ctypes.c_int]
    lib.gsit_trace_read.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)]
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().gsit_status_string(int(code)).decode()


def version() -> int:
    return int(load().gsit_version())


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.float32:
        return DTYPE_F32
    if t == torch.bfloat16:
        return DTYPE_BF16
    raise TypeError(f"unsupported dtype {t}")


def make_shape(batch, seg_len, d_model, heads, valid_len, dtype_code, phase, custom_mask=0, scale=0.0,
               row_start=None, capacity=0) -> Shape:
    """row_start (int32 device tensor of >= 3 * batch + 1 entries, from plan_rows) selects the packed row layout with
    `capacity` rows."""
    if valid_len is not None:
        assert valid_len.is_cuda and valid_len.dtype == torch.int32 and valid_len.is_contiguous()
        assert tuple(valid_len.shape) == (batch, 3)
    if row_start is not None:
        assert row_start.is_cuda and row_start.dtype == torch.int32 and row_start.is_contiguous()
        assert row_start.numel() >= 3 * batch + 1 and valid_len is not None and capacity >= 1
    return Shape(int(batch), (ctypes.c_int32 * 3)(*[int(s) for s in seg_len]), int(d_model), int(heads),
                 _ptr(valid_len), int(dtype_code), int(phase), int(custom_mask), float(scale), _ptr(row_start), int(capacity))


def _check(code: int, what: str):
    if code != 0:
        raise GsitError(code, what)


def workspace_bytes(shape: Shape, which_call: int, d_ff: int = 0) -> int:
    n = load().gsit_workspace_bytes(ctypes.byref(shape), int(which_call), int(d_ff))
    if n == ctypes.c_size_t(-1).value:
        raise GsitError(1, "gsit_workspace_bytes")
    return int(n)


def last_device_status() -> tuple[int, int]:
    """Synchronises the current stream; returns (status code, flags) and clears the device flags."""
    flags = ctypes.c_uint32(0)
    code = load().gsit_last_device_status(_stream(), ctypes.byref(flags))
    return int(code), int(flags.value)


def tune_attention(variant: int):
    """Test / measurement hook: selects a kernel family (ATTN_* above, or 1..7 for alternative mma.sync tile shapes)."""
    _check(load().gsit_tune_attention(int(variant)), "gsit_tune_attention")


def expire_wait_selftest():
    """Test hook: launches the kernel whose bounded wait must run out (see include/gsit_test.h)."""
    lib = load()
    lib.gsit_test_expire_wait.argtypes = [ctypes.c_void_p]
    _check(lib.gsit_test_expire_wait(_stream()), "gsit_test_expire_wait")


def trace_enable(on: bool):
    _check(load().gsit_trace_enable(int(bool(on))), "gsit_trace_enable")
    _check(load().gsit_trace_reset(), "gsit_trace_reset")


def trace_read(kind: int) -> tuple[float, int]:
    """(total device ms, launches) of one kernel kind since tracing was (re)enabled."""
    ms, n = ctypes.c_float(0), ctypes.c_int32(0)
    _check(load().gsit_trace_read(int(kind), ctypes.byref(ms), ctypes.byref(n)), "gsit_trace_read")
    return float(ms.value), int(n.value)


def trace_launches(kind: int, capacity: int = 8192) -> list[float]:
    """Per-launch device times (ms) of one kernel kind, in launch order."""
    buf, n = (ctypes.c_float * capacity)(), ctypes.c_int32(0)
    _check(load().gsit_trace_launches(int(kind), buf, capacity, ctypes.byref(n)), "gsit_trace_launches")
    return [float(buf[i]) for i in range(n.value)]


def im_qkv_proj(x, w_qkv, b_qkv, seg_len, heads, valid_len=None, out=None, row_start=None):
    """x [B, L, d] (last dim contiguous) -> qkv [B, L, 3, H, hd].
    With row_start (from plan_rows; bf16, d a multiple of 64) x is the packed matrix [capacity, d] and qkv
    [capacity, 3, H, hd]; valid_len gives the batch size, and only the rows of these samples are computed and written."""
    if row_start is not None:
        cap, d = x.shape
        assert x.is_cuda and x.stride(1) == 1 and w_qkv.is_contiguous() and valid_len is not None
        shape = make_shape(valid_len.shape[0], seg_len, d, heads, valid_len, _dtype_code(x.dtype), PHASE_INTRA, 0, 0.0, row_start, cap)
        if out is None:
            out = torch.zeros((cap, 3, heads, d // heads), dtype=x.dtype, device=x.device)
        _check(load().gsit_im_qkv_proj(ctypes.byref(shape), _ptr(x), x.stride(0), _ptr(w_qkv), _ptr(b_qkv), _ptr(out),
                                       _stream()), "gsit_im_qkv_proj")
        return out
    B, L, d = x.shape
    assert x.is_cuda and x.stride(2) == 1 and x.stride(0) == L * x.stride(1) and w_qkv.is_contiguous()
    shape = make_shape(B, seg_len, d, heads, valid_len, _dtype_code(x.dtype), PHASE_INTRA)
    if out is None:
        out = torch.empty((B, L, 3, heads, d // heads), dtype=x.dtype, device=x.device)
    _check(load().gsit_im_qkv_proj(ctypes.byref(shape), _ptr(x), x.stride(1), _ptr(w_qkv), _ptr(b_qkv), _ptr(out),
                                   _stream()), "gsit_im_qkv_proj")
    return out


def im_attention_fwd(q, k, v, seg_len, valid_len=None, phase=PHASE_INTER_FWD, custom_mask=0, scale=0.0,
                     want_lse=False, out=None, workspace=None):
    """q, k, v: [B, L, H, hd] views sharing strides (e.g. qkv[:, :, i] of the fused buffer).  Returns out [B, L, d]
    (and lse [B, H, L] float when want_lse).  workspace: uint8 device tensor of workspace_bytes(shape, CALL_ATTENTION)
    bytes (allocated here when not given)."""
    B, L, H, hd = q.shape
    d = H * hd
    for t in (q, k, v):
        assert t.is_cuda and t.shape == q.shape and t.stride() == q.stride() and t.dtype == q.dtype
    assert q.stride(3) == 1 and q.stride(2) == hd and q.stride(0) == L * q.stride(1)
    shape = make_shape(B, seg_len, d, H, valid_len, _dtype_code(q.dtype), phase, custom_mask, scale)
    if out is None:
        out = torch.empty((B, L, d), dtype=q.dtype, device=q.device)
    lse = torch.empty((B, H, L), dtype=torch.float32, device=q.device) if want_lse else None
    need = workspace_bytes(shape, CALL_ATTENTION)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    _check(load().gsit_im_attention_fwd(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), q.stride(1), _ptr(out),
                                        _ptr(lse), _ptr(workspace), 0 if workspace is None else workspace.numel(),
                                        _stream()), "gsit_im_attention_fwd")
    return (out, lse) if want_lse else out


def plan_rows(valid_len, seg_len, split_sample=0, out=None):
    """Packed row layout: int32 device tensor of 3 B + 1 entries, entry 3 b + s = first packed row of segment s of sample
    b, entry 3 B = rows in use.  split_sample > 0 starts that sample on a multiple of 128 rows.  Runs on the device."""
    Bn = valid_len.shape[0]
    shape = make_shape(Bn, seg_len, 16, 1, valid_len, DTYPE_F32, PHASE_INTRA)
    if out is None:
        out = torch.empty(3 * Bn + 1, dtype=torch.int32, device=valid_len.device)
    assert out.is_cuda and out.dtype == torch.int32 and out.is_contiguous() and out.numel() >= 3 * Bn + 1
    _check(load().gsit_plan_rows(ctypes.byref(shape), int(split_sample), _ptr(out), _stream()), "gsit_plan_rows")
    return out


def _move_rows(fn_name, padded, packed, seg_len, valid_len, row_start):
    Bn, L, cols = padded.shape
    for t in (padded, packed):
        assert t.is_cuda and t.dtype == torch.float32 and t.stride(-1) == 1
    assert padded.stride(0) == L * padded.stride(1) and packed.dim() == 2 and packed.shape[1] == cols
    shape = make_shape(Bn, seg_len, 16, 1, valid_len, DTYPE_F32, PHASE_INTRA, row_start=row_start, capacity=packed.shape[0])
    fn = getattr(load(), fn_name)
    if fn_name == "gsit_pack_rows":
        _check(fn(ctypes.byref(shape), _ptr(padded), padded.stride(1), _ptr(packed), packed.stride(0), cols, _stream()), fn_name)
    else:
        _check(fn(ctypes.byref(shape), _ptr(packed), packed.stride(0), _ptr(padded), padded.stride(1), cols, _stream()), fn_name)


def pack_rows(x, x_packed, seg_len, valid_len, row_start):
    """x float32 [B, L, cols] -> the real rows, in x_packed float32 [capacity, cols] at the rows the plan gives."""
    _move_rows("gsit_pack_rows", x, x_packed, seg_len, valid_len, row_start)
    return x_packed


def unpack_rows(y_packed, y, seg_len, valid_len, row_start):
    """The inverse of pack_rows; padded positions of y float32 [B, L, cols] become +0."""
    _move_rows("gsit_unpack_rows", y, y_packed, seg_len, valid_len, row_start)
    return y


_W_KEYS = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o", "ln2_g", "ln2_b", "w_1", "b_1", "w_2", "b_2")


def make_layer_weights(w: dict, ln_eps: float = 1e-5) -> LayerWeights:
    """w maps ln1_g, ln1_b, w_qkv, b_qkv, w_o, b_o, ln2_g, ln2_b, w_1, b_1, w_2, b_2 to device tensors or None."""
    for kk in ("w_qkv", "w_o", "w_1", "w_2"):
        assert w[kk].is_cuda and w[kk].is_contiguous()
    for kk in ("ln1_g", "ln1_b", "b_qkv", "b_o", "ln2_g", "ln2_b", "b_1", "b_2"):
        assert w.get(kk) is None or (w[kk].dtype == torch.float32 and w[kk].is_contiguous())
    return LayerWeights(*[_ptr(w.get(kk)) for kk in _W_KEYS], int(w["w_1"].shape[0]), float(ln_eps))


def im_layer_fwd(x, weights: dict, seg_len, heads, valid_len=None, phase=PHASE_INTER_FWD, custom_mask=0, scale=0.0,
                 ln_eps=1e-5, out=None, workspace=None, row_start=None):
    """x float32 [B, L, d] (row stride free) -> y float32 [B, L, d]; weights in bf16 or float32 select the path.
    With row_start (from plan_rows) x and out are packed matrices [capacity, d] (row stride free) and the batch size is
    that of valid_len."""
    code = _dtype_code(weights["w_qkv"].dtype)
    lw = make_layer_weights(weights, ln_eps)
    if row_start is not None:
        cap, d = x.shape
        assert x.is_cuda and x.dtype == torch.float32 and x.stride(1) == 1 and out is not None and out.shape[0] == cap
        assert out.stride(1) == 1
        shape = make_shape(valid_len.shape[0], seg_len, d, heads, valid_len, code, phase, custom_mask, scale, row_start, cap)
        need = workspace_bytes(shape, CALL_LAYER, lw.d_ff)
        if workspace is None:
            workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
        _check(load().gsit_im_layer_fwd(ctypes.byref(shape), ctypes.byref(lw), _ptr(x), x.stride(0), _ptr(out),
                                        out.stride(0), _ptr(workspace), workspace.numel(), _stream()), "gsit_im_layer_fwd")
        return out
    B, L, d = x.shape
    assert x.is_cuda and x.dtype == torch.float32 and x.stride(2) == 1 and x.stride(0) == L * x.stride(1)
    shape = make_shape(B, seg_len, d, heads, valid_len, code, phase, custom_mask, scale)
    if out is None:
        out = torch.empty((B, L, d), dtype=torch.float32, device=x.device)
    assert out.stride(2) == 1 and out.stride(0) == L * out.stride(1)
    need = workspace_bytes(shape, CALL_LAYER, lw.d_ff)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
    _check(load().gsit_im_layer_fwd(ctypes.byref(shape), ctypes.byref(lw), _ptr(x), x.stride(1), _ptr(out),
                                    out.stride(1), _ptr(workspace), workspace.numel(), _stream()), "gsit_im_layer_fwd")
    return out


def im_layer_pair_fwd(x_a, x_b, weights_a: dict, weights_b: dict, seg_len, heads, valid_len=None, phase_a=PHASE_INTER_FWD,
                      phase_b=PHASE_INTER_BWD, ln_eps=1e-5, out_a=None, out_b=None, workspace=None, row_start=None):
    """Two layers of one geometry in one call (the two ring encoders' layers of equal depth): same results as two
    im_layer_fwd calls.  x_* float32 [B, L, d] (or packed [capacity, d] with row_start), out_* likewise (required in the
    packed layout); workspace: 2 x the layer's workspace bytes."""
    code = _dtype_code(weights_a["w_qkv"].dtype)
    lwa, lwb = make_layer_weights(weights_a, ln_eps), make_layer_weights(weights_b, ln_eps)
    if row_start is not None:
        cap, d = x_a.shape
        Bn = valid_len.shape[0]
        mk = lambda ph: make_shape(Bn, seg_len, d, heads, valid_len, code, ph, 0, 0.0, row_start, cap)
        strides = lambda t: t.stride(0)
        assert out_a is not None and out_b is not None
    else:
        Bn, L, d = x_a.shape
        mk = lambda ph: make_shape(Bn, seg_len, d, heads, valid_len, code, ph)
        strides = lambda t: t.stride(1)
        if out_a is None:
            out_a = torch.empty((Bn, L, d), dtype=torch.float32, device=x_a.device)
        if out_b is None:
            out_b = torch.empty((Bn, L, d), dtype=torch.float32, device=x_a.device)
    for t in (x_a, x_b, out_a, out_b):
        assert t.is_cuda and t.dtype == torch.float32 and t.stride(-1) == 1 and t.shape == x_a.shape
    sha, shb = mk(phase_a), mk(phase_b)
    need = 2 * workspace_bytes(sha, CALL_LAYER, lwa.d_ff)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=x_a.device)
    _check(load().gsit_im_layer_pair_fwd(ctypes.byref(sha), ctypes.byref(shb), ctypes.byref(lwa), ctypes.byref(lwb), _ptr(x_a),
                                         strides(x_a), _ptr(x_b), strides(x_b), _ptr(out_a), strides(out_a), _ptr(out_b),
                                         strides(out_b), _ptr(workspace), workspace.numel(), _stream()), "gsit_im_layer_pair_fwd")
    return out_a, out_b


def im_layer_fwd_static(x, weights: dict, seg_len, heads, valid_len=None, phase=PHASE_INTER_FWD, custom_mask=0,
                        scale=0.0, ln_eps=1e-5, out=None):
    """im_layer_fwd without a workspace: the library's built-in scratch array is used, so the call allocates no
    device memory as long as ``out`` is given.  Problems whose scratch exceeds STATIC_SCRATCH_BYTES raise GsitError
    (status 3).  Calls on one GPU must not overlap in time; they share the array."""
    B, L, d = x.shape
    assert x.is_cuda and x.dtype == torch.float32 and x.stride(2) == 1 and x.stride(0) == L * x.stride(1)
    shape = make_shape(B, seg_len, d, heads, valid_len, _dtype_code(weights["w_qkv"].dtype), phase, custom_mask, scale)
    lw = make_layer_weights(weights, ln_eps)
    if out is None:
        out = torch.empty((B, L, d), dtype=torch.float32, device=x.device)
    assert out.stride(2) == 1 and out.stride(0) == L * out.stride(1)
    _check(load().gsit_im_layer_fwd_static(ctypes.byref(shape), ctypes.byref(lw), _ptr(x), x.stride(1), _ptr(out),
                                           out.stride(1), _stream()), "gsit_im_layer_fwd_static")
    return out


def stack_head_fwd(c, w_f, b_f, seg_len, valid_len=None, out=None):
    """c float32 [B, L, dc] (row stride free) -> float32 [B, out_features]: the last real step of each modality segment,
    concatenated, through the linear map w_f [out_features, 3*dc] (float32 or bfloat16) and bias b_f."""
    B, L, dc = c.shape
    assert c.is_cuda and c.dtype == torch.float32 and c.stride(2) == 1 and c.stride(0) == L * c.stride(1)
    assert w_f.is_contiguous() and w_f.shape[1] == 3 * dc
    shape = make_shape(B, seg_len, 16, 1, valid_len, _dtype_code(w_f.dtype), PHASE_INTRA)
    if out is None:
        out = torch.empty((B, w_f.shape[0]), dtype=torch.float32, device=c.device)
    _check(load().gsit_stack_head_fwd(ctypes.byref(shape), _ptr(c), c.stride(1), dc, _ptr(w_f), _ptr(b_f), _ptr(out),
                                      w_f.shape[0], _stream()), "gsit_stack_head_fwd")
    return out
