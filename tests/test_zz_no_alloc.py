"""gsit_im_layer_fwd_static, the layer call for hosts that cannot allocate device memory (embedded in another
application's memory budget, inside a latency-critical loop, or after all pools were frozen).  It must give the
same result as gsit_im_layer_fwd, whose workspace the caller provides, and keep doing so when called again while
its built-in scratch still holds the previous call's intermediates.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import workloads as wk
from gpu_util import to_dev, to_np64, weights_to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def g():
    import paper_2505_01068_b200 as lib
    lib.load()
    return lib


def _case(g, dtype, B, seg, d, heads, valid, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((B, sum(seg), d), dtype=np.float32)
    w = weights_to_dev(wk.draw_layer_weights(rng, d, 4 * d, dtype, affine=True), dtype)
    vl = None if valid is None else torch.from_numpy(np.asarray(valid, dtype=np.int32)).cuda()
    return to_dev(x), w, vl


@pytest.mark.parametrize("dtype,B,seg,d,heads,valid", [
    ("f32", 2, (8, 12, 10), 32, 4, None),
    ("bf16", 2, (50, 300, 270), 64, 8, [[50, 300, 270], [25, 151, 200]]),
])
def test_static_scratch_layer_matches_workspace_layer_twice(g, dtype, B, seg, d, heads, valid):
    tol = 1e-4 if dtype == "f32" else 2e-2
    # two different inputs in a row through the shared scratch, each against the caller-workspace entry point
    for call, phase in enumerate((g.PHASE_INTER_FWD, g.PHASE_INTRA)):
        x, w, vl = _case(g, dtype, B, seg, d, heads, valid, 900 + call)
        want = g.im_layer_fwd(x, w, seg, heads, vl, phase)
        out = torch.full_like(want, float("nan"))
        got = g.im_layer_fwd_static(x, w, seg, heads, vl, phase, out=out)
        torch.cuda.synchronize()
        err = np.abs(to_np64(got) - to_np64(want))
        assert np.isfinite(to_np64(got)).all() and err.max() <= tol, (call, err.max())
    code, flags = g.last_device_status()
    assert code == 0 and flags == 0


def test_static_scratch_rejects_oversized_problem(g):
    x, w, vl = _case(g, "bf16", 8, (50, 500, 500), 64, 8, None, 5)
    sh = g.make_shape(8, (50, 500, 500), 64, 8, None, g.DTYPE_BF16, g.PHASE_INTRA)
    assert g.workspace_bytes(sh, g.CALL_LAYER, 256) > g.STATIC_SCRATCH_BYTES
    with pytest.raises(g.GsitError) as e:
        g.im_layer_fwd_static(x, w, (50, 500, 500), 8, None, g.PHASE_INTRA)
    assert e.value.code == 3
