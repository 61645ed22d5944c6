"""gsit_im_layer_fwd_static, the layer call for hosts that cannot allocate device memory (embedded in another
application's memory budget, inside a latency-critical loop, or after all pools were frozen).  It must give the
same result as gsit_im_layer_fwd, whose workspace the caller provides, and keep doing so when called again while
its built-in scratch still holds the previous call's intermediates.  Collected last on purpose."""
import gc
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


def _free_bytes():
    return torch.cuda.mem_get_info()[0]


def test_static_scratch_layer_matches_workspace_layer_bit_for_bit(g):
    """A sequence of calls of different shapes, types and block patterns through the one shared scratch array -- a large
    bf16 problem first, then smaller ones that find its leftovers under a different layout, then the first again.
    Both entry points run the same deterministic kernels on the same scratch layout, so every result must equal the
    caller-workspace call's bit for bit; and a call that is given its output buffer must leave the amount of allocated
    device memory exactly as it found it."""
    cases = [
        ("bf16", 2, (50, 300, 270), 64, 8, [[50, 300, 270], [25, 151, 200]], g.PHASE_INTER_FWD),
        ("f32", 2, (8, 12, 10), 32, 4, None, g.PHASE_INTRA),
        ("bf16", 1, (37, 150, 64), 128, 8, [[20, 150, 33]], g.PHASE_INTRA),
        ("bf16", 3, (40, 33, 20), 32, 4, [[40, 33, 20], [1, 0, 20], [17, 30, 3]], g.PHASE_INTER_BWD),
        ("bf16", 2, (50, 300, 270), 64, 8, [[50, 300, 270], [25, 151, 200]], g.PHASE_INTER_FWD),
    ]
    # The first call on a GPU is the set-up call: it asks for the array's device address, and the driver, which loads
    # kernels and device arrays lazily, maps the array with the library image at that moment (free memory drops by the
    # array's size, once).  Make it before measuring anything, as a caller would before entering its no-allocation phase.
    x, w, vl = _case(g, "f32", 1, (4, 4, 4), 32, 4, None, 1)
    g.im_layer_fwd_static(x, w, (4, 4, 4), 4, None, g.PHASE_INTRA)
    torch.cuda.synchronize()
    got = want = out = None
    for call, (dtype, B, seg, d, heads, valid, phase) in enumerate(cases):
        del got, want, out  # the previous round's tensors go now, not in the middle of the measurement below
        x, w, vl = _case(g, dtype, B, seg, d, heads, valid, 900 + call)
        want = g.im_layer_fwd(x, w, seg, heads, vl, phase)
        out = torch.full_like(want, float("nan"))
        gc.collect()  # unreachable tensors of earlier tests go now, not when the collector happens to run below
        torch.cuda.synchronize()
        held, free = torch.cuda.memory_allocated(), _free_bytes()
        got = g.im_layer_fwd_static(x, w, seg, heads, vl, phase, out=out)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == held and _free_bytes() == free, call
        assert got.data_ptr() == out.data_ptr() and torch.isfinite(got).all()
        assert torch.equal(got, want), (call, float((got - want).abs().max()))
    code, flags = g.last_device_status()
    assert code == 0 and flags == 0


def test_static_scratch_rejects_oversized_problem(g):
    x, w, vl = _case(g, "bf16", 8, (50, 500, 500), 64, 8, None, 5)
    sh = g.make_shape(8, (50, 500, 500), 64, 8, None, g.DTYPE_BF16, g.PHASE_INTRA)
    assert g.workspace_bytes(sh, g.CALL_LAYER, 256) > g.STATIC_SCRATCH_BYTES
    with pytest.raises(g.GsitError) as e:
        g.im_layer_fwd_static(x, w, (50, 500, 500), 8, None, g.PHASE_INTRA)
    assert e.value.code == 3
