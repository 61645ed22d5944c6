"""The C-ABI library builds, loads without a GPU, and exports every function the headers under include/ declare."""
import ctypes
import re
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def _declared():
    names = set()
    for header in sorted((ROOT / "include").glob("*.h")):
        text = re.sub(r"/\*.*?\*/", "", header.read_text(), flags=re.S)
        names |= set(re.findall(r"\b(gsit_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    from paper_2505_01068_b200 import build as lib_build
    import paper_2505_01068_b200 as g

    lib_build.build()
    lib = g.load()
    names = _declared()
    assert set(g.EXPORTS) <= set(names) and len(names) >= 7
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings_and_shape_struct_layout():
    import paper_2505_01068_b200 as g

    assert g.version() >= 100
    assert g.status_string(0) == "ok" and "workspace" in g.status_string(3)
    assert ctypes.sizeof(g.binding.Shape) == 64 and g.binding.Shape.valid_len.offset == 24
    assert g.binding.Shape.row_start.offset == 48 and g.binding.Shape.packed_capacity.offset == 56
    assert ctypes.sizeof(g.binding.LayerWeights) == 12 * 8 + 8


def test_workspace_query_needs_no_gpu():
    import paper_2505_01068_b200 as g

    sh = g.make_shape(2, (8, 12, 10), 32, 4, None, g.DTYPE_F32, g.PHASE_INTRA)
    assert g.workspace_bytes(sh, g.CALL_ATTENTION) == 0
    sh16 = g.make_shape(2, (8, 12, 10), 32, 4, None, g.DTYPE_BF16, g.PHASE_INTRA)
    assert 0 < g.workspace_bytes(sh16, g.CALL_ATTENTION) <= 4096
    rows = 2 * 30
    assert g.workspace_bytes(sh, g.CALL_LAYER, 128) >= rows * (32 * 4 * 3 + 96 * 4 + 128 * 4)
    bad = g.make_shape(2, (8, 12, 10), 30, 4, None, g.DTYPE_F32, g.PHASE_INTRA)
    try:
        g.workspace_bytes(bad, g.CALL_LAYER, 128)
        raise AssertionError("expected an error")
    except g.GsitError:
        pass
