"""No-GPU checks of the boundary: the shared library loads, exports every symbol the header declares,
and rejects bad arguments on the host before any launch."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def fb():
    from paper_2609_17652_b200 import build
    build.build()
    from paper_2609_17652_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fathom.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fathom_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(fb):
    names = declared_functions()
    assert len(names) >= 12 and {"fathom_build_planes", "fathom_alloc_depth", "fathom_scan", "fathom_topk",
                                 "fathom_sparse_attend"} <= set(names)
    for name in names:
        assert hasattr(fb.lib, name), name
    assert set(fb.EXPORTS) == set(names)


def test_version_and_error_text(fb):
    assert fb.fathom_version() >= 100
    for code in range(0, -6, -1):
        assert len(fb.lib.fathom_strerror(code)) > 1
    assert b"unknown" in fb.lib.fathom_strerror(-99)


def test_layout_struct_matches_header(fb):
    assert C.sizeof(fb.Layout) == 4 * 4 + 4 * 8
    lay = fb.make_layout(8, 32, 1 << 20)
    assert lay.plane_stride_words == 16384 and lay.scale_stride == 16384 and lay.score_stride == 1 << 20
    odd = fb.make_layout(1, 1, 65)
    assert odd.plane_stride_words == 2 and odd.scale_stride == 8 and odd.score_stride == 68


def test_scratch_bytes_and_host_side_rejection(fb):
    lay = fb.make_layout(8, 32, 1 << 20)
    need = fb.fathom_scratch_bytes(lay, 4096)
    assert need >= 32 * (1 << 20) * 4                      # candidate list can hold every token
    bad = fb.make_layout(8, 32, 1 << 20); bad.d = 64
    assert fb.fathom_scratch_bytes(bad, 4096) == 0
    bad = fb.make_layout(8, 32, 1 << 20); bad.n_q_heads = 30
    assert fb.fathom_scratch_bytes(bad, 4096) == 0
    # a NULL context is refused before anything touches a device
    assert fb.lib.fathom_scan(None, C.byref(lay), 16, 16, 16, 16, 4, 16, None) == -1
    assert fb.lib.fathom_topk(None, C.byref(lay), 16, 10, 0, 0, 16, None) == -1
    assert fb.lib.fathom_build_planes(None, C.byref(lay), 16, 0, 16, 16, None) == -1
    assert fb.lib.fathom_alloc_depth(None, C.byref(lay), 16, 16, 0, 48, 4, 16, None) == -1
    assert fb.lib.fathom_sparse_attend(None, C.byref(lay), 16, 16, 16, 1, 16, 10, C.c_float(1.0), 16, None) == -1
    assert fb.lib.fathom_destroy(None) == 0
