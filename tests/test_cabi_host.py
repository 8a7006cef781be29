"""Host-side checks of the C ABI that need no GPU: the library loads, exports what include/gswa.h
declares, validates descriptors and reports errors before anything is enqueued."""
import ctypes
import os
import re

import pytest

from paper_2409_06206_b200 import binding as gb
from paper_2409_06206_b200 import build as gbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    gbuild.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "gswa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gswa_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared()
    assert set(gb.EXPORTS) <= set(names)
    L = ctypes.CDLL(gb.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n


def test_workspace_query_and_descriptor_validation():
    d = gb.Desc(2, 16, 16, 60, 6, 8, (3, 3), (0, 4), "f32")
    saved, fwd, infer, bwd = gb.gswa_workspace_query(d)
    assert saved > 0 and infer >= saved - 1 and bwd > 0 and fwd >= 0
    bad = [
        (gb.Desc(1, 12, 16, 60, 6, 8, (3, 3), (0, 4)), -2),       # H not a multiple of M
        (gb.Desc(1, 16, 16, 60, 6, 8, (3, 2), (0, 4)), -2),       # heads do not add up
        (gb.Desc(1, 16, 16, 60, 6, 8, (3, 3), (0, 8)), -2),       # shift out of range
        (gb.Desc(1, 16, 16, 62, 6, 8, (3, 3), (0, 4)), -2),       # C not divisible by heads
        (gb.Desc(1, 16, 16, 60, 6, 8, (3, 3), (0, 4), qk_dim=65), -4),     # wider than the kernels' head-dim limit
        (gb.Desc(1, 24, 24, 128, 2, 12, (1, 1), (0, 6), "f32"), -4),        # a 12 x 12 window with head dim 64: more shared memory than a block has
        (gb.Desc(1, 16, 16, 60, 6, 8, (), ()), -2),
    ]
    # narrowed Q/K projections (Sec. "Parameter Allocation") and the paper's window 12 are accepted
    narrow = gb.Desc(2, 24, 24, 180, 6, 12, (3, 3), (0, 6), "bf16", qk_dim=16)
    wide = gb.Desc(2, 24, 24, 180, 6, 12, (3, 3), (0, 6), "bf16")
    assert gb.gswa_workspace_query(narrow)[0] < gb.gswa_workspace_query(wide)[0]
    assert gb.gswa_workspace_query(gb.Desc(1, 24, 24, 180, 6, 12, (3, 3), (0, 6), "bf16"))[3] > 0   # window 12, head dim 30
    for desc, code in bad:
        with pytest.raises(gb.GswaError) as e:
            gb.gswa_workspace_query(desc)
        assert e.value.status == code, (desc.shape, e.value.status)


def test_argument_errors_are_reported_before_any_launch():
    d = gb.Desc(1, 16, 16, 60, 6, 8, (3, 3), (0, 4), "f32")
    n0 = gb.gswa_launch_count()
    with pytest.raises(gb.GswaError) as e:
        gb.gswa_forward(d, None, 256, None, 256, None, 256, 256, 256, 256, 1 << 30, stream=0)
    assert e.value.status == -1
    with pytest.raises(gb.GswaError) as e:                       # misaligned x
        gb.gswa_forward(d, 264, 256, None, 256, None, 256, 256, 256, 256, 1 << 30, stream=0)
    assert e.value.status == -3
    with pytest.raises(gb.GswaError) as e:                       # inference scratch too small
        gb.gswa_forward(d, 256, 256, None, 256, None, 256, 256, None, 256, 16, stream=0)
    assert e.value.status == -5
    with pytest.raises(gb.GswaError) as e:                       # backward scratch too small
        gb.gswa_backward(d, 256, 256, None, 256, 256, 256, 256, 256, 256, 256, 256, 256, 256, 256, 16, stream=0)
    assert e.value.status == -5
    assert gb.gswa_launch_count() == n0
    assert gb.gswa_step_host_arena_bytes(d) > 0
    assert "NULL" in gb.gswa_status_string(-1) and gb.gswa_status_string(0) == "ok"


def test_binding_constants_match_the_header():
    text = open(os.path.join(ROOT, "include", "gswa.h")).read()
    vals = dict(re.findall(r"(GSWA_[A-Z0-9_]+)\s*=\s*(-?\d+)u?", text))
    assert int(vals["GSWA_FLAG_ACCUMULATE"]) == gb.FLAG_ACCUMULATE
    assert int(vals["GSWA_FLAG_GENERIC"]) == gb.FLAG_GENERIC
    assert int(vals["GSWA_FLAG_FUSED_FWD"]) == gb.FLAG_FUSED_FWD
    assert int(vals["GSWA_FLAG_TCGEN05_ATTN"]) == gb.FLAG_TCGEN05_ATTN
    assert int(vals["GSWA_FLAG_COPY_LOADERS"]) == gb.FLAG_COPY_LOADERS
    assert int(vals["GSWA_F32"]) == gb.GSWA_F32 and int(vals["GSWA_BF16"]) == gb.GSWA_BF16
    m = re.search(r"GSWA_STATIC_SCRATCH_BYTES \((\d+)u << (\d+)\)", text)
    assert int(m.group(1)) << int(m.group(2)) == gb.STATIC_SCRATCH_BYTES
    assert set(gb.EXPORTS) == set(_declared())
