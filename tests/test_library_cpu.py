"""Host-side checks of the CUDA library that need no GPU: it loads, exports every symbol the
header declares, and its host-only queries follow the documented layout arithmetic."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hb():
    from paper_1804_01526_b200 import build
    build.build()
    from paper_1804_01526_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(hb):
    header = open(os.path.join(ROOT, "include", "hbfp.h")).read()
    declared = set(re.findall(r"HBFP_API\s+[\w\s\*]+?\b(hbfp_\w+)\s*\(", header))
    assert declared, "no declarations found"
    L = ctypes.CDLL(hb.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name
    assert declared == set(hb.EXPORTS)


def test_struct_sizes_match_header(hb):
    assert ctypes.sizeof(hb._CFormat) == 40
    assert ctypes.sizeof(hb._COperand) == 80


def test_status_strings(hb):
    assert hb.status_string(0) == "ok"
    assert len({hb.status_string(i) for i in range(9)}) == 9


@pytest.mark.parametrize("rows,k,m,b,exp", [
    (256, 256, 8, 32, dict(bp=32, nkb=8, kst=256, planes=1, rs=256)),
    (100, 784, 8, 24, dict(bp=32, nkb=33, kst=1152, planes=1, rs=112)),
    (10, 1024, 12, 64, dict(bp=64, nkb=16, kst=1024, planes=2, rs=16)),
    (7, 300, 8, 0, dict(b=300, bp=384, nkb=1, kst=384)),
    (7, 300, 8, 100, dict(bp=128, nkb=3, kst=384)),
    (3, 70, 8, 32, dict(nkb=3, kst=128)),
])
def test_packed_layout(hb, rows, k, m, b, exp):
    lay = hb.packed_layout(rows, k, hb.Format(m, b))
    for key, val in exp.items():
        assert lay[key] == val, (key, lay)
    assert lay["plane_stride"] % 1024 == 0 and lay["plane_stride"] >= rows * lay["kst"]
    assert lay["mant_bytes"] == lay["planes"] * lay["plane_stride"]
    assert lay["exp_bytes"] % 128 == 0 and lay["exp_bytes"] >= lay["nkb"] * lay["rs"]
    assert hb.packed_sizes(rows, k, hb.Format(m, b)) == (lay["mant_bytes"], lay["exp_bytes"])


def test_bad_formats_are_rejected(hb):
    for f in (hb.Format(1, 32), hb.Format(13, 32), hb.Format(8, -1), hb.Format(8, 32, tile=16),
              hb.Format(8, 32, rounding=2), hb.Format(8, 32, exp_mode=3)):
        with pytest.raises(hb.HbfpError):
            hb.packed_layout(4, 64, f)
    with pytest.raises(hb.HbfpError):          # 2047^2 * 1024 does not fit int32
        hb.packed_layout(4, 4096, hb.Format(12, 1024))
    hb.packed_layout(4, 4096, hb.Format(12, 512))
    with pytest.raises(hb.HbfpError):
        hb.packed_layout(-1, 4, hb.Format())


def test_workspace_query_is_host_only_and_monotone(hb):
    f = hb.Format(8, 64)
    w1 = hb.gemm_workspace(0, 0, 128, 128, 256, f, f)
    w2 = hb.gemm_workspace(0, 0, 256, 128, 256, f, f)
    assert 0 < w1 <= w2
    with pytest.raises(hb.HbfpError):           # blocks of the operands must coincide
        hb.gemm_workspace(0, 0, 128, 128, 256, hb.Format(8, 32), hb.Format(8, 64))
