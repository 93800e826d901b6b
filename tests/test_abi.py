"""The C boundary: the library loads, exports every symbol the headers declare, and its host-only
queries and argument checks work without a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2003_03477_b200 import binding as ss
from paper_2003_03477_b200 import build as ssbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ssbuild.build()
    return ss.lib()


def _declared():
    names = set()
    for h in ("shadowsync.h", "shadowsync_harness.h", "shadowsync_profile.h"):
        src = open(os.path.join(ROOT, "include", h)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names |= set(re.findall(r"\b(ssh?_[a-z0-9_]+)\s*\(", src))
    return names


def test_every_declared_symbol_is_exported(lib):
    declared = _declared()
    assert declared == set(ss.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert ss.ss_status_str(0) == "ok"
    assert "NULL" in ss.ss_status_str(-1) and "unknown" in ss.ss_status_str(-99)


def test_param_layout_matches_the_documented_rule(lib):
    spec = ss.MlpSpec((13, 64, 16), (144, 64, 1), False)
    # every tensor starts on a multiple of 32 floats, weight then bias, layers in order
    assert spec.w_off == [0, 896, 1952, 11232]
    assert spec.b_off == [832, 1920, 11168, 11296]
    assert spec.param_count == 11328
    unpadded = sum(i * o + o for i, o in spec.layer_dims)
    assert unpadded == 11281
    med = ss.MlpSpec((13, 512, 256, 64), (1728, 512, 256, 1), True)
    assert sum(i * o + o for i, o in med.layer_dims) == 1171777
    assert all(o % 32 == 0 for o in med.w_off + med.b_off)
    assert ss.ss_mlp_workspace_bytes(med, 2048) > 0
    assert ss.ss_embbag_bwd_workspace_bytes(26, 1_000_000, 64, 2048, 559_104) > 5 * 4 * 559_104


def test_bad_descriptors_are_rejected_on_the_host(lib):
    with pytest.raises(ss.SsError):
        ss.MlpSpec((13, 64, 16), (144, 64, 2), False)      # last layer must give one logit
    with pytest.raises(ss.SsError):
        ss.MlpSpec((13, 63, 16), (144, 64, 1), False)      # hidden width not a multiple of 8


def test_null_and_range_checks_need_no_gpu(lib):
    vp = C.c_void_p
    arr = (vp * 2)(0x1000, 0x2000)
    assert lib.ss_sync_easgd(None, 2, 0x1000, 16, 0.1, 0, None, None) == -1
    assert lib.ss_sync_easgd(arr, 2, None, 16, 0.1, 0, None, None) == -1
    assert lib.ss_sync_easgd(arr, 17, 0x1000, 16, 0.1, 0, None, None) == -2
    assert lib.ss_sync_easgd(arr, 2, 0x1000, 16, 1.5, 0, None, None) == -8
    bad = (vp * 2)(0x1004, 0x2000)
    assert lib.ss_sync_ma(bad, 2, None, 16, 0.1, 0, None, None) == -3
    assert lib.ss_embbag_fwd(0x1000, 2, 10, 6, 0x1000, 0x1000, 4, 0x1000, 16, None, 0, 0, None, None) == -2  # D % 4
    assert lib.ss_embbag_fwd(None, 2, 10, 8, 0x1000, 0x1000, 4, 0x1000, 16, None, 0, 0, None, None) == -1


def test_binding_constants_match_the_header():
    import os
    import re
    hdr = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "shadowsync.h")).read()
    m = re.search(r"#define\s+SS_TABLE_SORT_CAP\s+(\d+)", hdr)
    assert m and int(m.group(1)) == ss.SS_TABLE_SORT_CAP
