"""The C-ABI library loads and exports every symbol include/fi.h declares; host-side argument checks that
need no device return the documented status codes."""
import ctypes
import os
import re

import pytest

from paper_2002_02645_b200 import binding as fb
from paper_2002_02645_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return fb.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fi.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fi_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 14
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in fi.h but not exported"
    assert sorted(fb.EXPORTS) == names


def test_struct_layouts_match_header():
    # field order and sizes as in fi.h (int32 / int64 / float / pointers)
    assert ctypes.sizeof(fb.fi_cache_config_t) == 48
    assert fb.fi_cache_config_t.capacity.offset == 8 and fb.fi_cache_config_t.path.offset == 44
    assert ctypes.sizeof(fb.fi_lookup_out_t) == 5 * ctypes.sizeof(ctypes.c_void_p)
    assert ctypes.sizeof(fb.fi_cascade_state_t) == 7 * 8 + 8


def test_null_arguments_are_rejected_without_a_device(lib):
    h = ctypes.c_void_p()
    assert lib.fi_cache_create(None, ctypes.byref(h)) == 1 and not h.value
    assert b"null" in lib.fi_last_error()
    cfg = fb.fi_cache_config_t(12, fb.FI_BF16, 10, 4, 5, 0, 0, 0.0, 0, 8, 0)      # dim % 8 != 0
    assert lib.fi_cache_create(ctypes.byref(cfg), ctypes.byref(h)) == 1
    assert lib.fi_cache_insert(None, None, None, None, 1, None) == 1
    assert lib.fi_cache_set_threshold(None, 0.5) == 1
    assert lib.fi_cache_lookup_batch(None, None, 0, None, 0, None, None, None) == 1
    assert lib.fi_cascade_step(None, None, 0, None, None) == 1
    assert lib.fi_cache_destroy(None) == 0
    assert lib.fi_cache_size(None) == 0
    assert lib.fi_status_string(6) == b"FI_ERR_TIMEOUT" and lib.fi_status_string(0) == b"FI_OK"
    assert lib.fi_launch_count() >= 0


def test_gemm_plan_is_balanced():
    """Host-side mirror of the tile plan: every CTA gets the same number of 16-row blocks (+-1 block per tile
    rounding), no range is empty, and ranges cover all rows."""
    def plan(count, n, ctas):
        m_tiles = -(-count // 128)
        n16 = -(-n // 16)
        best = None
        for mg in range(1, min(m_tiles, 16, ctas) + 1):
            groups = -(-m_tiles // mg)
            mg_eff = -(-m_tiles // groups)
            parts = min(ctas // mg_eff, n16)
            r16 = -(-n16 // parts)
            cost = groups * r16
            if best is None or cost < best[0] or (cost == best[0] and mg_eff > best[1]):
                best = (cost, mg_eff)
        mg = best[1]
        groups = -(-m_tiles // mg)
        parts = min(ctas // mg, n16)
        r16 = -(-n16 // parts)
        parts = -(-n16 // r16)
        return mg, groups, parts, r16
    for count, n in [(1024, 10000), (8192, 200000), (4096, 100000), (16, 50000), (819, 10000), (1, 16), (300, 5003)]:
        mg, groups, parts, r16 = plan(count, n, 148)
        assert mg * parts <= 148 and parts >= 1
        assert (parts - 1) * r16 * 16 < n <= parts * r16 * 16
        ideal = (-(-count // 128)) * (-(-n // 16)) / 148
        assert groups * r16 <= max(1.35 * ideal, ideal + groups)      # within 35 % of a perfect split
