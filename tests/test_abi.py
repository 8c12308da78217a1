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


def test_spans_partition_every_tile_exactly_once():
    """Spans mode of the distance GEMM, from the library's own plan code (host only): for every query tile the pieces
    of all CTAs cover each (cache-row tile, k-block) pair exactly once, a CTA has at most three pieces, slots are
    distinct, and the half-full last query tile takes one 128-row MMA."""
    from paper_2002_02645_b200 import binding as fb
    cases = [  # count, entries, dim, max_batch
        (190, 10000, 8192, 1024), (482, 10000, 16384, 1024), (100, 10000, 8192, 1024), (300, 3000, 4096, 600),
        (270, 1500, 4096, 600), (200, 300, 4096, 200), (129, 16, 4096, 129), (600, 1500, 4096, 600), (35, 700, 65536, 1024)]
    seen_modes = set()
    for count, n, dim, max_batch in cases:
        plan, _ = fb.gemm_plan_describe(count, n, 148, 5, dim, max_batch)
        seen_modes.add(plan["mode"])
        if plan["mode"] != 3:
            continue
        num_kb = (dim + 63) // 64
        covered = {}
        slots = set()
        for cta in range(148):
            _, items = fb.gemm_plan_describe(count, n, 148, 5, dim, max_batch, cta)
            assert len(items) <= 3
            for m, tile, kb0, kb1, rows128, slot in items:
                assert 0 <= kb0 < kb1 <= num_kb and 0 <= tile < plan["n_tiles"] and 0 <= m < plan["m_tiles"]
                assert rows128 == (1 if plan["half"] and m == plan["m_tiles"] - 1 else 2)
                assert slot not in slots and slot // 3 == cta
                slots.add(slot)
                for kb in range(kb0, kb1):
                    assert (m, tile, kb) not in covered
                    covered[(m, tile, kb)] = cta
        assert len(covered) == plan["m_tiles"] * plan["n_tiles"] * num_kb
        # the pieces of one tile come from consecutive CTAs, in k order
        for m in range(plan["m_tiles"]):
            for tile in range(plan["n_tiles"]):
                owners = [covered[(m, tile, kb)] for kb in range(num_kb)]
                assert owners == sorted(owners) and set(owners) == set(range(owners[0], owners[-1] + 1))
        assert plan["lists"] == plan["n_tiles"] and plan["half"] == (1 if count - (plan["m_tiles"] - 1) * 256 <= 128 else 0)
    assert 3 in seen_modes


def test_plan_modes_of_the_bench_workloads():
    from paper_2002_02645_b200 import binding as fb
    mode = lambda count, n, dim, mb, k=5: fb.gemm_plan_describe(count, n, 148, k, dim, mb)[0]["mode"]
    assert mode(1024, 10000, 65536, 1024) == 1      # one full tile per CTA and a tail cut along the rows
    assert mode(803, 10000, 32768, 1024) == 1
    assert mode(482, 10000, 16384, 1024) == 3       # fewer tiles than CTAs: spans
    assert mode(190, 10000, 8192, 1024) == 3
    assert mode(8192, 200000, 8192, 8192, 10) == 0  # many tiles per CTA: ranges
    assert mode(4096, 100000, 256, 4096) == 0
    p, _ = fb.gemm_plan_describe(8192, 200000, 148, 10, 8192, 8192)
    assert p["mg"] * 256 * 8192 * 2 <= 48 << 20     # a group's query tiles stay under 48 MB over a cache beyond L2
    assert fb.load_library().fi_gemm_plan_describe(0, 10, 148, 5, 64, 16, -1, None, None, None) == 1
