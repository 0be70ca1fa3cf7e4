"""The C-ABI library loads and exports every symbol include/damoe.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "damoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(damoe_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib_path():
    import __graft_entry__ as g
    return g.load_build_module().build()


def test_header_symbols_are_exported(lib_path):
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert "damoe_fused_moe" in names and "damoe_route_stats" in names and "damoe_load_tuning_table" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in damoe.h but not exported"


def test_binding_lists_the_same_names(lib_path):
    import paper_2607_23099_b200 as d
    assert sorted(d.EXPORTS) == _declared()


def test_variant_family_is_described(lib_path):
    import paper_2607_23099_b200 as d
    V = d.variant_count()
    assert V >= 5
    ns = d.tile_ns()
    assert min(ns) <= 16 and max(ns) == 256
    for v in range(V):
        info = d.variant_info(v)
        assert info["tile_m"] in (64, 128, 256) and info["cta_group"] in (1, 2) and info["stages"] >= 2
    with pytest.raises(d.DamoeError):
        d.variant_info(V)


def test_argument_errors_need_no_gpu(lib_path):
    import paper_2607_23099_b200 as d
    lib = d._lib
    ctx = ctypes.c_void_p()
    assert lib.damoe_create(ctypes.byref(ctx), 0, 64, 2, 8, 1000, 512, d.BF16) == 2      # H not a multiple of 128
    assert lib.damoe_create(ctypes.byref(ctx), 0, 64, 64, 8, 1024, 512, d.BF16) == 2     # k too large
    assert lib.damoe_create(ctypes.byref(ctx), 0, 0, 2, 8, 1024, 512, d.BF16) == 1       # max_T < 1
    assert lib.damoe_create(ctypes.byref(ctx), 0, 64, 2, 8, 1024, 512, 7) == 2          # unknown dtype
    assert lib.damoe_fused_moe(None, None, None, None, None, None, 1, 0, None, None) == 1
    assert lib.damoe_destroy(None) == 0


def test_table_packing_layout():
    from paper_2607_23099_b200 import tuning
    t = dict(mode=0, buckets=[dict(T=64, static_variant=2, exemplars=[[1 << 30] + [0] * 7], exemplar_variants=[1])])
    blob = tuning.pack_table(t, E=8, k=2, H=1024, I=512, dtype=0, V=5)
    assert blob[:8] == b"DAMOETB1"
    # header 8 + 9*4, bucket 16 + (4 + 32) + 8 + 0 + 0 + 4*V*8
    assert len(blob) == 8 + 36 + 16 + 36 + 8 + 160
