"""CPU-only checks of the boundary: the library builds, loads, and exports every entry point
the header declares; struct layouts match the header; host-side argument checks that need
no device."""
import ctypes as C
import os
import re

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "atrex_agg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(atrex_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2607_14541_b200.build import build
    path = build()
    L = C.CDLL(path)
    declared = _declared_functions()
    assert len(declared) >= 12
    for name in declared:
        assert hasattr(L, name), name
    import paper_2607_14541_b200 as p
    assert sorted(p.EXPORTED_SYMBOLS) == declared


def test_struct_layouts_match_the_header():
    import paper_2607_14541_b200 as p
    assert p.RECORD_DTYPE.itemsize == 16 and p.WORK_DTYPE.itemsize == 24 and p.ENTRY_DTYPE.itemsize == 48
    assert C.sizeof(p.atrex_hw_peaks_t) == 72
    assert C.sizeof(p.atrex_agg_config_t) == 56
    assert C.sizeof(p.atrex_stats_t) == 8 * (4 + 3 * 8 + 7)
    assert p.RECORD_DTYPE.fields["shape_id"][1] == 8 and p.RECORD_DTYPE.fields["phase"][1] == 6
    assert p.WORK_DTYPE.fields["flops"][1] == 8 and p.ENTRY_DTYPE.fields["phase_weight"][1] == 32


def test_host_side_checks_without_a_device():
    import paper_2607_14541_b200 as p
    cfg = p.atrex_agg_config_t()
    assert p.atrex_agg_workspace_bytes(C.byref(cfg)) == 0            # n_apps == 0
    cfg.n_apps, cfg.n_phases, cfg.max_keys = 4, 2, 1000
    small = p.atrex_agg_workspace_bytes(C.byref(cfg))
    cfg.max_keys = 1 << 20
    big = p.atrex_agg_workspace_bytes(C.byref(cfg))
    assert 0 < small < big and big - small >= (1 << 21) * 32 - 2048 * 32
    cfg.n_phases = 9
    assert p.atrex_agg_workspace_bytes(C.byref(cfg)) == 0
    assert p.atrex_strerror(0) == b"ok" and b"keys" in p.atrex_strerror(p.ATREX_ERR_CAPACITY)
    assert p.atrex_agg_ingest(None, None, 0, None) == p.ATREX_ERR_INVALID
    assert p.atrex_agg_launch_count(None) == 0


def test_product_package_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2607_14541_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dirpath, f)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".cpp")):
            assert "paper_2607_14541_b200" not in open(os.path.join(ROOT, "oracle", f)).read()
