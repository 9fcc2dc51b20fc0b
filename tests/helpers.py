"""Harness helpers: fixture loading and a Python-integer restatement used to pin the oracle.

The brute-force group-by here uses Python's arbitrary-precision integers and
``float(int)`` (correctly rounded), i.e. a different language and different arithmetic
from both the C++ oracle and the CUDA kernels.
"""
import json
import os
import struct

import numpy as np

from tracegen.layout import RECORD_DTYPE, WORK_DTYPE


def load_golden(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return json.load(f)


def f64_bits(x: float) -> int:
    return struct.unpack("<Q", struct.pack("<d", x))[0]


def records_from_dicts(rows, default_app=0, default_phase=0) -> np.ndarray:
    out = np.zeros(len(rows), dtype=RECORD_DTYPE)
    for i, r in enumerate(rows):
        out[i] = (r.get("app", default_app), r["op"], r.get("phase", default_phase), 0,
                  r["shape"], r["duration_ns"])
    return out


def work_from_dicts(rows) -> np.ndarray:
    out = np.zeros(len(rows), dtype=WORK_DTYPE)
    for i, r in enumerate(rows):
        out[i] = (r["shape"], r["op"], r.get("dtype", 0), r["flops"], r["bytes"])
    return out


def brute_force(records: np.ndarray, app_weights, n_phases: int):
    """dict group-by with Python ints. Returns (groups {key: [count, wt]}, totals, n_rejected)."""
    groups = {}
    rejected = 0
    w = [int(x) for x in app_weights]
    for a, o, p, s, d in zip(records["app_id"].tolist(), records["op_id"].tolist(),
                             records["phase"].tolist(), records["shape_id"].tolist(),
                             records["duration_ns"].tolist()):
        if a >= len(w) or p >= n_phases:
            rejected += 1
            continue
        k = (p << 48) | (o << 32) | s
        g = groups.setdefault(k, [0, 0])
        g[0] += 1
        g[1] += w[a] * d
    totals = [0] * 8
    for k, (c, wt) in groups.items():
        totals[k >> 48] += wt
    return groups, totals, rejected


def expected_entry_fields(groups, totals, work, peak_bw, peak_flops):
    """Per key: (count, wt, phase_weight bits, roofline bits) from Python arithmetic."""
    wmap = {(int(r["op_id"]) << 32) | int(r["shape_id"]): r for r in work}
    out = {}
    for k, (c, wt) in groups.items():
        t = totals[k >> 48]
        pw = 0.0 if t == 0 else float(wt) / float(t)
        r = wmap.get(k & 0xFFFFFFFFFFFF)
        if r is None:
            rb = 0x7FF8000000000000
        else:
            rb = f64_bits(max(float(int(r["flops"])) / peak_flops[int(r["dtype"])],
                              float(int(r["bytes"])) / peak_bw))
        out[k] = (c, wt, f64_bits(pw), rb)
    return out


def entry_wt(e) -> int:
    return int(e["wt_lo"]) | (int(e["wt_hi"]) << 64)


def check_entries_against(entries: np.ndarray, exp: dict):
    """entries (any order) must match the expected per-key fields bit for bit."""
    assert len(entries) == len(exp)
    seen = set()
    pw_bits = entries["phase_weight"].view(np.uint64)
    rf_bits = entries["roofline_s"].view(np.uint64)
    for i, e in enumerate(entries):
        k = int(e["key"])
        assert k in exp and k not in seen
        seen.add(k)
        c, wt, pb, rb = exp[k]
        assert int(e["count"]) == c, hex(k)
        assert entry_wt(e) == wt, hex(k)
        assert int(pw_bits[i]) == pb, hex(k)
        assert int(rf_bits[i]) == rb, hex(k)


def sorted_by_key(entries: np.ndarray) -> np.ndarray:
    return entries[np.argsort(entries["key"], kind="stable")]
