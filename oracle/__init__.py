"""TEST INFRASTRUCTURE -- ctypes access to the CPU oracle (``atrex_oracle.cpp``).

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s CPU-baseline legs may import
this package.  The product package never does, and this package never imports the product.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "atrex_oracle.cpp")
_LIB = os.path.join(_HERE, "libatrex_oracle.so")

ENTRY_DTYPE = np.dtype([("key", "<u8"), ("count", "<u8"), ("wt_lo", "<u8"), ("wt_hi", "<u8"),
                        ("phase_weight", "<f8"), ("roofline_s", "<f8")])


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-ffp-contract=off", "-std=c++17", "-fPIC", "-shared",
                               "-pthread", "-o", _LIB, _SRC])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.oracle_create.restype = C.c_void_p
        L.oracle_create.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32]
        L.oracle_destroy.argtypes = [C.c_void_p]
        L.oracle_reset.argtypes = [C.c_void_p]
        L.oracle_ingest.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.oracle_ingest_threads.restype = C.c_uint32
        L.oracle_ingest_threads.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32]
        L.oracle_ingest_filtered.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint64]
        L.oracle_ingest_slice.restype = C.c_uint32
        L.oracle_ingest_slice.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint32]
        L.oracle_slice_classes.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p]
        L.oracle_finalize_given_totals.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p]
        L.oracle_direct_totals.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p]
        L.oracle_set_work.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.oracle_n_keys.restype = C.c_uint64
        L.oracle_n_keys.argtypes = [C.c_void_p]
        L.oracle_stats.argtypes = [C.c_void_p, C.c_void_p]
        L.oracle_finalize.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p]
        L.oracle_topk.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p]
        L.oracle_score_candidate.restype = C.c_double
        L.oracle_score_candidate.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_uint32, C.c_void_p, C.c_void_p]
        L.oracle_eq3_weights.restype = C.c_uint64
        L.oracle_eq3_weights.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32, C.c_void_p,
                                         C.c_void_p, C.c_void_p]
        L.oracle_sort_by_key.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        L.oracle_rank_phase.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p,
                                        C.c_uint64, C.c_void_p]
        L.oracle_u128_to_f64.restype = C.c_double
        L.oracle_u128_to_f64.argtypes = [C.c_uint64, C.c_uint64]
        _lib = L
    return _lib


def _peaks_buf(peak_bw: float, peak_flops) -> np.ndarray:
    pf = list(peak_flops) + [1.0] * (8 - len(peak_flops))
    return np.array([peak_bw] + pf[:8], dtype=np.float64)


class Oracle:
    """Thin handle around the C++ oracle."""

    def __init__(self, app_weights, n_phases: int):
        w = np.ascontiguousarray(app_weights, dtype=np.uint32)
        self._h = lib().oracle_create(w.ctypes.data, w.shape[0], n_phases)
        if not self._h:
            raise ValueError("oracle_create rejected its arguments")

    def close(self):
        if self._h:
            lib().oracle_destroy(self._h)
            self._h = None

    __del__ = close

    def reset(self):
        lib().oracle_reset(self._h)

    def ingest(self, records: np.ndarray, threads: int = 1) -> int:
        r = np.ascontiguousarray(records)
        assert r.dtype.itemsize == 16
        if threads == 1:
            lib().oracle_ingest(self._h, r.ctypes.data, r.shape[0])
            return 1
        return lib().oracle_ingest_threads(self._h, r.ctypes.data, r.shape[0], threads)

    def ingest_filtered(self, records: np.ndarray, keys) -> None:
        r = np.ascontiguousarray(records)
        k = np.ascontiguousarray(keys, dtype=np.uint64)
        lib().oracle_ingest_filtered(self._h, r.ctypes.data, r.shape[0], k.ctypes.data, k.shape[0])

    def ingest_slice(self, records: np.ndarray, modulus: int, residue: int, threads: int = 0) -> int:
        """Aggregate only the valid records whose key's slice class (a fixed scramble of the key,
        modulo ``modulus``) equals ``residue``; returns the threads used."""
        r = np.ascontiguousarray(records)
        assert r.dtype.itemsize == 16
        return lib().oracle_ingest_slice(self._h, r.ctypes.data, r.shape[0], modulus, residue, threads)

    def finalize_given_totals(self, peak_bw: float, peak_flops, totals) -> np.ndarray:
        """Entries of this handle's keys with Eq. 3's denominators taken from ``totals`` (ints, one per phase)."""
        n = self.n_keys()
        out = np.zeros(n, dtype=ENTRY_DTYPE)
        n_out = C.c_uint64(0)
        pk = _peaks_buf(peak_bw, peak_flops)
        t = np.zeros(16, dtype=np.uint64)
        for q, v in enumerate(list(totals)[:8]):
            t[2 * q], t[2 * q + 1] = v & 0xFFFFFFFFFFFFFFFF, v >> 64
        rc = lib().oracle_finalize_given_totals(self._h, pk.ctypes.data, t.ctypes.data, out.ctypes.data, n, C.byref(n_out))
        assert rc == 0 and n_out.value == n
        return out

    def direct_totals(self, records: np.ndarray, acc: np.ndarray, valid: np.ndarray) -> None:
        """acc: uint64[16] (lo, hi per phase), valid: uint64[2]; both updated in place."""
        r = np.ascontiguousarray(records)
        assert acc.dtype == np.uint64 and acc.shape == (16,) and valid.dtype == np.uint64 and valid.shape == (2,)
        lib().oracle_direct_totals(self._h, r.ctypes.data, r.shape[0], acc.ctypes.data, valid.ctypes.data)

    def set_work(self, rows: np.ndarray) -> int:
        r = np.ascontiguousarray(rows)
        assert r.dtype.itemsize == 24
        return lib().oracle_set_work(self._h, r.ctypes.data, r.shape[0])

    def n_keys(self) -> int:
        return lib().oracle_n_keys(self._h)

    def stats(self) -> dict:
        out = np.zeros(19, dtype=np.uint64)
        lib().oracle_stats(self._h, out.ctypes.data)
        totals = [int(out[3 + 2 * p]) | (int(out[4 + 2 * p]) << 64) for p in range(8)]
        return {"n_valid": int(out[0]), "n_rejected": int(out[1]), "n_keys": int(out[2]), "totals": totals}

    def finalize(self, peak_bw: float, peak_flops) -> np.ndarray:
        n = self.n_keys()
        out = np.zeros(n, dtype=ENTRY_DTYPE)
        n_out = C.c_uint64(0)
        pk = _peaks_buf(peak_bw, peak_flops)
        rc = lib().oracle_finalize(self._h, pk.ctypes.data, out.ctypes.data, n, C.byref(n_out))
        assert rc == 0 and n_out.value == n
        return out

    def topk(self, peak_bw: float, peak_flops, phase: int, k: int) -> np.ndarray:
        out = np.zeros(max(k, 1), dtype=ENTRY_DTYPE)
        n_out = C.c_uint32(0)
        pk = _peaks_buf(peak_bw, peak_flops)
        lib().oracle_topk(self._h, pk.ctypes.data, phase, k, out.ctypes.data, C.byref(n_out))
        return out[:n_out.value].copy()


def slice_class(keys, modulus: int) -> np.ndarray:
    """Slice class of each key, as ``Oracle.ingest_slice`` assigns it."""
    k = np.ascontiguousarray(keys, dtype=np.uint64)
    out = np.zeros(k.shape[0], dtype=np.uint64)
    lib().oracle_slice_classes(k.ctypes.data, k.shape[0], modulus, out.ctypes.data)
    return out


def u128_to_f64(x: int) -> float:
    return lib().oracle_u128_to_f64((x >> 64) & 0xFFFFFFFFFFFFFFFF, x & 0xFFFFFFFFFFFFFFFF)


def score_candidates(roofline_s, unit_op, t_cand, correct, w):
    """Eq. 4-6 for a batch: t_cand, correct are [B, n_units]. Returns (S_agg[B], S_op[B, n_ops], errors[B])."""
    roofline_s = np.ascontiguousarray(roofline_s, dtype=np.float64)
    unit_op = np.ascontiguousarray(unit_op, dtype=np.uint32)
    t_cand = np.ascontiguousarray(t_cand, dtype=np.float64)
    correct = np.ascontiguousarray(correct, dtype=np.uint8)
    w = np.ascontiguousarray(w, dtype=np.float64)
    b, n = t_cand.shape
    agg = np.zeros(b, dtype=np.float64)
    s_op = np.zeros((b, w.shape[0]), dtype=np.float64)
    err = np.zeros(b, dtype=np.uint64)
    for c in range(b):
        e = C.c_uint64(0)
        agg[c] = lib().oracle_score_candidate(roofline_s.ctypes.data, unit_op.ctypes.data, n, t_cand[c].ctypes.data,
                                              correct[c].ctypes.data, w.ctypes.data, w.shape[0], s_op[c].ctypes.data,
                                              C.byref(e))
        err[c] = e.value
    return agg, s_op, err


def eq3_weights(records, app_weights, n_ops: int, n_phases: int, retained=None):
    """Literal Eq. 2-3 operator weights. Returns (w[n_ops], wtilde[n_ops], n_rejected)."""
    r = np.ascontiguousarray(records)
    aw = np.ascontiguousarray(app_weights, dtype=np.uint32)
    w = np.zeros(n_ops, dtype=np.float64)
    wt = np.zeros(n_ops, dtype=np.float64)
    ret = None if retained is None else np.ascontiguousarray(retained, dtype=np.uint8)
    rej = lib().oracle_eq3_weights(r.ctypes.data, r.shape[0], aw.ctypes.data, aw.shape[0], n_ops, n_phases,
                                   None if ret is None else ret.ctypes.data, w.ctypes.data, wt.ctypes.data)
    return w, wt, int(rej)


def sort_by_key(entries: np.ndarray) -> np.ndarray:
    """Entries ordered by packed key ascending."""
    e = np.ascontiguousarray(entries, dtype=ENTRY_DTYPE)
    out = np.zeros(e.shape[0], dtype=ENTRY_DTYPE)
    lib().oracle_sort_by_key(e.ctypes.data, e.shape[0], out.ctypes.data)
    return out


def rank_phase(entries: np.ndarray, phase: int, coverage_ppm: int, out_cap=None):
    """Ranked units of one phase, running share, coverage cut (the construction behind Table 2).
    Returns (ranked entries, cum share, dict(n_phase, n_keep, total, covered))."""
    e = np.ascontiguousarray(entries, dtype=ENTRY_DTYPE)
    cap = e.shape[0] if out_cap is None else int(out_cap)
    out = np.zeros(max(cap, 1), dtype=ENTRY_DTYPE)
    cum = np.zeros(max(cap, 1), dtype=np.float64)
    res = np.zeros(6, dtype=np.uint64)
    lib().oracle_rank_phase(e.ctypes.data, e.shape[0], phase, coverage_ppm, out.ctypes.data, cum.ctypes.data, cap,
                            res.ctypes.data)
    m = min(int(res[0]), cap)
    return out[:m].copy(), cum[:m].copy(), {
        "n_phase": int(res[0]), "n_keep": int(res[1]),
        "total": int(res[2]) | (int(res[3]) << 64), "covered": int(res[4]) | (int(res[5]) << 64)}
