"""ctypes binding of the C ABI declared in ``include/atrex_agg.h``.

Argument marshalling only: every step of the aggregation path runs in the library's CUDA
kernels.  PyTorch appears here for device memory (workspace, output buffers) and streams.
There is no CPU fallback: if the shared library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# ATREX_AGG_LIBRARY selects another build of the same library (e.g. the bounds-checked one)
LIB_PATH = os.environ.get("ATREX_AGG_LIBRARY") or os.path.join(_HERE, "libatrex_agg.so")

ATREX_MAX_PHASES = 8
ATREX_MAX_DTYPES = 8
ATREX_MAX_TOPK = 65536
ATREX_FLAG_NO_HOT_DIRECTORY = 1

ATREX_OK = 0
ATREX_ERR_INVALID = -1
ATREX_ERR_CAPACITY = -2
ATREX_ERR_OUT_TOO_SMALL = -3
ATREX_ERR_CUDA = -4
ATREX_ERR_TIMEOUT = -5
ATREX_ERR_STATE = -6
ATREX_ERR_NOMEM = -7
ATREX_ERR_TOO_LARGE = -8
ATREX_ERR_BOUNDS = -9
ATREX_RELEASE_MAX_ENTRIES = 1 << 28
ATREX_STATIC_TOPK_MAX_ENTRIES = 65536
ATREX_MAX_WORLD = 1024

RECORD_DTYPE = np.dtype([("app_id", "<u4"), ("op_id", "<u2"), ("phase", "u1"), ("pad", "u1"),
                         ("shape_id", "<u4"), ("duration_ns", "<u4")])
WORK_DTYPE = np.dtype([("shape_id", "<u4"), ("op_id", "<u2"), ("dtype", "<u2"), ("flops", "<u8"), ("bytes", "<u8")])
ENTRY_DTYPE = np.dtype([("key", "<u8"), ("count", "<u8"), ("wt_lo", "<u8"), ("wt_hi", "<u8"),
                        ("phase_weight", "<f8"), ("roofline_s", "<f8")])

EXPORTED_SYMBOLS = [
    "atrex_agg_workspace_bytes", "atrex_agg_create", "atrex_agg_set_work_table", "atrex_agg_ingest",
    "atrex_agg_ingest_host", "atrex_agg_merge", "atrex_agg_finalize", "atrex_agg_topk", "atrex_agg_stats",
    "atrex_agg_reset", "atrex_agg_destroy", "atrex_strerror", "atrex_agg_last_cuda_error",
    "atrex_agg_launch_count", "atrex_topk_entries_static", "atrex_agg_hot_directory",
    "atrex_agg_finalize_with_totals", "atrex_score_aggregate", "atrex_eq3_create", "atrex_eq3_ingest",
    "atrex_eq3_finalize", "atrex_eq3_reset", "atrex_eq3_destroy", "atrex_release_scratch_bytes",
    "atrex_entries_sort_by_key", "atrex_entries_rank", "atrex_agg_totals", "atrex_key_owner", "atrex_keys_owner",
    "atrex_entries_bucket_by_owner", "atrex_totals_combine", "atrex_build_has_bounds_checks",
]


class atrex_agg_config_t(C.Structure):
    _fields_ = [("n_apps", C.c_uint32), ("n_phases", C.c_uint32), ("max_keys", C.c_uint64),
                ("max_work_rows", C.c_uint64), ("app_weights", C.c_void_p), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_uint64), ("device", C.c_int32), ("flags", C.c_uint32)]


class atrex_hw_peaks_t(C.Structure):
    _fields_ = [("peak_bw", C.c_double), ("peak_flops", C.c_double * ATREX_MAX_DTYPES)]


class atrex_rank_result_t(C.Structure):
    _fields_ = [("n_phase", C.c_uint64), ("n_keep", C.c_uint64), ("total_lo", C.c_uint64), ("total_hi", C.c_uint64),
                ("covered_lo", C.c_uint64), ("covered_hi", C.c_uint64)]


class atrex_stats_t(C.Structure):
    _fields_ = [("n_valid", C.c_uint64), ("n_rejected", C.c_uint64), ("n_dropped", C.c_uint64),
                ("n_keys", C.c_uint64), ("total_lo", C.c_uint64 * ATREX_MAX_PHASES),
                ("total_hi", C.c_uint64 * ATREX_MAX_PHASES), ("keys_per_phase", C.c_uint64 * ATREX_MAX_PHASES),
                ("table_slots", C.c_uint64), ("hot_slots", C.c_uint64), ("n_spilled", C.c_uint64),
                ("n_overflow", C.c_uint64), ("max_spill_fill", C.c_uint64), ("spill_cap", C.c_uint64),
                ("n_drains", C.c_uint64)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is not built; run `python -m paper_2607_14541_b200.build` "
                          "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, u64, u32 = C.c_void_p, C.c_uint64, C.c_uint32
    L.atrex_agg_workspace_bytes.restype = u64
    L.atrex_agg_workspace_bytes.argtypes = [C.POINTER(atrex_agg_config_t)]
    L.atrex_agg_create.argtypes = [C.POINTER(atrex_agg_config_t), C.POINTER(vp)]
    L.atrex_agg_set_work_table.argtypes = [vp, vp, u64, vp]
    L.atrex_agg_ingest.argtypes = [vp, vp, u64, vp]
    L.atrex_agg_ingest_host.argtypes = [vp, vp, u64, vp]
    L.atrex_agg_merge.argtypes = [vp, vp, u64, vp]
    L.atrex_agg_finalize.argtypes = [vp, C.POINTER(atrex_hw_peaks_t), vp, u64, C.POINTER(u64), vp]
    L.atrex_agg_finalize_with_totals.argtypes = [vp, C.POINTER(atrex_hw_peaks_t), vp, vp, vp, u64, C.POINTER(u64), vp]
    L.atrex_agg_topk.argtypes = [vp, u32, u32, vp, C.POINTER(u32), vp]
    L.atrex_agg_stats.argtypes = [vp, C.POINTER(atrex_stats_t), vp]
    L.atrex_agg_reset.argtypes = [vp, vp]
    L.atrex_agg_hot_directory.argtypes = [vp, vp, u32, C.POINTER(u32), vp]
    L.atrex_agg_destroy.argtypes = [vp]
    L.atrex_agg_destroy.restype = None
    L.atrex_strerror.restype = C.c_char_p
    L.atrex_strerror.argtypes = [C.c_int]
    L.atrex_agg_last_cuda_error.argtypes = [vp]
    L.atrex_agg_launch_count.restype = u64
    L.atrex_agg_launch_count.argtypes = [vp]
    L.atrex_eq3_create.argtypes = [u32, u32, u32, vp, C.c_int32, C.POINTER(vp)]
    L.atrex_eq3_ingest.argtypes = [vp, vp, u64, vp]
    L.atrex_eq3_finalize.argtypes = [vp, vp, vp, vp, C.POINTER(u64), vp]
    L.atrex_eq3_reset.argtypes = [vp, vp]
    L.atrex_eq3_destroy.argtypes = [vp]
    L.atrex_eq3_destroy.restype = None
    L.atrex_score_aggregate.argtypes = [vp, vp, u64, vp, vp, u64, vp, u32, vp, vp, vp, vp]
    L.atrex_topk_entries_static.argtypes = [vp, u64, u32, u32, vp, C.POINTER(u32), vp]
    L.atrex_release_scratch_bytes.restype = u64
    L.atrex_release_scratch_bytes.argtypes = [u64]
    L.atrex_entries_sort_by_key.argtypes = [vp, u64, vp, vp, u64, vp]
    L.atrex_entries_rank.argtypes = [vp, u64, u32, u32, vp, vp, u64, C.POINTER(atrex_rank_result_t), vp, u64, vp]
    L.atrex_build_has_bounds_checks.argtypes = []
    L.atrex_agg_totals.argtypes = [vp, vp, vp]
    L.atrex_key_owner.restype = u32
    L.atrex_key_owner.argtypes = [u64, u32]
    L.atrex_keys_owner.restype = None
    L.atrex_keys_owner.argtypes = [vp, u64, u32, vp]
    L.atrex_entries_bucket_by_owner.argtypes = [vp, u64, u32, vp, vp, vp, vp]
    L.atrex_totals_combine.argtypes = [vp, vp, u32, vp, vp]
    return L


lib = _load()

# the C entry points under their own names
atrex_agg_workspace_bytes = lib.atrex_agg_workspace_bytes
atrex_agg_create = lib.atrex_agg_create
atrex_agg_set_work_table = lib.atrex_agg_set_work_table
atrex_agg_ingest = lib.atrex_agg_ingest
atrex_agg_ingest_host = lib.atrex_agg_ingest_host
atrex_agg_merge = lib.atrex_agg_merge
atrex_agg_finalize = lib.atrex_agg_finalize
atrex_agg_topk = lib.atrex_agg_topk
atrex_agg_finalize_with_totals = lib.atrex_agg_finalize_with_totals
atrex_agg_stats = lib.atrex_agg_stats
atrex_agg_reset = lib.atrex_agg_reset
atrex_agg_hot_directory = lib.atrex_agg_hot_directory
atrex_agg_destroy = lib.atrex_agg_destroy
atrex_strerror = lib.atrex_strerror
atrex_agg_last_cuda_error = lib.atrex_agg_last_cuda_error
atrex_agg_launch_count = lib.atrex_agg_launch_count
atrex_topk_entries_static = lib.atrex_topk_entries_static
atrex_score_aggregate = lib.atrex_score_aggregate
atrex_eq3_create = lib.atrex_eq3_create
atrex_eq3_ingest = lib.atrex_eq3_ingest
atrex_eq3_finalize = lib.atrex_eq3_finalize
atrex_eq3_reset = lib.atrex_eq3_reset
atrex_eq3_destroy = lib.atrex_eq3_destroy
atrex_release_scratch_bytes = lib.atrex_release_scratch_bytes
atrex_entries_sort_by_key = lib.atrex_entries_sort_by_key
atrex_entries_rank = lib.atrex_entries_rank
atrex_agg_totals = lib.atrex_agg_totals
atrex_build_has_bounds_checks = lib.atrex_build_has_bounds_checks
atrex_key_owner = lib.atrex_key_owner
atrex_keys_owner = lib.atrex_keys_owner
atrex_entries_bucket_by_owner = lib.atrex_entries_bucket_by_owner
atrex_totals_combine = lib.atrex_totals_combine


class AtrexError(RuntimeError):
    def __init__(self, status: int, where: str, cuda_error: int = 0):
        self.status = status
        msg = f"{where}: {atrex_strerror(status).decode()} ({status})"
        if cuda_error:
            msg += f" [cudaError {cuda_error}]"
        super().__init__(msg)


def make_peaks(peak_bw: float, peak_flops) -> atrex_hw_peaks_t:
    pk = atrex_hw_peaks_t()
    pk.peak_bw = float(peak_bw)
    pf = list(peak_flops) + [1.0] * (ATREX_MAX_DTYPES - len(peak_flops))
    for i in range(ATREX_MAX_DTYPES):
        pk.peak_flops[i] = float(pf[i])
    return pk


class OperatorWeights:
    """Operator importance weights per Eq. 2-3 as written (per-application denominators)."""

    def __init__(self, app_weights, n_ops: int, n_phases: int, device: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the aggregation path is CUDA-only and no CUDA device is available")
        self._torch, self.device, self.n_ops = torch, int(device), int(n_ops)
        w = np.ascontiguousarray(app_weights, dtype=np.uint32)
        h = C.c_void_p()
        rc = atrex_eq3_create(int(w.shape[0]), int(n_ops), int(n_phases), w.ctypes.data, self.device, C.byref(h))
        if rc != ATREX_OK:
            raise AtrexError(rc, "atrex_eq3_create")
        self._h = h

    def _stream(self, stream=None):
        return self._torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream.cuda_stream

    def ingest(self, records, n: int | None = None, stream=None):
        if n is None:
            n = records.numel() * records.element_size() // 16
        rc = atrex_eq3_ingest(self._h, records.data_ptr(), int(n), self._stream(stream))
        if rc != ATREX_OK:
            raise AtrexError(rc, "atrex_eq3_ingest")

    def finalize(self, retained=None, stream=None):
        """Returns (w, wtilde, n_rejected)."""
        w, wt = np.zeros(self.n_ops), np.zeros(self.n_ops)
        rej = C.c_uint64(0)
        ret = None if retained is None else np.ascontiguousarray(retained, dtype=np.uint8)
        rc = atrex_eq3_finalize(self._h, None if ret is None else ret.ctypes.data, w.ctypes.data, wt.ctypes.data,
                                C.byref(rej), self._stream(stream))
        if rc != ATREX_OK:
            raise AtrexError(rc, "atrex_eq3_finalize")
        return w, wt, int(rej.value)

    def reset(self, stream=None):
        atrex_eq3_reset(self._h, self._stream(stream))

    def close(self):
        if getattr(self, "_h", None):
            atrex_eq3_destroy(self._h)
            self._h = None

    __del__ = close


def score_aggregate(roofline_s, unit_op, t_cand, correct, w, stream=None):
    """Eq. 4-6 on the GPU.  CUDA tensors: roofline_s f64[n], unit_op int32[n], t_cand f64[B, n],
    correct uint8[B, n], w f64[n_ops].  Returns (S_agg f64[B], S_op f64[B, n_ops], errors int64[B])."""
    import torch
    b, n = t_cand.shape
    n_ops = w.numel()
    dev = t_cand.device
    s_agg = torch.empty(b, dtype=torch.float64, device=dev)
    s_op = torch.empty(b, n_ops, dtype=torch.float64, device=dev)
    err = torch.empty(b, dtype=torch.int64, device=dev)
    s = torch.cuda.current_stream(dev).cuda_stream if stream is None else stream.cuda_stream
    rc = atrex_score_aggregate(roofline_s.data_ptr(), unit_op.data_ptr(), n, t_cand.data_ptr(), correct.data_ptr(), b,
                               w.data_ptr(), n_ops, s_agg.data_ptr(), s_op.data_ptr(), err.data_ptr(), s)
    if rc != ATREX_OK:
        raise AtrexError(rc, "atrex_score_aggregate")
    return s_agg, s_op, err


def topk_entries_static(entries, n: int, phase: int, k: int, out, stream=None) -> int:
    """Rank ``n`` entries held in the CUDA tensor ``entries`` without any device allocation.

    For callers that cannot allocate on the device: the selection buffer is a fixed array inside
    the library, so ``n`` and ``k`` may be at most ATREX_STATIC_TOPK_MAX_ENTRIES.  ``out`` is a
    caller-provided CUDA tensor with room for ``k`` 48-byte entries; returns how many were written.
    """
    n_out = C.c_uint32(0)
    s = None if stream is None else (stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))
    rc = atrex_topk_entries_static(entries.data_ptr() if n else None, int(n), int(phase), int(k),
                                   out.data_ptr() if k else None, C.byref(n_out), s)
    if rc != ATREX_OK:
        raise AtrexError(rc, "atrex_topk_entries_static")
    return int(n_out.value)


def _stream_ptr(stream):
    return None if stream is None else (stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _release_scratch(entries, n: int):
    import torch
    nbytes = atrex_release_scratch_bytes(int(n))
    if nbytes == 0:
        raise AtrexError(ATREX_ERR_TOO_LARGE, "atrex_release_scratch_bytes")
    buf = torch.empty(nbytes + 256, dtype=torch.uint8, device=entries.device)
    return buf, (buf.data_ptr() + 255) // 256 * 256, nbytes


def sort_entries_by_key(entries, n: int, stream=None):
    """The ``n`` entries of the CUDA byte tensor ``entries`` in packed-key order (a new CUDA tensor)."""
    import torch
    out = torch.empty(max(int(n), 1) * 48, dtype=torch.uint8, device=entries.device)
    if n:
        buf, base, nbytes = _release_scratch(entries, n)
        rc = atrex_entries_sort_by_key(entries.data_ptr(), int(n), out.data_ptr(), base, nbytes, _stream_ptr(stream))
        if rc != ATREX_OK:
            raise AtrexError(rc, "atrex_entries_sort_by_key")
    return out[: int(n) * 48]


def rank_entries(entries, n: int, phase: int, coverage_ppm: int = 0, out_cap=None, stream=None):
    """Ranked entries of one phase with their running share and the coverage cut.

    Returns (ranked CUDA byte tensor, cum-share CUDA float64 tensor, dict with n_phase, n_keep,
    total, covered); the two tensors hold min(n_phase, out_cap) rows."""
    import torch
    cap = int(n) if out_cap is None else int(out_cap)
    ranked = torch.empty(max(cap, 1) * 48, dtype=torch.uint8, device=entries.device)
    cum = torch.empty(max(cap, 1), dtype=torch.float64, device=entries.device)
    res = atrex_rank_result_t()
    if n:
        buf, base, nbytes = _release_scratch(entries, n)
        rc = atrex_entries_rank(entries.data_ptr(), int(n), int(phase), int(coverage_ppm),
                                ranked.data_ptr() if cap else None, cum.data_ptr() if cap else None, cap,
                                C.byref(res), base, nbytes, _stream_ptr(stream))
        if rc != ATREX_OK:
            raise AtrexError(rc, "atrex_entries_rank")
    m = min(int(res.n_phase), cap)
    return ranked[: m * 48], cum[:m], {
        "n_phase": int(res.n_phase), "n_keep": int(res.n_keep),
        "total": int(res.total_lo) | (int(res.total_hi) << 64),
        "covered": int(res.covered_lo) | (int(res.covered_hi) << 64)}


def bucket_entries_by_owner(entries, n: int, world: int, stream=None):
    """Group the ``n`` entries of the CUDA byte tensor ``entries`` by owner rank (``atrex_entries_bucket_by_owner``).
    Returns (grouped CUDA byte tensor, list of per-rank entry counts)."""
    import torch
    out = torch.empty(max(int(n), 1) * 48, dtype=torch.uint8, device=entries.device)
    scratch = torch.empty(2 * int(world), dtype=torch.int64, device=entries.device)
    counts = np.zeros(int(world), dtype=np.uint64)
    rc = atrex_entries_bucket_by_owner(entries.data_ptr() if n else None, int(n), int(world), out.data_ptr(),
                                       scratch.data_ptr(), counts.ctypes.data, _stream_ptr(stream))
    if rc != ATREX_OK:
        raise AtrexError(rc, "atrex_entries_bucket_by_owner")
    return out[: int(n) * 48], [int(c) for c in counts]


def combine_totals(lo_rows: np.ndarray, hi_rows: np.ndarray):
    """Exact per-phase sums of the shards' totals (``atrex_totals_combine``); rows are [n_ranks, 8] uint64.
    Returns (lo[8], hi[8]) as uint64 arrays."""
    lo = np.ascontiguousarray(lo_rows, dtype=np.uint64).reshape(-1, ATREX_MAX_PHASES)
    hi = np.ascontiguousarray(hi_rows, dtype=np.uint64).reshape(-1, ATREX_MAX_PHASES)
    out_lo, out_hi = np.zeros(ATREX_MAX_PHASES, dtype=np.uint64), np.zeros(ATREX_MAX_PHASES, dtype=np.uint64)
    rc = atrex_totals_combine(lo.ctypes.data, hi.ctypes.data, lo.shape[0], out_lo.ctypes.data, out_hi.ctypes.data)
    if rc != ATREX_OK:
        raise AtrexError(rc, "atrex_totals_combine")
    return out_lo, out_hi


class Aggregator:
    """One aggregation handle on one GPU.  Thin object wrapper over the C calls."""

    def __init__(self, app_weights, n_phases: int, max_keys: int, max_work_rows: int = 0, device: int = 0,
                 flags: int = 0, own_workspace: bool = False):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the aggregation path is CUDA-only and no CUDA device is available")
        self._torch = torch
        self.device = int(device)
        w = np.ascontiguousarray(app_weights, dtype=np.uint32)
        cfg = atrex_agg_config_t()
        cfg.n_apps, cfg.n_phases = int(w.shape[0]), int(n_phases)
        cfg.max_keys, cfg.max_work_rows = int(max_keys), int(max_work_rows)
        cfg.app_weights = w.ctypes.data
        cfg.device, cfg.flags = self.device, int(flags)
        self._ws = None
        if not own_workspace:
            nbytes = atrex_agg_workspace_bytes(C.byref(cfg))
            if nbytes == 0:
                raise AtrexError(ATREX_ERR_INVALID, "atrex_agg_workspace_bytes")
            self._ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=f"cuda:{self.device}")
            base = (self._ws.data_ptr() + 255) // 256 * 256
            cfg.workspace, cfg.workspace_bytes = base, nbytes
        h = C.c_void_p()
        rc = atrex_agg_create(C.byref(cfg), C.byref(h))
        if rc != ATREX_OK:
            raise AtrexError(rc, "atrex_agg_create")
        self._h = h
        self.workspace_bytes = int(cfg.workspace_bytes)

    # -- helpers
    def _stream(self, stream=None):
        if stream is None:
            return self._torch.cuda.current_stream(self.device).cuda_stream
        return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)

    def _check(self, rc, where):
        if rc != ATREX_OK:
            raise AtrexError(rc, where, atrex_agg_last_cuda_error(self._h))

    def close(self):
        if getattr(self, "_h", None):
            atrex_agg_destroy(self._h)
            self._h = None
            self._ws = None

    __del__ = close

    # -- the path
    def set_work_table(self, rows: np.ndarray, stream=None):
        r = np.ascontiguousarray(rows)
        assert r.dtype.itemsize == 24
        self._check(atrex_agg_set_work_table(self._h, r.ctypes.data, r.shape[0], self._stream(stream)),
                    "atrex_agg_set_work_table")

    def ingest(self, records, n: int | None = None, stream=None):
        """``records``: CUDA uint8 tensor holding 16-byte records (or a raw device pointer with ``n``)."""
        if isinstance(records, int):
            ptr = records
        else:
            assert records.is_cuda and records.device.index == self.device
            ptr = records.data_ptr()
            if n is None:
                n = records.numel() * records.element_size() // 16
        self._check(atrex_agg_ingest(self._h, ptr, int(n), self._stream(stream)), "atrex_agg_ingest")

    def ingest_host(self, records, n: int | None = None, stream=None):
        """``records``: numpy array or CPU (ideally pinned) tensor of 16-byte records."""
        if isinstance(records, np.ndarray):
            r = np.ascontiguousarray(records)
            ptr, nb = r.ctypes.data, r.nbytes
        else:
            assert not records.is_cuda and records.is_contiguous()
            ptr, nb = records.data_ptr(), records.numel() * records.element_size()
        if n is None:
            n = nb // 16
        self._check(atrex_agg_ingest_host(self._h, ptr, int(n), self._stream(stream)), "atrex_agg_ingest_host")

    def merge(self, entries, n: int | None = None, stream=None):
        assert entries.is_cuda
        if n is None:
            n = entries.numel() * entries.element_size() // 48
        self._check(atrex_agg_merge(self._h, entries.data_ptr(), int(n), self._stream(stream)), "atrex_agg_merge")

    def finalize(self, peak_bw: float, peak_flops, out=None, stream=None, global_totals=None):
        """Returns (entries, n): a CUDA uint8 tensor of 48-byte entries and the entry count.

        ``global_totals`` (a list of per-phase 128-bit integers summed over all shards) switches to
        ``atrex_agg_finalize_with_totals``."""
        torch = self._torch
        pk = make_peaks(peak_bw, peak_flops)
        n_out = C.c_uint64(0)
        if global_totals is not None:
            if isinstance(global_totals, tuple) and len(global_totals) == 2 and isinstance(global_totals[0], np.ndarray):
                lo, hi = (np.ascontiguousarray(x, dtype=np.uint64) for x in global_totals)   # (lo[8], hi[8]) words
            else:
                t = list(global_totals) + [0] * (ATREX_MAX_PHASES - len(global_totals))
                lo = np.array([x & 0xFFFFFFFFFFFFFFFF for x in t[:ATREX_MAX_PHASES]], dtype=np.uint64)
                hi = np.array([x >> 64 for x in t[:ATREX_MAX_PHASES]], dtype=np.uint64)

            def call(ptr, cap):
                return atrex_agg_finalize_with_totals(self._h, C.byref(pk), lo.ctypes.data, hi.ctypes.data, ptr, cap,
                                                      C.byref(n_out), self._stream(stream))
            name = "atrex_agg_finalize_with_totals"
        else:
            def call(ptr, cap):
                return atrex_agg_finalize(self._h, C.byref(pk), ptr, cap, C.byref(n_out), self._stream(stream))
            name = "atrex_agg_finalize"
        if out is None:
            self._check(call(None, 0), name)
            out = torch.empty(max(int(n_out.value), 1) * 48, dtype=torch.uint8, device=f"cuda:{self.device}")
        cap = out.numel() * out.element_size() // 48
        self._check(call(out.data_ptr(), cap), name)
        return out, int(n_out.value)

    def finalize_numpy(self, peak_bw: float, peak_flops, stream=None, global_totals=None) -> np.ndarray:
        out, n = self.finalize(peak_bw, peak_flops, stream=stream, global_totals=global_totals)
        return out[: n * 48].cpu().numpy().view(ENTRY_DTYPE).copy()

    def topk(self, phase: int, k: int, stream=None) -> np.ndarray:
        out = np.zeros(max(k, 1), dtype=ENTRY_DTYPE)
        n_out = C.c_uint32(0)
        rc = atrex_agg_topk(self._h, int(phase), int(k), out.ctypes.data, C.byref(n_out), self._stream(stream))
        self._check(rc, "atrex_agg_topk")
        return out[: n_out.value].copy()

    def stats(self, stream=None, check: bool = True) -> dict:
        st = atrex_stats_t()
        rc = atrex_agg_stats(self._h, C.byref(st), self._stream(stream))
        if check:
            self._check(rc, "atrex_agg_stats")
        return {"status": rc, "n_valid": st.n_valid, "n_rejected": st.n_rejected, "n_dropped": st.n_dropped,
                "n_keys": st.n_keys,
                "totals": [int(st.total_lo[p]) | (int(st.total_hi[p]) << 64) for p in range(ATREX_MAX_PHASES)],
                "keys_per_phase": [int(x) for x in st.keys_per_phase], "table_slots": st.table_slots,
                "hot_slots": st.hot_slots, "n_spilled": st.n_spilled, "n_overflow": st.n_overflow,
                "max_spill_fill": st.max_spill_fill, "spill_cap": st.spill_cap, "n_drains": st.n_drains}

    def totals_words(self):
        """(lo[8], hi[8]) uint64 arrays: the per-phase totals of the last finalize (``atrex_agg_totals``)."""
        lo, hi = np.zeros(ATREX_MAX_PHASES, dtype=np.uint64), np.zeros(ATREX_MAX_PHASES, dtype=np.uint64)
        self._check(atrex_agg_totals(self._h, lo.ctypes.data, hi.ctypes.data), "atrex_agg_totals")
        return lo, hi

    def hot_directory(self, stream=None) -> np.ndarray:
        """Keys currently in the shared-memory hot directory (diagnostic)."""
        out = np.zeros(16384, dtype=np.uint64)
        n = C.c_uint32(0)
        self._check(atrex_agg_hot_directory(self._h, out.ctypes.data, out.shape[0], C.byref(n), self._stream(stream)),
                    "atrex_agg_hot_directory")
        return out[: min(n.value, out.shape[0])].copy()

    def reset(self, stream=None):
        self._check(atrex_agg_reset(self._h, self._stream(stream)), "atrex_agg_reset")

    def launch_count(self) -> int:
        return int(atrex_agg_launch_count(self._h))
