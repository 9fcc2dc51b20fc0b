"""numpy sampler: record ``i`` of a TraceSpec as a pure integer function of ``i``.

The CUDA sampler in ``tracegen/csrc/tracegen.cu`` restates exactly these steps.
"""
from __future__ import annotations

import numpy as np

from . import configs as C
from .hashing import word
from .layout import RECORD_DTYPE

_U32 = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def _rank(spec, h):
    r = np.searchsorted(spec.cum, h, side="right").astype(np.uint64)
    return np.minimum(r, np.uint64(spec.n_ranks - 1))


def _generate_block(spec, idx: np.ndarray) -> np.ndarray:
    h0, h1, h2 = word(spec.base, 0, idx), word(spec.base, 1, idx), word(spec.base, 2, idx)
    out = np.zeros(idx.shape[0], dtype=RECORD_DTYPE)
    out["app_id"] = (((h0 & _U32) * np.uint64(spec.n_apps)) >> _S32).astype(np.uint32)

    per_phase = np.uint64(spec.n_ops * spec.n_shapes)
    if spec.kind in (C.KIND_UNIFORM, C.KIND_ZIPF_PER_OP):
        op = ((((h0 >> _S32) & np.uint64(0xFFFF)) * np.uint64(spec.n_ops)) >> np.uint64(16))
        u16 = (h0 >> np.uint64(48)).astype(np.uint32)
        phase = np.zeros(idx.shape[0], dtype=np.uint32)
        for p in range(spec.n_phases - 1):
            phase += (u16 >= spec.phase_cum[p]).astype(np.uint32)
        if spec.kind == C.KIND_UNIFORM:
            shape = ((h1 & _U32) * np.uint64(spec.n_shapes)) >> _S32
        else:
            rank = _rank(spec, h1)
            a = spec.perm_a[op.astype(np.int64)].astype(np.uint64)
            b = spec.perm_b[op.astype(np.int64)].astype(np.uint64)
            shape = (rank * a + b) & np.uint64(spec.n_shapes - 1)
    elif spec.kind == C.KIND_KEYLIST:
        rank = _rank(spec, h1)
        t = (rank * np.uint64(spec.kl_a) + np.uint64(spec.kl_b)) % (np.uint64(3) * per_phase)
        phase = t // per_phase
        rem = t % per_phase
        op = rem // np.uint64(spec.n_shapes)
        shape = rem % np.uint64(spec.n_shapes)
    else:  # KIND_HOTKEY
        hot = (h1 & _U32) < np.uint64(spec.hot_thresh)
        cold = ((h1 >> _S32) * (np.uint64(spec.n_phases) * per_phase)) >> _S32
        phase = np.where(hot, np.uint64(spec.hot_phase), cold // per_phase)
        rem = cold % per_phase
        op = np.where(hot, np.uint64(spec.hot_op), rem // np.uint64(spec.n_shapes))
        shape = np.where(hot, np.uint64(spec.hot_shape), rem % np.uint64(spec.n_shapes))
    out["op_id"] = op.astype(np.uint16)
    out["phase"] = phase.astype(np.uint8)
    out["shape_id"] = shape.astype(np.uint32)

    if spec.dur_kind == C.DUR_UNIFORM:
        d = np.uint64(spec.dur_lo) + (((h2 & _U32) * np.uint64(spec.dur_range)) >> _S32)
    elif spec.dur_kind == C.DUR_QTABLE:
        d = spec.qtable[(h2 >> np.uint64(48)).astype(np.int64)]
    else:
        d = np.full(idx.shape[0], spec.dur_lo, dtype=np.uint64)
    out["duration_ns"] = d.astype(np.uint32)
    return out


def generate(spec, start: int = 0, count: int | None = None, block: int = 1 << 22) -> np.ndarray:
    """Records ``start .. start+count`` of the trace described by ``spec``."""
    if count is None:
        count = spec.n - start
    out = np.empty(count, dtype=RECORD_DTYPE)
    with np.errstate(over="ignore"):
        for off in range(0, count, block):
            m = min(block, count - off)
            idx = np.arange(start + off, start + off + m, dtype=np.uint64)
            out[off:off + m] = _generate_block(spec, idx)
    return out
