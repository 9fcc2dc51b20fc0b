"""Byte layouts of the buffers that cross the library boundary (little-endian).

These are descriptions of input/output buffers only, used by the generators and
by the test harness to view raw bytes; each implementation declares its own
structs.
"""
import numpy as np

# One device-kernel invocation observed by the tracer (Sec. 3.1, Eq. 2's d_{a,phi,r,l}).
RECORD_DTYPE = np.dtype(
    [("app_id", "<u4"), ("op_id", "<u2"), ("phase", "u1"), ("pad", "u1"),
     ("shape_id", "<u4"), ("duration_ns", "<u4")], align=False)
assert RECORD_DTYPE.itemsize == 16

# Semantic work F_j / traffic M_j of one (operator, shape) unit (Sec. 3.3).
WORK_DTYPE = np.dtype(
    [("shape_id", "<u4"), ("op_id", "<u2"), ("dtype", "<u2"),
     ("flops", "<u8"), ("bytes", "<u8")], align=False)
assert WORK_DTYPE.itemsize == 24

# One aggregated (operator, shape, phase) unit.
ENTRY_DTYPE = np.dtype(
    [("key", "<u8"), ("count", "<u8"), ("wt_lo", "<u8"), ("wt_hi", "<u8"),
     ("phase_weight", "<f8"), ("roofline_s", "<f8")], align=False)
assert ENTRY_DTYPE.itemsize == 48
