"""Seeded synthetic production-trace generator.

Stands in for the proprietary inference traces the paper aggregates (Sec. 3.1):
16-byte records (application, operator, serving phase, shape, duration) with the
cardinalities and skews of the five benchmark configurations.  Record ``i`` is a
pure integer function of ``(seed, config, i)`` over host-built tables, so the
numpy sampler (``tracegen.cpu``) and the CUDA sampler (``tracegen.gpu``) emit the
same bytes.

This package holds input recipes only: none of the aggregation, weighting or
roofline arithmetic lives here.  Both the CPU oracle's tests and the CUDA path's
tests draw their inputs from it.
"""
from .layout import RECORD_DTYPE, WORK_DTYPE, ENTRY_DTYPE  # noqa: F401
from .configs import TraceSpec, make_spec, CONFIG_NAMES  # noqa: F401
from .cpu import generate  # noqa: F401
