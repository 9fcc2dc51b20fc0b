"""Recipes for the five benchmark traces.

Index -> workload (record counts use binary units: 1M = 2^20, 1B = 2^30):

0. tiny: 2^20 records, 8 apps, 32 ops x 64 shapes uniform, 2 phases, uniform durations.
1. 2^26 records, 1024 apps with Zipf(1.1) card-hour weights, 64 ops, 4096 shapes drawn
   Zipf(1.2) per op, 30/70 prefill/decode, log-normal durations.
2. 2^28 records over a live-key list of 2^22 (op, shape, phase) triples out of
   256 ops x 2^20 shapes x 3 phases, key rank ~ Zipf(0.8); top-512 per phase.
3. 2^30 records in 8 chunks of 2^27; 4096 apps, 128 ops x 65536 shapes Zipf(1.1).
4. skew: 2^29 records, 90 % on one key, 10 % uniform over 2^21 keys; every weight
   2^20-1 and every duration 2^28-1.

Everything random is drawn through the counter-based mixer in ``tracegen.hashing``
from ``(seed, config, index)``; tables (Zipf CDFs, duration quantiles, per-operator
rank->shape permutations) are built once on the host in float64 and then only looked
up with integer arithmetic, which is what lets the numpy and CUDA samplers agree
byte for byte.  Key domains can be shrunk (``small=True``) and ``n`` overridden so
that the same laws drive second-scale test cases.
"""
from __future__ import annotations

from dataclasses import dataclass, field
import math

import numpy as np

from .hashing import mix64_scalar, mix64, GOLD
from .layout import WORK_DTYPE

CONFIG_NAMES = ["tiny_1M", "zipf_64M", "highcard_256M", "chunked_1B", "skew_512M"]

KIND_UNIFORM = 0      # op, shape, phase uniform
KIND_ZIPF_PER_OP = 1  # op uniform, shape rank ~ Zipf per op, phase Bernoulli
KIND_KEYLIST = 2      # key rank ~ Zipf over a list of distinct (op, shape, phase) triples
KIND_HOTKEY = 3       # one hot key with fixed probability, rest uniform

DUR_UNIFORM = 0
DUR_QTABLE = 1
DUR_CONST = 2

MAX_PHASES = 8
MAX_DTYPES = 8


@dataclass
class TraceSpec:
    """Everything needed to generate one trace and to configure an aggregator for it."""
    index: int
    name: str
    seed: int
    n: int                      # records
    n_chunks: int               # ingest calls the config asks for
    n_apps: int
    n_phases: int
    app_weights: np.ndarray     # uint32[n_apps] card-hour weights
    kind: int
    n_ops: int
    n_shapes: int
    phase_cum: np.ndarray       # uint32[MAX_PHASES]: phase = #(phase_cum[p] <= u16)
    # Zipf law (kinds 1, 2)
    zipf_s: float = 0.0
    n_ranks: int = 0
    cum: np.ndarray | None = None       # uint64[n_ranks], floor(2^64 * CDF), last = 2^64-1
    perm_a: np.ndarray | None = None    # uint32[n_ops] odd multipliers (kind 1)
    perm_b: np.ndarray | None = None    # uint32[n_ops] offsets (kind 1)
    kl_a: int = 0                       # key-list affine map (kind 2)
    kl_b: int = 0
    # hot key (kind 3)
    hot_thresh: int = 0                 # P(hot) = hot_thresh / 2^32
    hot_phase: int = 0
    hot_op: int = 0
    hot_shape: int = 0
    # durations
    dur_kind: int = DUR_UNIFORM
    dur_lo: int = 1000
    dur_range: int = (1 << 28) - 1000
    qtable: np.ndarray | None = None    # uint32[65536]
    # aggregator provisioning and outputs
    max_keys: int = 0
    topk: int = 10
    n_dtypes: int = 1
    base: int = 0                       # 64-bit stream base derived from (seed, index)
    peak_bw: float = 8.0e12
    peak_flops: tuple = (1.0e15, 2.0e15, 4.0e15, 5.0e14, 2.5e14, 1.0e15, 1.0e15, 1.0e15)
    _work: np.ndarray | None = field(default=None, repr=False)

    @property
    def chunk_records(self) -> int:
        return self.n // self.n_chunks

    def work_table(self) -> np.ndarray:
        """Per-(op, shape) semantic FLOPs and bytes, log-uniform in [1e6, 1e13]."""
        if self._work is None:
            self._work = _build_work_table(self)
        return self._work


def _zipf_cum(n_ranks: int, s: float) -> np.ndarray:
    r = np.arange(1, n_ranks + 1, dtype=np.float64)
    p = r ** (-s)
    cdf = np.cumsum(p)
    cdf /= cdf[-1]
    # floor(2^64 * cdf) without overflowing the float -> uint64 conversion at cdf == 1
    scaled = np.minimum(cdf * 18446744073709551616.0, 18446744073709549568.0)
    cum = scaled.astype(np.uint64)
    cum[-1] = np.uint64(0xFFFFFFFFFFFFFFFF)
    return np.maximum.accumulate(cum)


def _lognormal_qtable(mu: float, sigma: float, lo: int, hi: int) -> np.ndarray:
    from scipy.special import ndtri
    q = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
    d = np.rint(np.exp(mu + sigma * ndtri(q)))
    return np.clip(d, lo, hi).astype(np.uint32)


def _zipf_weights(n_apps: int, s: float, base: int) -> np.ndarray:
    # the app at popularity rank rho (1-based) gets max(1, floor((2^20-1) * rho^-s));
    # ranks are assigned to app ids by a seeded permutation
    rho = np.arange(1, n_apps + 1, dtype=np.float64)
    w = np.maximum(1, np.floor(((1 << 20) - 1) * rho ** (-s))).astype(np.uint32)
    order = np.argsort(mix64(np.uint64(base) + np.arange(n_apps, dtype=np.uint64) * GOLD), kind="stable")
    out = np.empty(n_apps, dtype=np.uint32)
    out[order] = w
    return out


def _uniform_weights(n_apps: int, base: int) -> np.ndarray:
    h = mix64(np.uint64(base) + np.arange(n_apps, dtype=np.uint64) * GOLD)
    return (np.uint64(1) + (((h >> np.uint64(32)) * np.uint64((1 << 20) - 1)) >> np.uint64(32))).astype(np.uint32)


def _log2(x: int) -> int:
    assert x > 0 and x & (x - 1) == 0, "power of two expected"
    return x.bit_length() - 1


def make_spec(index: int, *, seed: int = 0, n: int | None = None, small: bool = False,
              n_dtypes: int = 1) -> TraceSpec:
    """Build the recipe for benchmark configuration ``index`` (0..4).

    ``n`` overrides the record count; ``small`` shrinks the key domain (same law, fewer
    operators/shapes) so the oracle finishes in seconds; ``n_dtypes`` > 1 spreads the
    work-table rows over several dtype indices to exercise per-dtype compute peaks.
    """
    if not 0 <= index < 5:
        raise ValueError("config index must be 0..4")
    base = mix64_scalar((seed * 0xD1342543DE82EF95 + (index + 1) * 0xA0761D6478BD642F) & 0xFFFFFFFFFFFFFFFF)
    wbase = mix64_scalar(base ^ 0x5851F42D4C957F2D)
    pc = np.full(MAX_PHASES, 0xFFFFFFFF, dtype=np.uint32)
    common = dict(index=index, name=CONFIG_NAMES[index], seed=seed, base=base, n_dtypes=n_dtypes)
    qt = lambda: _lognormal_qtable(math.log(5e4), 1.5, 1000, (1 << 28) - 1)

    if index == 0:
        pc[0] = 32768
        return TraceSpec(n=n or 1 << 20, n_chunks=1, n_apps=8, n_phases=2,
                         app_weights=_uniform_weights(8, wbase), kind=KIND_UNIFORM,
                         n_ops=32, n_shapes=64, phase_cum=pc, dur_kind=DUR_UNIFORM,
                         max_keys=32 * 64 * 2, topk=10, **common)
    if index == 1:
        n_ops, n_shapes = (16, 512) if small else (64, 4096)
        pc[0] = 19661  # 0.3 * 65536
        return TraceSpec(n=n or 1 << 26, n_chunks=1, n_apps=1024, n_phases=2,
                         app_weights=_zipf_weights(1024, 1.1, wbase), kind=KIND_ZIPF_PER_OP,
                         n_ops=n_ops, n_shapes=n_shapes, phase_cum=pc, zipf_s=1.2,
                         n_ranks=n_shapes, cum=_zipf_cum(n_shapes, 1.2),
                         perm_a=_perm_tables(n_ops, base)[0], perm_b=_perm_tables(n_ops, base)[1],
                         dur_kind=DUR_QTABLE, qtable=qt(), max_keys=n_ops * n_shapes * 2, topk=10, **common)
    if index == 2:
        n_ops, n_shapes, n_live = (32, 1 << 14, 1 << 16) if small else (256, 1 << 20, 1 << 22)
        domain = 3 * n_ops * n_shapes
        kl_a = (mix64_scalar(base ^ 0x1234567) % domain) | 1
        while math.gcd(kl_a, domain) != 1:
            kl_a += 2
        kl_b = mix64_scalar(base ^ 0x89ABCDEF) % domain
        return TraceSpec(n=n or 1 << 28, n_chunks=1, n_apps=256, n_phases=3,
                         app_weights=_uniform_weights(256, wbase), kind=KIND_KEYLIST,
                         n_ops=n_ops, n_shapes=n_shapes, phase_cum=pc, zipf_s=0.8,
                         n_ranks=n_live, cum=_zipf_cum(n_live, 0.8), kl_a=kl_a, kl_b=kl_b,
                         dur_kind=DUR_QTABLE, qtable=qt(), max_keys=n_live, topk=512, **common)
    if index == 3:
        n_ops, n_shapes = (16, 2048) if small else (128, 65536)
        pc[0] = 19661
        pa, pb = _perm_tables(n_ops, base)
        return TraceSpec(n=n or 1 << 30, n_chunks=8, n_apps=4096, n_phases=2,
                         app_weights=_zipf_weights(4096, 1.1, wbase), kind=KIND_ZIPF_PER_OP,
                         n_ops=n_ops, n_shapes=n_shapes, phase_cum=pc, zipf_s=1.1,
                         n_ranks=n_shapes, cum=_zipf_cum(n_shapes, 1.1), perm_a=pa, perm_b=pb,
                         dur_kind=DUR_QTABLE, qtable=qt(), max_keys=n_ops * n_shapes * 2, topk=10, **common)
    # index == 4
    n_ops, n_shapes = (16, 1024) if small else (64, 16384)
    return TraceSpec(n=n or 1 << 29, n_chunks=1, n_apps=64, n_phases=2,
                     app_weights=np.full(64, (1 << 20) - 1, dtype=np.uint32), kind=KIND_HOTKEY,
                     n_ops=n_ops, n_shapes=n_shapes, phase_cum=pc,
                     hot_thresh=int(0.9 * (1 << 32)), hot_phase=1, hot_op=0, hot_shape=0,
                     dur_kind=DUR_CONST, dur_lo=(1 << 28) - 1, dur_range=1,
                     max_keys=2 * n_ops * n_shapes, topk=10, **common)


def _perm_tables(n_ops: int, base: int):
    i = np.arange(n_ops, dtype=np.uint64)
    a = (mix64(np.uint64(base ^ 0x0A0A0A0A) + i * GOLD) >> np.uint64(32)).astype(np.uint32) | np.uint32(1)
    b = (mix64(np.uint64(base ^ 0x0B0B0B0B) + i * GOLD) >> np.uint64(32)).astype(np.uint32)
    return a, b


def _build_work_table(spec: TraceSpec) -> np.ndarray:
    if spec.kind == KIND_KEYLIST:
        # one row per (op, shape) pair that a live key uses
        domain = 3 * spec.n_ops * spec.n_shapes
        r = np.arange(spec.n_ranks, dtype=np.uint64)
        t = (r * np.uint64(spec.kl_a) + np.uint64(spec.kl_b)) % np.uint64(domain)
        pair = np.unique(t % np.uint64(spec.n_ops * spec.n_shapes))
        op = (pair // np.uint64(spec.n_shapes)).astype(np.uint16)
        shape = (pair % np.uint64(spec.n_shapes)).astype(np.uint32)
    else:
        pair = np.arange(spec.n_ops * spec.n_shapes, dtype=np.uint64)
        op = (pair // np.uint64(spec.n_shapes)).astype(np.uint16)
        shape = (pair % np.uint64(spec.n_shapes)).astype(np.uint32)
    rows = np.zeros(pair.shape[0], dtype=WORK_DTYPE)
    rows["op_id"] = op
    rows["shape_id"] = shape
    wb = np.uint64(mix64_scalar(spec.base ^ 0x77777777))
    two53 = float(1 << 53)
    for col, off in (("flops", 0), ("bytes", 1)):
        h = mix64(wb + (pair * np.uint64(2) + np.uint64(off)) * GOLD)
        u = (h >> np.uint64(11)).astype(np.float64) / two53
        rows[col] = np.floor(np.power(10.0, 6.0 + 7.0 * u)).astype(np.uint64)
    if spec.n_dtypes > 1:
        h = mix64(wb + (pair * np.uint64(2) + np.uint64(7)) * GOLD)
        rows["dtype"] = ((h >> np.uint64(40)) % np.uint64(spec.n_dtypes)).astype(np.uint16)
    return rows
