"""Parity of the literal Eq. 2-3 operator weights (CUDA) with the oracle, bit for bit."""
import numpy as np
import pytest

import oracle
import tracegen as tg
from tracegen.configs import make_spec
from tests.helpers import load_golden, records_from_dicts

pytestmark = pytest.mark.gpu


def to_dev(recs):
    import torch
    return torch.from_numpy(np.ascontiguousarray(recs).view(np.uint8).reshape(-1)).cuda()


def test_eq3_worked_example_on_gpu(golden_dir):
    import paper_2607_14541_b200 as p
    g = load_golden(golden_dir, "eq3_example.json")
    recs = records_from_dicts(g["records"])
    ow = p.OperatorWeights(g["app_weights"], g["n_ops"], g["n_phases"])
    ow.ingest(to_dev(recs), n=len(recs))
    w, wt, rej = ow.finalize()
    assert list(wt) == g["wtilde"] and rej == 0 and list(w) == [x / 1.78125 for x in g["wtilde"]]
    w, _, _ = ow.finalize(retained=[1, 1, 0])
    assert list(w) == [0.21875 / g["retained_01_sum"], 0.75 / g["retained_01_sum"], 0.0]


@pytest.mark.parametrize("index,n", [(0, 1 << 20), (1, (1 << 22) + 11), (3, (1 << 22) + 5), (4, 1 << 21)])
def test_eq3_parity(index, n):
    import paper_2607_14541_b200 as p
    spec = make_spec(index, small=True, n=n)
    recs = tg.generate(spec)
    recs["op_id"][:7] = 60000                       # outside the operator table: rejected
    recs["app_id"][7:9] = spec.n_apps
    n_ops = spec.n_ops
    retained = (np.arange(n_ops) % 3 != 0).astype(np.uint8)
    ow = p.OperatorWeights(spec.app_weights, n_ops, spec.n_phases)
    for c in np.array_split(recs, 5):               # chunked ingest
        ow.ingest(to_dev(c), n=len(c))
    for ret in (None, retained):
        w, wt, rej = ow.finalize(retained=ret)
        ew, ewt, erej = oracle.eq3_weights(recs, spec.app_weights, n_ops, spec.n_phases, retained=ret)
        assert rej == erej == 9
        assert wt.tobytes() == ewt.tobytes() and w.tobytes() == ew.tobytes()
        assert abs(float(w.sum()) - 1.0) < n_ops * 2.0**-52
    ow.reset()
    w, wt, rej = ow.finalize()
    assert not w.any() and not wt.any() and rej == 0


def test_eq3_beyond_two_to_the_32_records_switches_to_counted_carries():
    """Below 2^32 ingested records no 64-bit cell sum can wrap and ingest uses fire-and-forget
    reductions; from the 2^32-th record on every add returns the old value and wraps are counted.
    A 2^26-record trace is ingested 64 times (the 64th pass crosses the line) and a second trace once
    more.  Cell sums are linear in the durations, so the oracle gets the equivalent trace: the first
    one with every duration multiplied by 64 (they stay below 2^32), followed by the second."""
    import torch
    import paper_2607_14541_b200 as p
    rng = np.random.default_rng(2024)
    n_apps, n_ops, n_phases, n_x, n_y = 64, 16, 2, 1 << 26, (1 << 20) + 3

    def trace(n):
        r = np.zeros(n, dtype=tg.RECORD_DTYPE)
        r["app_id"] = rng.integers(0, n_apps, n, dtype=np.uint32)
        r["op_id"] = rng.integers(0, n_ops, n).astype(np.uint16)
        r["phase"] = rng.integers(0, n_phases, n).astype(np.uint8)
        r["shape_id"] = rng.integers(0, 1 << 20, n, dtype=np.uint32)
        r["duration_ns"] = rng.integers(1, 1 << 26, n, dtype=np.uint32)
        return r
    x, y = trace(n_x), trace(n_y)
    weights = rng.integers(1, 1 << 20, n_apps, dtype=np.uint32)
    ow = p.OperatorWeights(weights, n_ops, n_phases)
    dx, dy = to_dev(x), to_dev(y)
    for _ in range(64):
        ow.ingest(dx, n=n_x)
    ow.ingest(dy, n=n_y)
    w, wt, rej = ow.finalize()
    x["duration_ns"] *= np.uint32(64)
    ew, ewt, erej = oracle.eq3_weights(np.concatenate([x, y]), weights, n_ops, n_phases)
    assert rej == erej == 0
    assert wt.tobytes() == ewt.tobytes() and w.tobytes() == ew.tobytes()
