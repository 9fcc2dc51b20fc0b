"""The seeded generator: determinism, slicing, and the distributional shape of each law."""
import numpy as np
import pytest

import tracegen as tg
from tracegen.configs import make_spec


@pytest.mark.parametrize("index", [0, 1, 2, 3, 4])
def test_slices_concatenate_and_seed_matters(index):
    spec = make_spec(index, small=True, n=50_000)
    whole = tg.generate(spec)
    parts = np.concatenate([tg.generate(spec, 0, 12_345), tg.generate(spec, 12_345, 50_000 - 12_345)])
    assert whole.tobytes() == parts.tobytes()
    assert whole.tobytes() == tg.generate(make_spec(index, small=True, n=50_000)).tobytes()
    assert whole.tobytes() != tg.generate(make_spec(index, small=True, n=50_000, seed=1)).tobytes()
    assert whole["app_id"].max() < spec.n_apps and whole["phase"].max() < spec.n_phases
    assert whole["op_id"].max() < spec.n_ops and whole["shape_id"].max() < spec.n_shapes
    assert not whole["pad"].any()


def test_law_shapes():
    s = make_spec(1, n=1 << 20)
    r = tg.generate(s)
    assert abs((r["phase"] == 0).mean() - 0.3) < 0.005
    assert r["duration_ns"].min() >= 1000 and r["duration_ns"].max() < (1 << 28)
    assert 3.0e4 < np.median(r["duration_ns"]) < 7.0e4              # log-normal, median 5e4
    s = make_spec(4, small=True, n=1 << 18)
    r = tg.generate(s)
    hot = (r["phase"] == 1) & (r["op_id"] == 0) & (r["shape_id"] == 0)
    assert abs(hot.mean() - 0.9) < 0.01
    assert (r["duration_ns"] == (1 << 28) - 1).all() and (s.app_weights == (1 << 20) - 1).all()
    s = make_spec(0)
    r = tg.generate(s)
    assert r["duration_ns"].min() >= 1000 and len(np.unique(r["shape_id"])) == 64 and len(np.unique(r["op_id"])) == 32
    s = make_spec(2, small=True, n=1 << 18)
    assert len(s.work_table()) <= s.n_ranks and len(np.unique(tg.generate(s)["phase"])) == 3
