"""Parity of the score-aggregation kernel (Eq. 4-6) with the oracle, bit for bit."""
import numpy as np
import pytest

import oracle
from tests.helpers import load_golden

pytestmark = pytest.mark.gpu


def run_gpu(roof, unit_op, t, ok, w):
    import torch
    import paper_2607_14541_b200 as p
    d = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).cuda()
    s_agg, s_op, err = p.score_aggregate(d(roof, np.float64), d(unit_op, np.int32), d(t, np.float64),
                                         d(ok, np.uint8), d(w, np.float64))
    torch.cuda.synchronize()
    return s_agg.cpu().numpy(), s_op.cpu().numpy(), err.cpu().numpy().astype(np.uint64)


def test_score_worked_example_on_gpu(golden_dir):
    g = load_golden(golden_dir, "score_example.json")
    u = g["units"]
    agg, s_op, err = run_gpu([x["roofline_s"] for x in u], [x["op"] for x in u], [[x["t_cand"] for x in u]],
                             [[x["correct"] for x in u]], g["w"])
    assert list(s_op[0]) == g["S_op"] and float(agg[0]) == g["S_agg"] and int(err[0]) == g["errors"]


@pytest.mark.parametrize("n_ops,n_units,batch,seed", [(30, 440, 64, 0), (1, 1, 3, 1), (257, 5000, 17, 2), (4, 16384, 2, 3)])
def test_score_parity_random_batches(n_ops, n_units, batch, seed):
    rng = np.random.default_rng(seed)
    unit_op = rng.integers(0, n_ops, n_units).astype(np.uint32)            # unsorted on purpose
    if n_units > 10:
        unit_op[:3] = n_ops + 5                                           # out-of-range operators are ignored
    roof = np.exp(rng.uniform(np.log(1e-6), np.log(1e-1), n_units))
    w = rng.dirichlet(np.ones(n_ops))
    ratio = rng.uniform(0.01, 1.1, (batch, n_units))
    ratio[:, ::7] = 0.5                                                   # plenty of exact ties
    t = roof[None, :] / ratio
    ok = rng.random((batch, n_units)) < 0.6
    ok[0] = False                                                         # a candidate with nothing correct
    if n_units > 10:
        t[1, 4], t[1, 5], t[1, 6] = np.inf, -1.0, np.nan
        ok[1, 4:7] = True
    exp = oracle.score_candidates(roof, unit_op, t, ok, w)
    got = run_gpu(roof, unit_op, t, ok, w)
    assert got[0].tobytes() == exp[0].tobytes()
    assert got[1].tobytes() == exp[1].tobytes()
    assert np.array_equal(got[2], exp[2])
    assert float(got[0][0]) == 0.0


def test_score_limits():
    import torch
    import paper_2607_14541_b200 as p
    z = torch.zeros(8, dtype=torch.float64, device="cuda")
    assert p.atrex_score_aggregate(z.data_ptr(), z.data_ptr(), p.lib.atrex_score_aggregate.argtypes and 16385, z.data_ptr(),
                                   z.data_ptr(), 1, z.data_ptr(), 1, z.data_ptr(), None, None, None) == p.ATREX_ERR_TOO_LARGE
    assert p.atrex_score_aggregate(None, z.data_ptr(), 4, z.data_ptr(), z.data_ptr(), 1, z.data_ptr(), 1, z.data_ptr(),
                                   None, None, None) == p.ATREX_ERR_INVALID
    assert p.atrex_score_aggregate(None, None, 4, None, None, 0, None, 1, None, None, None, None) == p.ATREX_OK
