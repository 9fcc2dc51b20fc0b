"""Parity at the benchmark's full sizes and launch configuration (up to 2^30 records in 8 chunks of
2^27, the workload bench.py times): every entry of an oracle-chosen slice of the key space (all of
it for the 2^26-record config), recomputed by the oracle from the very same bytes, plus properties
that hold at any size."""
import numpy as np
import pytest

import oracle
from tracegen.configs import make_spec
from tracegen.layout import RECORD_DTYPE
from tests.helpers import f64_bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("index", [1, 2, 3, 4])
def test_full_size_trace_key_slice_and_invariants(index):
    import torch
    import paper_2607_14541_b200 as p
    from tracegen.gpu import GpuSampler

    free, _ = torch.cuda.mem_get_info()
    if free < 40 << 30:
        pytest.skip("needs ~30 GB of device memory")
    spec = make_spec(index)
    n, chunk = spec.n, spec.chunk_records
    work = spec.work_table()
    agg = p.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys, max_work_rows=len(work))
    agg.set_work_table(work)
    sampler = GpuSampler(spec)
    records = torch.empty(n * 16, dtype=torch.uint8, device="cuda:0")
    sampler.fill(records, 0, n)
    for c in range(spec.n_chunks):
        agg.ingest(records[c * chunk * 16:(c + 1) * chunk * 16], n=chunk)
    ent = agg.finalize_numpy(spec.peak_bw, spec.peak_flops)
    st = agg.stats()

    # properties that hold at any size
    assert st["n_valid"] == n and st["n_rejected"] == 0 and st["n_dropped"] == 0 and st["n_overflow"] == 0
    assert int(ent["count"].sum()) == n and len(ent) == st["n_keys"] == len(np.unique(ent["key"]))
    for ph in range(spec.n_phases):
        sel = ent[(ent["key"] >> np.uint64(48)) == ph]
        tot = int(sel["wt_lo"].astype(object).sum()) + (int(sel["wt_hi"].astype(object).sum()) << 64)
        assert tot == st["totals"][ph]
        assert abs(float(np.sum(sel["phase_weight"], dtype=np.longdouble)) - 1.0) < 3 * len(sel) * 2.0**-53

    # A slice of the key space chosen by a predicate on the key alone (a fixed scramble of the packed
    # key, modulo SLICES; the GPU's output plays no part in the choice): the oracle aggregates exactly
    # that slice from the very same bytes, chunk by chunk, and EVERY entry of the slice is compared,
    # both doubles included -- a key the GPU lost, invented or mixed up inside the slice fails.
    # Config 1 (2^26 records) is compared in full (one class).  The per-phase totals that Eq. 3
    # divides by are summed by the oracle straight from the records.
    slices = 1 if index == 1 else 64
    residue = (7 * index + 3) % slices
    o = oracle.Oracle(spec.app_weights, spec.n_phases)
    o.set_work(work)
    acc, valid = np.zeros(16, dtype=np.uint64), np.zeros(2, dtype=np.uint64)
    piece = 1 << 27                                         # host copies of at most 2 GiB at a time
    for lo in range(0, n, piece):
        host = records[lo * 16:min(lo + piece, n) * 16].cpu().numpy().view(RECORD_DTYPE)
        o.ingest_slice(host, slices, residue, threads=0)
        o.direct_totals(host, acc, valid)
    assert int(valid[0]) == n and int(valid[1]) == 0
    totals = [int(acc[2 * q]) | (int(acc[2 * q + 1]) << 64) for q in range(8)]
    assert totals == st["totals"]
    exp = o.finalize_given_totals(spec.peak_bw, spec.peak_flops, totals)
    mine = ent[oracle.slice_class(ent["key"], slices) == residue]
    got = mine[np.argsort(mine["key"], kind="stable")]
    assert len(exp) == len(got) and len(got) >= len(ent) // (2 * slices)
    assert np.array_equal(exp["key"], got["key"])
    assert exp.tobytes() == got.tobytes()
    del o, exp, mine

    # the ranking: top-k must be the k largest (wt, then smaller key) of the phase's entries
    for ph in range(spec.n_phases):
        sel = ent[(ent["key"] >> np.uint64(48)) == ph]
        # pre-select by the high word and the top of the low word, then rank exactly
        coarse = sel["wt_hi"].astype(np.float64) * 2.0**64 + sel["wt_lo"].astype(np.float64)
        keep = sel[np.argsort(-coarse, kind="stable")[: 4 * spec.topk + 64]]
        wt = keep["wt_hi"].astype(object) * (1 << 64) + keep["wt_lo"].astype(object)
        best = sorted(zip((-wt).tolist(), keep["key"].tolist()))[: spec.topk]
        top = agg.topk(ph, spec.topk)
        assert [int(k) for k in top["key"]] == [k for _, k in best]
        assert float(coarse[np.argsort(-coarse, kind="stable")[4 * spec.topk + 63]]) < float(-best[-1][0]) or len(sel) <= 4 * spec.topk + 64

    if index == 4:   # every weight 2^20-1, every duration 2^28-1: wt = count * P, with carries into the high word
        P = (2**20 - 1) * (2**28 - 1)
        wt_all = ent["wt_hi"].astype(object) * (1 << 64) + ent["wt_lo"].astype(object)
        assert (wt_all == ent["count"].astype(object) * P).all()
        assert int(ent["wt_hi"].max()) > 6000

    # chunking must not matter: the same 2^30 records in ONE call give the same entries
    if index == 3:
        agg1 = p.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys, max_work_rows=len(work))
        agg1.set_work_table(work)
        agg1.ingest(records, n=n)
        a, na = agg1.finalize(spec.peak_bw, spec.peak_flops)
        b, nb = agg.finalize(spec.peak_bw, spec.peak_flops)
        assert na == nb and torch.equal(p.sort_entries_by_key(a, na), p.sort_entries_by_key(b, nb))
        del agg1, a, b

    # the release artefacts made from this entry list (config 2's three phases and config 3's
    # 16 M entries exercise every word of the ranking order and several sort tiles per digit)
    if index in (2, 3):
        check_release_artefacts(p, agg, spec, ent, st)


def _prefix_ints(wt_lo, wt_hi, positions):
    """Exact inclusive prefix sums of 128-bit values at the given positions: numpy running sums of
    32-bit pieces (no overflow below 2^32 rows), recombined as Python integers."""
    mask = np.uint64(0xFFFFFFFF)
    pieces = [wt_lo & mask, wt_lo >> np.uint64(32), wt_hi & mask, wt_hi >> np.uint64(32)]
    sums = [np.cumsum(x, dtype=np.uint64) for x in pieces]
    return [sum(int(s[i]) << (32 * j) for j, s in enumerate(sums)) for i in positions]


def check_release_artefacts(p, agg, spec, ent, st):
    dev_ent, n_ent = agg.finalize(spec.peak_bw, spec.peak_flops)
    by_key = p.sort_entries_by_key(dev_ent, n_ent).cpu().numpy().view(p.ENTRY_DTYPE)
    assert by_key.tobytes() == ent[np.argsort(ent["key"], kind="stable")].tobytes()    # keys are unique
    for ph in range(spec.n_phases):
        ppm = (900_000, 500_000, 999_999)[ph % 3]
        ranked, cum, res = p.rank_entries(dev_ent, n_ent, ph, ppm)
        ranked = ranked.cpu().numpy().view(p.ENTRY_DTYPE)
        cum = cum.cpu().numpy()
        sel = ent[(ent["key"] >> np.uint64(48)) == ph]
        total = st["totals"][ph]
        assert res["n_phase"] == len(sel) == len(ranked) and res["total"] == total
        # same entries, in (weighted time descending, key ascending) order
        assert np.array_equal(np.sort(ranked["key"]), np.sort(sel["key"]))
        assert ranked[np.argsort(ranked["key"], kind="stable")].tobytes() == sel[np.argsort(sel["key"], kind="stable")].tobytes()
        hi, lo, key = ranked["wt_hi"], ranked["wt_lo"], ranked["key"]
        in_order = (hi[:-1] > hi[1:]) | ((hi[:-1] == hi[1:]) & ((lo[:-1] > lo[1:]) | ((lo[:-1] == lo[1:]) & (key[:-1] < key[1:]))))
        assert in_order.all()
        assert agg.topk(ph, spec.topk).tobytes() == ranked[: spec.topk].tobytes()
        # running share at sampled rows, and the cut, against exact integer prefix sums
        k = res["n_keep"]
        rows = sorted(set([0, 1, len(ranked) // 3, len(ranked) - 1] + [max(k - 2, 0), max(k - 1, 0), min(k, len(ranked) - 1)]
                          + list(range(0, len(ranked), max(1, len(ranked) // 200)))))
        prefix = dict(zip(rows, _prefix_ints(lo, hi, rows)))
        for r in rows:
            assert f64_bits(float(cum[r])) == f64_bits(oracle.u128_to_f64(prefix[r]) / oracle.u128_to_f64(total)), (ph, r)
        assert (np.diff(cum) >= 0).all() and cum[-1] == 1.0
        assert k >= 1 and prefix[k - 1] * 1_000_000 >= ppm * total and res["covered"] == prefix[k - 1]
        assert k == 1 or prefix[k - 2] * 1_000_000 < ppm * total
