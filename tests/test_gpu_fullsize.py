"""Parity at the benchmark's full size and launch configuration (2^30 records in 8 chunks of
2^27, the workload bench.py times): sampled outputs the oracle computes one by one from the
very same bytes, plus properties that hold at any size."""
import numpy as np
import pytest

import oracle
from tracegen.configs import make_spec
from tracegen.layout import RECORD_DTYPE
from tests.helpers import entry_wt, f64_bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("index", [1, 2, 3, 4])
def test_full_size_trace_sampled_keys_and_invariants(index):
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

    # sampled keys: hottest, coldest and a spread in between, recomputed by the oracle from
    # the same bytes (chunk by chunk), together with the per-phase totals as a plain sum
    order = np.argsort(ent["count"], kind="stable")
    pick = np.unique(np.concatenate([order[:40], order[-40:], order[:: max(1, len(order) // 120)]]))
    keys = ent["key"][pick]
    o = oracle.Oracle(spec.app_weights, spec.n_phases)
    o.set_work(work)
    acc, valid = np.zeros(16, dtype=np.uint64), np.zeros(2, dtype=np.uint64)
    piece = 1 << 27                                         # host copies of at most 2 GiB at a time
    for lo in range(0, n, piece):
        host = records[lo * 16:min(lo + piece, n) * 16].cpu().numpy().view(RECORD_DTYPE)
        o.ingest_filtered(host, keys)
        o.direct_totals(host, acc, valid)
    assert int(valid[0]) == n and int(valid[1]) == 0
    totals = [int(acc[2 * q]) | (int(acc[2 * q + 1]) << 64) for q in range(8)]
    assert totals == st["totals"]
    exp = o.finalize(spec.peak_bw, spec.peak_flops)          # weights here are relative to the sample only
    got = ent[pick][np.argsort(ent["key"][pick], kind="stable")]
    assert np.array_equal(exp["key"], got["key"])
    assert np.array_equal(exp["count"], got["count"])
    assert np.array_equal(exp["wt_lo"], got["wt_lo"]) and np.array_equal(exp["wt_hi"], got["wt_hi"])
    assert np.array_equal(exp["roofline_s"].view(np.uint64), got["roofline_s"].view(np.uint64))
    for e in got:                                            # Eq. 3 against the independently summed totals
        t = totals[int(e["key"]) >> 48]
        assert f64_bits(float(e["phase_weight"])) == f64_bits(oracle.u128_to_f64(entry_wt(e)) / oracle.u128_to_f64(t))

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
