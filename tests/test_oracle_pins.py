"""Pins for the CPU oracle: hand-computed traces, closed forms, brute force, invariants.

Each test is chosen so that a plausible slip in the oracle (a dropped weight, a swapped
operand, a wrong shift in the key, a per-trace instead of per-phase normaliser, a double
rounding) makes it fail.  None of them calls the CUDA path.
"""
from fractions import Fraction
import math
import random
import struct

import numpy as np
import pytest

import oracle
import tracegen as tg
from tracegen.configs import make_spec
from tracegen.layout import RECORD_DTYPE, WORK_DTYPE
from tests.helpers import (load_golden, f64_bits, records_from_dicts, work_from_dicts, brute_force,
                           expected_entry_fields, check_entries_against, entry_wt, sorted_by_key)

PEAK_BW = 8.0e12
PEAK_FLOPS = [1.0e15, 2.0e15, 4.0e15, 5.0e14, 2.5e14, 1.0e15, 1.0e15, 1.0e15]


def run_oracle(records, app_weights, n_phases, work=None, threads=1, peak_bw=PEAK_BW, peak_flops=PEAK_FLOPS):
    o = oracle.Oracle(app_weights, n_phases)
    if work is not None:
        assert o.set_work(work) == 0
    o.ingest(records, threads=threads)
    return o, o.finalize(peak_bw, peak_flops)


# ---------------------------------------------------------------- hand-computed traces

def test_worked_example_a(golden_dir):
    g = load_golden(golden_dir, "worked_example_a.json")
    recs = records_from_dicts(g["records"])
    work = work_from_dicts(g["work"])
    o, ent = run_oracle(recs, g["app_weights"], g["n_phases"], work, peak_bw=g["peak_bw"], peak_flops=g["peak_flops"])
    assert len(ent) == len(g["expected"])
    for e, x in zip(ent, g["expected"]):  # finalize is key-ascending, so is the fixture
        assert int(e["key"]) == int(x["key"], 16)
        assert int(e["count"]) == x["count"]
        assert entry_wt(e) == x["wt"]
        assert f64_bits(float(e["phase_weight"])) == int(x["phase_weight_bits"], 16)
        assert f64_bits(float(e["roofline_s"])) == int(x["roofline_bits"], 16)
    st = o.stats()
    assert st["n_valid"] == 7 and st["n_rejected"] == 0 and st["n_keys"] == 4
    assert st["totals"][0] == g["phase_totals"]["0"] and st["totals"][1] == g["phase_totals"]["1"]
    for t in g["topk"]:
        top = o.topk(g["peak_bw"], g["peak_flops"], t["phase"], t["k"])
        assert [int(k) for k in top["key"]] == [int(k, 16) for k in t["keys"]]


def test_carry_closed_form(golden_dir):
    g = load_golden(golden_dir, "carry_closed_form.json")
    assert g["P"] == g["weight"] * g["duration_ns"] == (2**20 - 1) * (2**28 - 1)
    for case in g["cases"]:
        n = case["N"]
        recs = np.zeros(n, dtype=RECORD_DTYPE)
        recs["op_id"], recs["shape_id"], recs["phase"], recs["duration_ns"] = 3, 11, 1, g["duration_ns"]
        o, ent = run_oracle(recs, [g["weight"]], 2)
        assert len(ent) == 1
        assert int(ent[0]["count"]) == n
        assert int(ent[0]["wt_hi"]) == case["wt_hi"]
        assert int(ent[0]["wt_lo"]) == int(case["wt_lo"], 16)
        assert entry_wt(ent[0]) == n * g["P"]
        assert f64_bits(oracle.u128_to_f64(n * g["P"])) == int(case["f64_bits"], 16)
        assert f64_bits(float(ent[0]["phase_weight"])) == f64_bits(1.0)
    big = g["large_case_not_run_on_cpu"]
    x = big["N"] * g["P"]
    assert x >> 64 == big["wt_hi"] and x & (2**64 - 1) == int(big["wt_lo"], 16)
    assert f64_bits(oracle.u128_to_f64(x)) == int(big["f64_bits"], 16)


def test_topk_uses_exact_integers_then_key(golden_dir):
    g = load_golden(golden_dir, "topk_ties.json")
    c = g["case_rounding"]
    rows = []
    for name in ("x", "y"):
        k = c[name]
        rows += [{"app": 0, "op": k["op"], "shape": k["shape"], "duration_ns": k["big_duration"]}] * k["n_big"]
        if "extra_duration" in k:
            rows.append({"app": 1, "op": k["op"], "shape": k["shape"], "duration_ns": k["extra_duration"]})
    recs = records_from_dicts(rows)
    o, ent = run_oracle(recs, c["app_weights"], 1)
    by_key = {int(e["key"]): e for e in ent}
    assert entry_wt(by_key[5]) == c["x"]["wt"] == 2**54 + 1
    assert entry_wt(by_key[3]) == c["y"]["wt"] == 2**54
    # the two doubles coincide, the integers do not
    assert f64_bits(float(by_key[5]["phase_weight"])) == f64_bits(float(by_key[3]["phase_weight"]))
    top = o.topk(PEAK_BW, PEAK_FLOPS, 0, 2)
    assert [int(k) for k in top["key"]] == [int(k, 16) for k in c["top2_keys"]]

    t = g["case_exact_ties"]
    o, _ = run_oracle(records_from_dicts(t["records"]), t["app_weights"], 1)
    assert [int(k) for k in o.topk(PEAK_BW, PEAK_FLOPS, 0, 3)["key"]] == [int(k, 16) for k in t["top3_keys"]]
    assert [int(k) for k in o.topk(PEAK_BW, PEAK_FLOPS, 0, 9)["key"]] == [int(k, 16) for k in t["top4_keys"]]
    assert len(o.topk(PEAK_BW, PEAK_FLOPS, 0, 0)) == 0


# ---------------------------------------------------------------- integer -> binary64

def test_u128_to_f64_vectors(golden_dir):
    g = load_golden(golden_dir, "u128_to_f64_vectors.json")
    for v in g["vectors"]:
        x = (int(v["hi"], 16) << 64) | int(v["lo"], 16)
        assert f64_bits(oracle.u128_to_f64(x)) == int(v["bits"], 16), v
        if v.get("double_rounding_trap"):
            naive = float(int(v["hi"], 16)) * 2.0**64 + float(int(v["lo"], 16))
            assert f64_bits(naive) != int(v["bits"], 16)


def _rne_reference(x: int) -> float:
    """Round-to-nearest-even of a non-negative integer to binary64, from first principles."""
    if x == 0:
        return 0.0
    e = x.bit_length() - 53
    if e <= 0:
        return math.ldexp(float(x), 0)
    q, r = x >> e, x & ((1 << e) - 1)
    half = 1 << (e - 1)
    if r > half or (r == half and (q & 1)):
        q += 1
    return math.ldexp(float(q), e)


def test_u128_to_f64_random_against_first_principles():
    rng = random.Random(1234)
    for _ in range(20000):
        bits = rng.randrange(1, 129)
        x = rng.getrandbits(bits)
        if rng.random() < 0.3:  # force values near a rounding boundary
            e = max(x.bit_length() - 53, 1)
            x = ((x >> e) << e) | (1 << (e - 1)) | rng.choice([0, 0, 1])
        x &= (1 << 128) - 1
        assert oracle.u128_to_f64(x) == _rne_reference(x)


# ---------------------------------------------------------------- brute force, every law

@pytest.mark.parametrize("index", [0, 1, 2, 3, 4])
def test_brute_force_python_ints(index):
    spec = make_spec(index, small=True, n=4096, n_dtypes=3)
    recs = tg.generate(spec)
    # add a few invalid records and a key with no work row
    bad = recs[:5].copy()
    bad["app_id"][:2] = spec.n_apps
    bad["app_id"][2] = 0xFFFFFFFF
    bad["phase"][3:] = spec.n_phases
    orphan = recs[:1].copy()
    orphan["op_id"], orphan["shape_id"], orphan["pad"] = 0xFFFF, 0xFFFFFFFF, 0xAB
    recs = np.concatenate([recs, bad, orphan])
    work = spec.work_table()
    o, ent = run_oracle(recs, spec.app_weights, spec.n_phases, work)
    groups, totals, rejected = brute_force(recs, spec.app_weights, spec.n_phases)
    assert rejected == 5 and o.stats()["n_rejected"] == 5
    assert o.stats()["n_valid"] == len(recs) - 5
    assert o.stats()["totals"] == totals
    exp = expected_entry_fields(groups, totals, work, PEAK_BW, PEAK_FLOPS)
    check_entries_against(ent, exp)
    assert list(ent["key"]) == sorted(groups)  # key ascending
    orphan_key = (int(orphan["phase"][0]) << 48) | (0xFFFF << 32) | 0xFFFFFFFF
    assert exp[orphan_key][3] == 0x7FF8000000000000
    for phase in range(spec.n_phases):
        ranked = sorted((k for k in groups if k >> 48 == phase), key=lambda k: (-groups[k][1], k))
        for k in (1, 7, len(ranked) + 3):
            top = o.topk(PEAK_BW, PEAK_FLOPS, phase, k)
            assert [int(x) for x in top["key"]] == ranked[:k]
            check = {int(e["key"]): exp[int(e["key"])] for e in top}
            check_entries_against(top, check)


def test_phase_weight_is_quotient_of_rounded_operands_and_near_exact_ratio():
    spec = make_spec(1, small=True, n=20000)
    recs = tg.generate(spec)
    o, ent = run_oracle(recs, spec.app_weights, spec.n_phases)
    totals = o.stats()["totals"]
    for e in ent[:: max(1, len(ent) // 200)]:
        wt, t = entry_wt(e), totals[int(e["key"]) >> 48]
        assert float(e["phase_weight"]) == float(wt) / float(t)
        exact = Fraction(wt, t)
        assert abs(Fraction(float(e["phase_weight"])) - exact) <= exact * Fraction(3, 2**53)


# ---------------------------------------------------------------- invariants

@pytest.mark.parametrize("index", [0, 1, 2, 3, 4])
def test_invariants(index):
    spec = make_spec(index, small=True, n=1 << 17)
    recs = tg.generate(spec)
    o, ent = run_oracle(recs, spec.app_weights, spec.n_phases, spec.work_table())
    st = o.stats()
    assert int(ent["count"].sum()) == st["n_valid"] == len(recs)
    for p in range(spec.n_phases):
        sel = ent[(ent["key"] >> np.uint64(48)) == p]
        assert sum(entry_wt(e) for e in sel) == st["totals"][p]
        s = math.fsum(sel["phase_weight"].tolist())
        assert abs(s - 1.0) <= 3 * len(sel) * 2.0**-53          # Eq. 3: weights sum to 1
    # independent total: sum of weight*duration over all records, per phase
    w = spec.app_weights.astype(object)
    for p in range(spec.n_phases):
        m = recs["phase"] == p
        tot = int(np.sum(w[recs["app_id"][m]] * recs["duration_ns"][m].astype(object)))
        assert tot == st["totals"][p]
    # permutation invariance
    perm = np.random.default_rng(7).permutation(len(recs))
    _, ent_p = run_oracle(recs[perm], spec.app_weights, spec.n_phases, spec.work_table())
    assert ent_p.tobytes() == ent.tobytes()
    # chunked == whole, threaded == single
    o2 = oracle.Oracle(spec.app_weights, spec.n_phases)
    o2.set_work(spec.work_table())
    for c in np.array_split(recs, 8):
        o2.ingest(c)
    assert o2.finalize(PEAK_BW, PEAK_FLOPS).tobytes() == ent.tobytes()
    _, ent_t = run_oracle(recs, spec.app_weights, spec.n_phases, spec.work_table(), threads=4)
    assert ent_t.tobytes() == ent.tobytes()


def test_unit_weights_reduce_to_a_library_group_sum():
    # with every weight 1, wt is a plain per-key sum of durations: numpy sort + reduceat
    spec = make_spec(0)
    recs = tg.generate(spec)
    _, ent = run_oracle(recs, np.ones(spec.n_apps, dtype=np.uint32), spec.n_phases)
    key = (recs["phase"].astype(np.uint64) << np.uint64(48)) | (recs["op_id"].astype(np.uint64) << np.uint64(32)) \
        | recs["shape_id"].astype(np.uint64)
    order = np.argsort(key, kind="stable")
    ks, first, counts = np.unique(key[order], return_index=True, return_counts=True)
    sums = np.add.reduceat(recs["duration_ns"][order].astype(np.uint64), first)
    assert np.array_equal(ent["key"], ks)
    assert np.array_equal(ent["count"], counts.astype(np.uint64))
    assert np.array_equal(ent["wt_lo"], sums) and not ent["wt_hi"].any()


def test_skew_config_closed_form():
    spec = make_spec(4, small=True, n=1 << 18)
    recs = tg.generate(spec)
    _, ent = run_oracle(recs, spec.app_weights, spec.n_phases)
    P = (2**20 - 1) * (2**28 - 1)
    for e in ent:
        assert entry_wt(e) == int(e["count"]) * P
    hot = ent[ent["key"] == ((1 << 48) | 0)]
    assert len(hot) == 1 and int(hot[0]["count"]) > 65537 and int(hot[0]["wt_hi"]) >= 1


# ---------------------------------------------------------------- edge cases

def test_edge_cases():
    o = oracle.Oracle([5], 2)
    assert len(o.finalize(PEAK_BW, PEAK_FLOPS)) == 0 and o.stats()["n_keys"] == 0
    # zero weight and zero durations: counts accumulate, totals stay 0, weight is +0.0
    o = oracle.Oracle([0, 7], 2)
    recs = records_from_dicts([{"app": 0, "op": 1, "shape": 1, "phase": 0, "duration_ns": 99},
                               {"app": 1, "op": 1, "shape": 2, "phase": 0, "duration_ns": 0},
                               {"app": 1, "op": 1, "shape": 2, "phase": 1, "duration_ns": 4}])
    o.ingest(recs)
    ent = o.finalize(PEAK_BW, PEAK_FLOPS)
    assert [int(c) for c in ent["count"]] == [1, 1, 1]
    assert f64_bits(float(ent[0]["phase_weight"])) == 0 and f64_bits(float(ent[1]["phase_weight"])) == 0
    assert float(ent[2]["phase_weight"]) == 1.0
    assert all(f64_bits(float(x)) == 0x7FF8000000000000 for x in ent["roofline_s"])
    # key packing: the three fields must not alias
    o = oracle.Oracle([1], 8)
    recs = records_from_dicts([{"op": 0, "shape": 1, "phase": 0, "duration_ns": 1},
                               {"op": 1, "shape": 0, "phase": 0, "duration_ns": 1},
                               {"op": 0, "shape": 0, "phase": 1, "duration_ns": 1},
                               {"op": 0xFFFF, "shape": 0xFFFFFFFF, "phase": 7, "duration_ns": 1}])
    o.ingest(recs)
    assert [int(k) for k in o.finalize(PEAK_BW, PEAK_FLOPS)["key"]] == [1, 1 << 32, 1 << 48, 0x0007FFFFFFFFFFFF]
    # duplicate work rows and out-of-range dtype are refused
    w = work_from_dicts([{"op": 1, "shape": 2, "flops": 1, "bytes": 1}, {"op": 1, "shape": 2, "flops": 2, "bytes": 2}])
    assert o.set_work(w) == -1
    w = work_from_dicts([{"op": 1, "shape": 2, "dtype": 8, "flops": 1, "bytes": 1}])
    assert o.set_work(w) == -1


def test_roofline_picks_the_larger_side_per_dtype():
    # F/P for dtype 2 (4e15) vs M/beta: rows constructed so each side wins once
    w = work_from_dicts([{"op": 0, "shape": 0, "dtype": 2, "flops": 8 * 10**15, "bytes": 8 * 10**12},   # 2 s vs 1 s
                         {"op": 0, "shape": 1, "dtype": 2, "flops": 4 * 10**15, "bytes": 24 * 10**12},  # 1 s vs 3 s
                         {"op": 0, "shape": 2, "dtype": 0, "flops": 4 * 10**15, "bytes": 8 * 10**12}])  # 4 s vs 1 s
    recs = records_from_dicts([{"op": 0, "shape": s, "duration_ns": 1} for s in (0, 1, 2)])
    _, ent = run_oracle(recs, [1], 1, w)
    assert [float(x) for x in ent["roofline_s"]] == [2.0, 3.0, 4.0]


def test_filtered_and_direct_totals_agree_with_the_full_group_by():
    spec = make_spec(3, small=True, n=1 << 16)
    recs = tg.generate(spec)
    recs[:3]["app_id"] = spec.n_apps  # a few invalid ones
    o, ent = run_oracle(recs, spec.app_weights, spec.n_phases, spec.work_table())
    groups, totals, rejected = brute_force(recs, spec.app_weights, spec.n_phases)
    pick = ent["key"][:: max(1, len(ent) // 50)]
    f = oracle.Oracle(spec.app_weights, spec.n_phases)
    for c in np.array_split(recs, 3):
        f.ingest_filtered(c, pick)
    got = f.finalize(PEAK_BW, PEAK_FLOPS)
    assert list(got["key"]) == sorted(int(k) for k in pick)
    for e in got:
        assert int(e["count"]) == groups[int(e["key"])][0] and entry_wt(e) == groups[int(e["key"])][1]
    acc, valid = np.zeros(16, dtype=np.uint64), np.zeros(2, dtype=np.uint64)
    for c in np.array_split(recs, 3):
        f.direct_totals(c, acc, valid)
    assert [int(acc[2 * p]) | (int(acc[2 * p + 1]) << 64) for p in range(8)] == totals
    assert int(valid[0]) == len(recs) - 3 and int(valid[1]) == 3 == rejected


def test_slice_ingest_is_the_full_group_by_cut_along_key_classes():
    """ingest_slice against brute force: the classes partition the key space (every key of the
    brute-force result turns up in exactly one class, with its count and weighted time), the class
    of a key does not depend on which records carry it, threads and chunking do not matter, and
    finalize_given_totals reproduces the full oracle's entries bit for bit when handed the totals
    that direct_totals sums from the records."""
    spec = make_spec(1, small=True, n=1 << 16)
    recs = tg.generate(spec)
    recs[5:9]["phase"] = spec.n_phases          # invalid records must not reach any slice
    work = spec.work_table()
    _, full = run_oracle(recs, spec.app_weights, spec.n_phases, work)
    groups, totals, rejected = brute_force(recs, spec.app_weights, spec.n_phases)
    modulus = 7
    classes = oracle.slice_class(full["key"], modulus)
    assert set(int(c) for c in classes) == set(range(modulus))
    seen = {}
    for r in range(modulus):
        o = oracle.Oracle(spec.app_weights, spec.n_phases)
        o.set_work(work)
        for c, th in zip(np.array_split(recs, 3), (1, 3, 2)):
            assert o.ingest_slice(c, modulus, r, threads=th) == th
        acc, valid = np.zeros(16, dtype=np.uint64), np.zeros(2, dtype=np.uint64)
        o.direct_totals(recs, acc, valid)
        assert int(valid[1]) == rejected == 4
        got = o.finalize_given_totals(PEAK_BW, PEAK_FLOPS, totals)
        assert got.tobytes() == full[classes == r].tobytes()       # both key-ascending
        for e in got:
            k = int(e["key"])
            assert k not in seen and [int(e["count"]), entry_wt(e)] == list(groups[k])
            seen[k] = r
    assert len(seen) == len(groups)
    # a second look at the scramble itself: restated with Python integers
    def py_class(key, m):
        z = (key + 0x9E3779B97F4A7C15) & (2**64 - 1)
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & (2**64 - 1)
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & (2**64 - 1)
        return (z ^ (z >> 31)) % m
    assert [py_class(int(k), 64) for k in full["key"][:200]] == [int(c) for c in oracle.slice_class(full["key"][:200], 64)]


# ---------------------------------------------------------------- score aggregation (Eq. 4-6)

def test_score_worked_example(golden_dir):
    g = load_golden(golden_dir, "score_example.json")
    u = g["units"]
    agg, s_op, err = oracle.score_candidates([x["roofline_s"] for x in u], [x["op"] for x in u],
                                             [[x["t_cand"] for x in u]], [[x["correct"] for x in u]], g["w"])
    assert list(s_op[0]) == g["S_op"] and float(agg[0]) == g["S_agg"] and int(err[0]) == g["errors"]
    for x in u:  # the fixture's own per-unit column
        if x["S_j"] is not None:
            assert x["roofline_s"] / x["t_cand"] == x["S_j"]


def test_score_against_python_statistics():
    import statistics
    rng = np.random.default_rng(5)
    n_ops, n_units, batch = 30, 440, 6              # the paper's release: 30 operators, 440 shapes
    unit_op = np.sort(rng.integers(0, n_ops, n_units)).astype(np.uint32)
    roof = np.exp(rng.uniform(np.log(1e-6), np.log(1e-1), n_units))
    w = rng.dirichlet(np.ones(n_ops) * 0.3)
    t = roof[None, :] / rng.uniform(0.01, 1.1, (batch, n_units))     # a few land above the roof
    ok = rng.random((batch, n_units)) < 0.6
    ok[0, unit_op == 3] = False                                        # an operator with no correct shape
    t[1, 5] = float("inf")
    t[1, 6] = -1.0
    t[1, 7] = float("nan")
    ok[1, 5:8] = True
    agg, s_op, err = oracle.score_candidates(roof, unit_op, t, ok, w)
    for b in range(batch):
        exp_err, total = 0, 0.0
        for i in range(n_ops):
            vals = []
            for j in np.nonzero((unit_op == i) & ok[b])[0]:
                if not (t[b, j] > 0.0) or math.isinf(t[b, j]):
                    exp_err += 1
                    continue
                s = float(roof[j]) / float(t[b, j])
                exp_err += s > 1.0
                vals.append(s)
            s_i = statistics.median(vals) if vals else 0.0
            assert float(s_op[b, i]) == s_i, (b, i)
            total = total + float(w[i]) * s_i
        assert float(agg[b]) == total and int(err[b]) == exp_err
    assert float(s_op[0, 3]) == 0.0
    # all weights on one operator whose shapes all sit exactly on the roof: S_agg = 1
    one = np.zeros(n_ops); one[0] = 1.0
    a, _, e = oracle.score_candidates(roof, unit_op, roof[None, :].copy(), np.ones((1, n_units), bool), one)
    assert float(a[0]) == 1.0 and int(e[0]) == 0


# ---------------------------------------------------------------- literal Eq. 2-3 operator weights

def test_eq3_worked_example(golden_dir):
    g = load_golden(golden_dir, "eq3_example.json")
    recs = records_from_dicts(g["records"])
    w, wt, rej = oracle.eq3_weights(recs, g["app_weights"], g["n_ops"], g["n_phases"])
    assert list(wt) == g["wtilde"] and rej == 0
    assert list(w) == [x / 1.78125 for x in g["wtilde"]]
    w, wt, _ = oracle.eq3_weights(recs, g["app_weights"], g["n_ops"], g["n_phases"], retained=[1, 1, 0])
    assert list(w) == [0.21875 / g["retained_01_sum"], 0.75 / g["retained_01_sum"], 0.0]


def test_eq3_special_cases_and_python_restatement():
    spec = make_spec(1, small=True, n=30_000)
    recs = tg.generate(spec)
    recs["op_id"][:4] = 999                           # operators outside the table are rejected
    n_ops = spec.n_ops
    # one application, one phase: the weight is the plain share of observed time (a library group-sum)
    one = recs.copy()
    one["app_id"], one["phase"] = 0, 0
    w, wt, rej = oracle.eq3_weights(one, [7], n_ops, 1)
    valid = one[one["op_id"] < n_ops]
    share = np.bincount(valid["op_id"], weights=None, minlength=n_ops) * 0
    sums = np.zeros(n_ops, dtype=np.uint64)
    np.add.at(sums, valid["op_id"], valid["duration_ns"].astype(np.uint64))
    total = int(sums.sum())
    assert rej == 4 and [float(x) for x in wt] == [float(int(s)) / float(total) * 1.0 for s in sums]
    assert abs(float(w.sum()) - 1.0) < n_ops * 2.0**-52
    # general case against a Python restatement with the same operation order
    w, wt, rej = oracle.eq3_weights(recs, spec.app_weights, n_ops, spec.n_phases)
    D, Da = {}, {}
    for a, o, p, d in zip(recs["app_id"].tolist(), recs["op_id"].tolist(), recs["phase"].tolist(), recs["duration_ns"].tolist()):
        if o >= n_ops:
            continue
        D[(o, a, p)] = D.get((o, a, p), 0) + d
        Da[(a, p)] = Da.get((a, p), 0) + d
    c_total = int(spec.app_weights.astype(np.uint64).sum())
    exp = []
    for i in range(n_ops):
        phi = [p for p in range(spec.n_phases) if any(D.get((i, a, p), 0) for a in range(spec.n_apps))]
        acc = 0.0
        for a in range(spec.n_apps):
            inner = 0.0
            for p in phi:
                if Da.get((a, p), 0):
                    inner = inner + float(D.get((i, a, p), 0)) / float(Da[(a, p)])
            acc = acc + (float(int(spec.app_weights[a])) / float(c_total)) * (inner / float(len(phi))) if phi else acc
        exp.append(acc)
    assert [float(x) for x in wt] == exp
    tot = 0.0
    for x in exp:
        tot = tot + x
    assert [float(x) for x in w] == [x / tot for x in exp]
    assert abs(float(w.sum()) - 1.0) < n_ops * 2.0**-52               # Eq. 3: the weights sum to 1
    # equal trace windows: if every application's phase total is the same, Eq. 3 reduces to the
    # card-hour-weighted share that the main aggregation path computes (checked to rounding)
    eq = recs[recs["op_id"] < n_ops].copy()
    eq["phase"] = 0
    eq["app_id"] = np.arange(len(eq)) % 2
    eq["duration_ns"] = 1000
    if (eq["app_id"] == 0).sum() != (eq["app_id"] == 1).sum():
        eq = eq[:-1]
    w2, _, _ = oracle.eq3_weights(eq, [1, 3], n_ops, 1)
    num = np.zeros(n_ops)
    np.add.at(num, eq["op_id"], np.where(eq["app_id"] == 0, 1.0, 3.0) * 1000.0)
    assert np.allclose(w2, num / num.sum(), rtol=1e-12, atol=0)


# ---------------------------------------------------------------- ranked list, running share, coverage cut

def _entries_from(keys, wts, counts=None):
    e = np.zeros(len(keys), dtype=oracle.ENTRY_DTYPE)
    e["key"] = np.asarray(keys, dtype=np.uint64)
    e["wt_lo"] = np.asarray([w & (2**64 - 1) for w in wts], dtype=np.uint64)
    e["wt_hi"] = np.asarray([w >> 64 for w in wts], dtype=np.uint64)
    e["count"] = np.arange(1, len(keys) + 1, dtype=np.uint64) if counts is None else counts
    return e


def test_rank_worked_example(golden_dir):
    g = load_golden(golden_dir, "rank_example.json")
    keys = [(r["phase"] << 48) | (r["key_op"] << 32) | r["key_shape"] for r in g["entries"]]
    e = _entries_from(keys, [int(r["wt"]) for r in g["entries"]])
    ranked, cum, res = oracle.rank_phase(e, g["phase"], 0)
    assert [[int(k >> 32) & 0xFFFF, int(k) & 0xFFFFFFFF] for k in ranked["key"]] == g["ranked_ops_shapes"]
    assert list(cum) == g["cum"] and res["n_phase"] == 5 and res["total"] == int(g["total"])
    assert [entry_wt(x) for x in ranked] == sorted([int(r["wt"]) for r in g["entries"] if r["phase"] == 1], reverse=True)
    for c in g["cuts"]:
        _, _, res = oracle.rank_phase(e, g["phase"], c["coverage_ppm"])
        assert res["n_keep"] == c["n_keep"] and res["covered"] == int(c["covered"]), c
    # a truncated output reports the same cut
    ranked2, cum2, res = oracle.rank_phase(e, g["phase"], 875001, out_cap=2)
    assert len(ranked2) == 2 and list(cum2) == g["cum"][:2] and res["n_keep"] == 4 and res["n_phase"] == 5
    # a phase that has no units
    ranked3, _, res = oracle.rank_phase(e, 5, 500000)
    assert len(ranked3) == 0 and res == {"n_phase": 0, "n_keep": 0, "total": 0, "covered": 0}


def test_rank_reproduces_the_printed_cumulative_column(golden_dir):
    g = load_golden(golden_dir, "table2_cumulative.json")
    wts = [10 * s for s in g["score_milli"]] + [10 * g["tail_score_milli"] // g["tail_operators"]] * g["tail_operators"]
    assert sum(wts[10:]) == 10 * g["tail_score_milli"]
    # keys in an order unrelated to the weights; the two pairs of equal printed scores get keys that
    # make the expected order unambiguous
    rng = random.Random(5)
    order = list(range(len(wts)))
    rng.shuffle(order)
    keys = [0] * len(wts)
    for rank, pos in enumerate(order):
        keys[rank] = (rank % 7 << 32) | (1000 + pos)
    shuffled = list(range(len(wts)))
    rng.shuffle(shuffled)
    e = _entries_from([keys[i] for i in shuffled], [wts[i] for i in shuffled])
    ranked, cum, res = oracle.rank_phase(e, 0, 0)
    assert [entry_wt(x) for x in ranked[:10]] == wts[:10]
    for i, printed in enumerate(g["cum_printed"]):
        assert abs(cum[i] - printed) <= (i + 1) * 0.0005 + 0.0005 + 0.001, (i, cum[i], printed)
    assert cum[-1] == g["tail_cum_printed"] and res["n_phase"] == 30
    for c in g["cuts"]:
        assert oracle.rank_phase(e, 0, c["coverage_ppm"])[2]["n_keep"] == c["n_keep"], c


def test_rank_against_python_integers_and_the_ranked_topk():
    spec = make_spec(1, small=True, n=40_000)
    recs = tg.generate(spec)
    o, entries = run_oracle(recs, spec.app_weights, spec.n_phases)
    rng = np.random.default_rng(3)
    entries = entries[rng.permutation(entries.shape[0])]
    for phase in range(spec.n_phases):
        mine = [x for x in entries if int(x["key"]) >> 48 == phase]
        py = sorted(mine, key=lambda x: (-entry_wt(x), int(x["key"])))
        total = sum(entry_wt(x) for x in py)
        for ppm in (0, 1, 333_333, 800_000, 999_999, 1_000_000):
            ranked, cum, res = oracle.rank_phase(entries, phase, ppm)
            assert [int(k) for k in ranked["key"]] == [int(x["key"]) for x in py]
            assert res["total"] == total and res["n_phase"] == len(py)
            prefix, acc = [], 0
            for x in py:
                acc += entry_wt(x)
                prefix.append(acc)
            assert [f64_bits(c) for c in cum] == [f64_bits(float(p) / float(total)) for p in prefix]
            k = res["n_keep"]
            before = prefix[k - 1] if k else 0
            assert before * 1_000_000 >= ppm * total and res["covered"] == before
            assert k == 0 or (prefix[k - 2] if k > 1 else 0) * 1_000_000 < ppm * total     # minimal
            assert all(cum[i] <= cum[i + 1] for i in range(len(cum) - 1)) and cum[-1] == 1.0
        # the head of the ranking is the ranked top-k (an independently pinned function)
        top = o.topk(PEAK_BW, PEAK_FLOPS, phase, 25)
        ranked, _, _ = oracle.rank_phase(entries, phase, 0, out_cap=25)
        assert ranked.tobytes() == top.tobytes()
    # all-zero weights: shares +0.0, nothing kept
    z = entries.copy()
    z["wt_lo"] = 0
    z["wt_hi"] = 0
    ranked, cum, res = oracle.rank_phase(z, 0, 900_000)
    assert res["n_keep"] == 0 and res["total"] == 0 and not cum.any() and not np.signbit(cum).any()
    assert [int(k) for k in ranked["key"]] == sorted(int(k) for k in z["key"] if int(k) >> 48 == 0)


def test_sort_by_key_is_a_library_sort():
    spec = make_spec(2, small=True, n=20_000)
    _, entries = run_oracle(tg.generate(spec), spec.app_weights, spec.n_phases)
    rng = np.random.default_rng(11)
    shuffled = entries[rng.permutation(entries.shape[0])]
    got = oracle.sort_by_key(shuffled)
    assert got.tobytes() == shuffled[np.argsort(shuffled["key"], kind="stable")].tobytes()
    assert got.tobytes() == entries.tobytes()          # finalize already walks the keys in order
    assert oracle.sort_by_key(entries[:0]).shape[0] == 0
