"""Parity of the CUDA path (through the C ABI) against the CPU oracle: bit-exact on every
field, on the same seeded inputs, for the five benchmark laws at sizes the oracle finishes
in seconds (several CTA tiles plus a ragged tail), and on the edge cases."""
import ctypes as C

import numpy as np
import pytest

import oracle
import tracegen as tg
from tracegen.configs import make_spec
from tracegen.layout import RECORD_DTYPE, WORK_DTYPE
from tests.helpers import (load_golden, f64_bits, records_from_dicts, work_from_dicts, entry_wt, sorted_by_key)

pytestmark = pytest.mark.gpu

PEAK_BW = 8.0e12
PEAK_FLOPS = [1.0e15, 2.0e15, 4.0e15, 5.0e14, 2.5e14, 1.0e15, 1.0e15, 1.0e15]


@pytest.fixture(scope="module")
def lib():
    import paper_2607_14541_b200 as p
    return p


def to_dev(recs: np.ndarray, misalign: bool = False):
    import torch
    raw = torch.from_numpy(np.ascontiguousarray(recs).view(np.uint8).reshape(-1))
    if misalign:  # 16-byte aligned but not 32-byte aligned start
        buf = torch.empty(raw.numel() + 64, dtype=torch.uint8, device="cuda:0")
        off = 16 if buf.data_ptr() % 32 == 0 else 0
        view = buf[off: off + raw.numel()]
        view.copy_(raw)
        assert view.data_ptr() % 32 == 16
        return view
    return raw.cuda()


def gpu_aggregate(lib, recs, app_weights, n_phases, work=None, max_keys=None, chunks=1, flags=0, misalign=False,
                  host=False):
    n_keys_bound = max_keys or max(len(recs), 16)
    agg = lib.Aggregator(app_weights, n_phases, n_keys_bound, max_work_rows=0 if work is None else len(work), flags=flags)
    if work is not None:
        agg.set_work_table(work)
    for c in np.array_split(recs, chunks):
        if host:
            agg.ingest_host(c)
        else:
            agg.ingest(to_dev(c, misalign), n=len(c))
    return agg


def assert_same_as_oracle(agg, o, n_phases, ks=(1, 10)):
    got = sorted_by_key(agg.finalize_numpy(PEAK_BW, PEAK_FLOPS))
    exp = o.finalize(PEAK_BW, PEAK_FLOPS)
    assert len(got) == len(exp)
    assert got.tobytes() == exp.tobytes()          # every field, bit for bit
    st, so = agg.stats(), o.stats()
    assert st["n_valid"] == so["n_valid"] and st["n_rejected"] == so["n_rejected"] and st["n_keys"] == so["n_keys"]
    assert st["totals"] == so["totals"] and st["n_dropped"] == 0
    for phase in range(n_phases):
        for k in ks:
            assert agg.topk(phase, k).tobytes() == o.topk(PEAK_BW, PEAK_FLOPS, phase, k).tobytes(), (phase, k)
    return got


def oracle_of(recs, app_weights, n_phases, work=None, threads=4):
    o = oracle.Oracle(app_weights, n_phases)
    if work is not None:
        assert o.set_work(work) == 0
    o.ingest(recs, threads=threads)
    return o


# ---------------------------------------------------------------- the five laws

CASES = [
    # index, small key domain, n (odd sizes leave a ragged tail), chunks
    (0, False, 1 << 20, 1),
    (1, False, (1 << 22) + 12345, 1),
    (2, True, (1 << 22) + 1, 1),
    (3, True, (1 << 23) + 777, 8),
    (4, True, (1 << 22) + 3, 1),
]


@pytest.mark.parametrize("index,small,n,chunks", CASES)
def test_parity_five_configs(lib, index, small, n, chunks):
    spec = make_spec(index, small=small, n=n, n_dtypes=3)
    recs = tg.generate(spec)
    work = spec.work_table()
    o = oracle_of(recs, spec.app_weights, spec.n_phases, work)
    agg = gpu_aggregate(lib, recs, spec.app_weights, spec.n_phases, work, max_keys=spec.max_keys, chunks=chunks)
    got = assert_same_as_oracle(agg, o, spec.n_phases, ks=(1, spec.topk, 4096))
    assert agg.stats()["hot_slots"] > 0            # the shared-memory stage was active
    if index == 4:  # the u128 carry path was exercised
        assert int(got["wt_hi"].max()) >= 1
    if chunks > 1:  # chunked == single pass
        agg1 = gpu_aggregate(lib, recs, spec.app_weights, spec.n_phases, work, max_keys=spec.max_keys, chunks=1)
        assert sorted_by_key(agg1.finalize_numpy(PEAK_BW, PEAK_FLOPS)).tobytes() == got.tobytes()


@pytest.mark.parametrize("index", [1, 4])
def test_parity_without_hot_directory_and_misaligned_start(lib, index):
    spec = make_spec(index, small=True, n=(1 << 20) + 5)
    recs = tg.generate(spec)
    o = oracle_of(recs, spec.app_weights, spec.n_phases)
    agg = gpu_aggregate(lib, recs, spec.app_weights, spec.n_phases, max_keys=spec.max_keys,
                        flags=lib.ATREX_FLAG_NO_HOT_DIRECTORY)
    assert_same_as_oracle(agg, o, spec.n_phases)
    assert agg.stats()["hot_slots"] == 0
    agg = gpu_aggregate(lib, recs, spec.app_weights, spec.n_phases, max_keys=spec.max_keys, misalign=True, chunks=3)
    assert_same_as_oracle(agg, o, spec.n_phases)


def test_host_ingest_equals_device_ingest(lib):
    spec = make_spec(1, small=True, n=(1 << 23) + 9)   # > one 64 MiB staging piece
    recs = tg.generate(spec)
    o = oracle_of(recs, spec.app_weights, spec.n_phases)
    agg = gpu_aggregate(lib, recs, spec.app_weights, spec.n_phases, max_keys=spec.max_keys, host=True)
    assert_same_as_oracle(agg, o, spec.n_phases)


def test_permutation_and_many_small_calls(lib):
    spec = make_spec(3, small=True, n=200_001)
    recs = tg.generate(spec)
    o = oracle_of(recs, spec.app_weights, spec.n_phases)
    perm = np.random.default_rng(3).permutation(len(recs))
    agg = gpu_aggregate(lib, recs[perm], spec.app_weights, spec.n_phases, max_keys=spec.max_keys, chunks=37)
    assert_same_as_oracle(agg, o, spec.n_phases)


def test_merge_of_partial_aggregates_equals_whole(lib):
    import torch
    spec = make_spec(2, small=True, n=1 << 20)
    recs = tg.generate(spec)
    o = oracle_of(recs, spec.app_weights, spec.n_phases)
    a = gpu_aggregate(lib, recs[: 400_000], spec.app_weights, spec.n_phases, max_keys=spec.max_keys)
    b = gpu_aggregate(lib, recs[400_000:], spec.app_weights, spec.n_phases, max_keys=spec.max_keys)
    part, n = b.finalize(PEAK_BW, PEAK_FLOPS)
    a.merge(part, n)
    assert_same_as_oracle(a, o, spec.n_phases)


# ---------------------------------------------------------------- hand-computed traces on the GPU

def test_worked_example_a_on_gpu(lib, golden_dir):
    g = load_golden(golden_dir, "worked_example_a.json")
    recs, work = records_from_dicts(g["records"]), work_from_dicts(g["work"])
    agg = lib.Aggregator(g["app_weights"], g["n_phases"], 64, max_work_rows=8)
    agg.set_work_table(work)
    agg.ingest(to_dev(recs), n=len(recs))
    ent = sorted_by_key(agg.finalize_numpy(g["peak_bw"], g["peak_flops"] + [1.0] * 7))
    assert len(ent) == 4
    for e, x in zip(ent, g["expected"]):
        assert int(e["key"]) == int(x["key"], 16) and int(e["count"]) == x["count"] and entry_wt(e) == x["wt"]
        assert f64_bits(float(e["phase_weight"])) == int(x["phase_weight_bits"], 16)
        assert f64_bits(float(e["roofline_s"])) == int(x["roofline_bits"], 16)
    for t in g["topk"]:
        assert [int(k) for k in agg.topk(t["phase"], t["k"])["key"]] == [int(k, 16) for k in t["keys"]]


def test_carry_closed_form_on_gpu(lib, golden_dir):
    g = load_golden(golden_dir, "carry_closed_form.json")
    for case in g["cases"]:
        n = case["N"]
        recs = np.zeros(n, dtype=RECORD_DTYPE)
        recs["op_id"], recs["shape_id"], recs["phase"], recs["duration_ns"] = 3, 11, 1, g["duration_ns"]
        for flags in (0, lib.ATREX_FLAG_NO_HOT_DIRECTORY):
            agg = lib.Aggregator([g["weight"]], 2, 16, flags=flags)
            agg.ingest(to_dev(recs), n=n)
            ent = agg.finalize_numpy(PEAK_BW, PEAK_FLOPS)
            assert len(ent) == 1 and int(ent[0]["count"]) == n
            assert int(ent[0]["wt_hi"]) == case["wt_hi"] and int(ent[0]["wt_lo"]) == int(case["wt_lo"], 16)
            assert float(ent[0]["phase_weight"]) == 1.0


def test_topk_ties_on_gpu(lib, golden_dir):
    g = load_golden(golden_dir, "topk_ties.json")
    c = g["case_rounding"]
    rows = []
    for name in ("x", "y"):
        k = c[name]
        rows += [{"app": 0, "op": k["op"], "shape": k["shape"], "duration_ns": k["big_duration"]}] * k["n_big"]
        if "extra_duration" in k:
            rows.append({"app": 1, "op": k["op"], "shape": k["shape"], "duration_ns": k["extra_duration"]})
    recs = records_from_dicts(rows)
    agg = lib.Aggregator(c["app_weights"], 1, 16)
    agg.ingest(to_dev(recs), n=len(recs))
    agg.finalize(PEAK_BW, PEAK_FLOPS)
    assert [int(k) for k in agg.topk(0, 2)["key"]] == [int(k, 16) for k in c["top2_keys"]]
    t = g["case_exact_ties"]
    recs = records_from_dicts(t["records"])
    agg = lib.Aggregator(t["app_weights"], 1, 16)
    agg.ingest(to_dev(recs), n=len(recs))
    agg.finalize(PEAK_BW, PEAK_FLOPS)
    assert [int(k) for k in agg.topk(0, 3)["key"]] == [int(k, 16) for k in t["top3_keys"]]
    assert [int(k) for k in agg.topk(0, 9)["key"]] == [int(k, 16) for k in t["top4_keys"]]


def test_topk_with_a_huge_tie_class_needs_deeper_digits(lib):
    # 150k keys with identical weighted time: the candidate class exceeds the sorter's
    # capacity until the radix select reaches the key digits
    n = 150_000
    recs = np.zeros(n, dtype=RECORD_DTYPE)
    recs["op_id"] = np.arange(n) % 50
    recs["shape_id"] = np.arange(n) // 50 + 17
    recs["duration_ns"] = 5000
    recs = np.concatenate([recs, recs[:3]])          # three keys get twice the weight
    o = oracle_of(recs, [9], 1)
    agg = lib.Aggregator([9], 1, 1 << 18)
    agg.ingest(to_dev(recs), n=len(recs))
    agg.finalize(PEAK_BW, PEAK_FLOPS)
    for k in (1, 3, 4, 100, 70_000 if False else 65_536):
        assert agg.topk(0, k).tobytes() == o.topk(PEAK_BW, PEAK_FLOPS, 0, k).tobytes(), k


# ---------------------------------------------------------------- edge cases and errors

def test_empty_single_and_invalid_records(lib):
    agg = lib.Aggregator([3, 5], 2, 64)
    assert len(agg.finalize_numpy(PEAK_BW, PEAK_FLOPS)) == 0
    assert len(agg.topk(0, 5)) == 0
    import torch
    agg.ingest(torch.empty(0, dtype=torch.uint8, device="cuda:0"), n=0)
    recs = records_from_dicts([{"app": 1, "op": 2, "shape": 3, "phase": 1, "duration_ns": 10}])
    agg.ingest(to_dev(recs), n=1)
    ent = agg.finalize_numpy(PEAK_BW, PEAK_FLOPS)
    assert len(ent) == 1 and int(ent[0]["key"]) == (1 << 48) | (2 << 32) | 3 and entry_wt(ent[0]) == 50
    assert f64_bits(float(ent[0]["roofline_s"])) == 0x7FF8000000000000
    bad = records_from_dicts([{"app": 2, "op": 1, "shape": 1, "duration_ns": 1},
                              {"app": 0xFFFFFFFF, "op": 1, "shape": 1, "duration_ns": 1},
                              {"app": 0, "op": 1, "shape": 1, "phase": 2, "duration_ns": 1},
                              {"app": 0, "op": 1, "shape": 1, "phase": 255, "duration_ns": 1}])
    bad["pad"] = 0x5A
    agg.ingest(to_dev(bad), n=4)
    st = agg.stats()
    assert st["n_rejected"] == 4 and st["n_valid"] == 1 and st["n_keys"] == 1
    # zero weight / zero duration: counted, total stays zero, weight +0.0
    agg = lib.Aggregator([0, 7], 2, 64)
    z = records_from_dicts([{"app": 0, "op": 1, "shape": 1, "duration_ns": 99},
                            {"app": 1, "op": 1, "shape": 2, "duration_ns": 0}])
    agg.ingest(to_dev(z), n=2)
    ent = sorted_by_key(agg.finalize_numpy(PEAK_BW, PEAK_FLOPS))
    assert [int(c) for c in ent["count"]] == [1, 1] and all(f64_bits(float(x)) == 0 for x in ent["phase_weight"])


def test_finalize_is_repeatable_and_peaks_only_change_the_roofline(lib):
    spec = make_spec(0, n=100_000, n_dtypes=3)
    recs, work = tg.generate(spec), spec.work_table()
    agg = gpu_aggregate(lib, recs[:50_000], spec.app_weights, spec.n_phases, work, max_keys=spec.max_keys)
    first = sorted_by_key(agg.finalize_numpy(PEAK_BW, PEAK_FLOPS))
    again = sorted_by_key(agg.finalize_numpy(PEAK_BW, PEAK_FLOPS))
    assert first.tobytes() == again.tobytes()
    other = sorted_by_key(agg.finalize_numpy(2 * PEAK_BW, [2 * x for x in PEAK_FLOPS]))
    assert np.array_equal(other["phase_weight"], first["phase_weight"])
    assert np.array_equal(other["roofline_s"], first["roofline_s"] / 2)
    agg.ingest(to_dev(recs[50_000:]), n=50_000)       # refresh: keep ingesting after a finalize
    o = oracle_of(recs, spec.app_weights, spec.n_phases, work)
    assert_same_as_oracle(agg, o, spec.n_phases)
    agg.reset()
    assert len(agg.finalize_numpy(PEAK_BW, PEAK_FLOPS)) == 0 and agg.stats()["n_rejected"] == 0
    agg.ingest(to_dev(recs), n=len(recs))
    assert_same_as_oracle(agg, o, spec.n_phases)


def test_error_codes(lib):
    import torch
    p = lib
    # capacity: far more distinct keys than provisioned -> ATREX_ERR_CAPACITY, no hang
    n = 60_000
    recs = np.zeros(n, dtype=RECORD_DTYPE)
    recs["shape_id"] = np.arange(n)
    recs["duration_ns"] = 1
    agg = p.Aggregator([1], 1, 8)
    agg.ingest(to_dev(recs), n=n)
    with pytest.raises(p.AtrexError) as ei:
        agg.finalize(PEAK_BW, PEAK_FLOPS)
    assert ei.value.status == p.ATREX_ERR_CAPACITY
    st = agg.stats(check=False)
    assert st["status"] == p.ATREX_ERR_CAPACITY and st["n_dropped"] > 0
    assert st["n_dropped"] + st["n_valid"] == n
    # output buffer too small
    agg = p.Aggregator([1], 1, 1 << 17)
    agg.ingest(to_dev(recs), n=n)
    small = torch.empty(48 * 10, dtype=torch.uint8, device="cuda:0")
    pk = p.make_peaks(PEAK_BW, PEAK_FLOPS)
    n_out = C.c_uint64(0)
    rc = p.atrex_agg_finalize(agg._h, C.byref(pk), small.data_ptr(), 10, C.byref(n_out), None)
    assert rc == p.ATREX_ERR_OUT_TOO_SMALL and n_out.value == n
    # invalid arguments
    assert p.atrex_agg_ingest(agg._h, small.data_ptr() + 8, 1, None) == p.ATREX_ERR_INVALID
    assert p.atrex_agg_ingest(agg._h, None, 1, None) == p.ATREX_ERR_INVALID
    bad = p.make_peaks(0.0, PEAK_FLOPS)
    assert p.atrex_agg_finalize(agg._h, C.byref(bad), None, 0, C.byref(n_out), None) == p.ATREX_ERR_INVALID
    bad = p.make_peaks(PEAK_BW, [float("nan")] * 8)
    assert p.atrex_agg_finalize(agg._h, C.byref(bad), None, 0, C.byref(n_out), None) == p.ATREX_ERR_INVALID
    out = np.zeros(4, dtype=p.ENTRY_DTYPE)
    k_out = C.c_uint32(0)
    assert p.atrex_agg_topk(agg._h, 5, 1, out.ctypes.data, C.byref(k_out), None) == p.ATREX_ERR_INVALID
    agg.ingest(to_dev(recs[:10]), n=10)
    assert p.atrex_agg_topk(agg._h, 0, 1, out.ctypes.data, C.byref(k_out), None) == p.ATREX_ERR_STATE
    cfg = p.atrex_agg_config_t()
    cfg.n_apps, cfg.n_phases, cfg.max_keys = 1, 9, 8
    h = C.c_void_p()
    w = np.array([1], dtype=np.uint32)
    cfg.app_weights = w.ctypes.data
    assert p.atrex_agg_create(C.byref(cfg), C.byref(h)) == p.ATREX_ERR_INVALID
    # duplicate work rows / bad dtype
    agg = p.Aggregator([1], 1, 16, max_work_rows=4)
    dup = work_from_dicts([{"op": 1, "shape": 2, "flops": 1, "bytes": 1}, {"op": 1, "shape": 2, "flops": 2, "bytes": 2}])
    assert p.atrex_agg_set_work_table(agg._h, dup.ctypes.data, 2, None) == p.ATREX_ERR_INVALID
    bad_dt = work_from_dicts([{"op": 1, "shape": 2, "dtype": 8, "flops": 1, "bytes": 1}])
    assert p.atrex_agg_set_work_table(agg._h, bad_dt.ctypes.data, 1, None) == p.ATREX_ERR_INVALID
    assert p.atrex_agg_set_work_table(agg._h, dup.ctypes.data, 5, None) == p.ATREX_ERR_INVALID


def test_gpu_sampler_matches_numpy_sampler():
    import torch
    from tracegen.gpu import GpuSampler
    for index in range(5):
        spec = make_spec(index, small=True, n=300_001)
        ref = tg.generate(spec, start=1000, count=200_001)
        out = torch.empty(200_001 * 16, dtype=torch.uint8, device="cuda:0")
        GpuSampler(spec).fill(out, start=1000, count=200_001)
        torch.cuda.synchronize()
        assert out.cpu().numpy().tobytes() == ref.tobytes(), index


def test_full_u32_range_of_weights_and_durations(lib):
    # products up to (2^32-1)^2 do not fit the 48-bit fast path; they must still be exact
    rng = np.random.default_rng(11)
    n = 300_000
    recs = np.zeros(n, dtype=RECORD_DTYPE)
    recs["app_id"] = rng.integers(0, 4, n)
    recs["op_id"] = rng.integers(0, 3, n)
    recs["shape_id"] = rng.integers(0, 50, n)
    recs["phase"] = rng.integers(0, 2, n)
    recs["duration_ns"] = rng.choice(np.array([0, 1, 70_000, 0x0FFFFFFF, 0x10000000, 0xFFFFFFFF], dtype=np.uint32), n)
    weights = np.array([0xFFFFFFFF, 1, 0x00100000, 0x000FFFFF], dtype=np.uint32)
    o = oracle_of(recs, weights, 2)
    for flags in (0, lib.ATREX_FLAG_NO_HOT_DIRECTORY):
        agg = gpu_aggregate(lib, recs, weights, 2, max_keys=1000, flags=flags, chunks=2)
        got = assert_same_as_oracle(agg, o, 2)
        assert int(got["wt_hi"].max()) > 0


def test_many_apps_eight_phases_and_largest_geometry(lib):
    # > 4096 applications (weights read from global memory), 8 phases, and the largest table
    # geometry (4096 partitions)
    spec = make_spec(1, small=True, n=400_003)
    recs = tg.generate(spec)
    rng = np.random.default_rng(3)
    recs["app_id"] = rng.integers(0, 5000, len(recs))
    recs["phase"] = rng.integers(0, 8, len(recs))
    weights = rng.integers(1, 1 << 20, 5000).astype(np.uint32)
    o = oracle_of(recs, weights, 8)
    agg = gpu_aggregate(lib, recs, weights, 8, max_keys=1 << 25)
    assert_same_as_oracle(agg, o, 8, ks=(3,))
    assert agg.stats()["table_slots"] >= 4096 * 11000


def test_topk_requests_in_any_order_and_after_more_records(lib):
    """The ranking keeps what it worked out for all phases until the next finalize: answers must not
    depend on the order of (phase, k) requests, and must follow the table after more records arrive."""
    spec = make_spec(2, small=True, n=600_000)                  # three phases
    recs = tg.generate(spec)
    first, second = recs[:350_000], recs[350_000:]
    agg = gpu_aggregate(lib, first, spec.app_weights, spec.n_phases, max_keys=spec.max_keys)
    o = oracle_of(first, spec.app_weights, spec.n_phases)
    agg.finalize(PEAK_BW, PEAK_FLOPS)
    for phase, k in ((2, 10), (0, 10), (1, 10), (1, 3), (0, 500), (2, 500), (1, 1), (0, 10), (2, 4096)):
        assert agg.topk(phase, k).tobytes() == o.topk(PEAK_BW, PEAK_FLOPS, phase, k).tobytes(), (phase, k)
    agg.ingest(to_dev(second), n=len(second))
    with pytest.raises(lib.AtrexError):
        agg.topk(0, 10)                                          # stale until the next finalize
    o.ingest(second, threads=4)
    agg.finalize(PEAK_BW, PEAK_FLOPS)
    for phase, k in ((1, 10), (0, 10), (2, 10), (0, 7)):
        assert agg.topk(phase, k).tobytes() == o.topk(PEAK_BW, PEAK_FLOPS, phase, k).tobytes(), (phase, k)
    agg.finalize(PEAK_BW, [2 * x for x in PEAK_FLOPS])          # other peaks: same ranking, other roofline times
    assert agg.topk(1, 10).tobytes() == o.topk(PEAK_BW, [2 * x for x in PEAK_FLOPS], 1, 10).tobytes()


def test_crowded_small_partitions_overflow_the_deferred_queue(lib):
    """Tiny partitions (a few hundred slots, the smallest geometry), no hot directory, about 500 K entries
    per partition in the first drain: the entries that fail the first look outnumber what the partition
    pass's per-CTA queue holds (32 K), so the in-line fallback runs as well.  Still exact."""
    rng = np.random.default_rng(77)
    n, n_keys = 1 << 27, 25_000
    k = rng.integers(0, n_keys, n, dtype=np.uint32)
    recs = np.zeros(n, dtype=RECORD_DTYPE)
    recs["app_id"] = rng.integers(0, 16, n, dtype=np.uint32)
    recs["op_id"] = (k % 50).astype(np.uint16)
    recs["shape_id"] = k // 50 * 7919
    recs["phase"] = (k % 2).astype(np.uint8)
    recs["duration_ns"] = rng.integers(1, 1 << 28, n, dtype=np.uint32)
    weights = rng.integers(1, 1 << 20, 16, dtype=np.uint32)
    agg = gpu_aggregate(lib, recs, weights, 2, max_keys=n_keys, chunks=1, flags=lib.ATREX_FLAG_NO_HOT_DIRECTORY)
    st = agg.stats()
    assert st["table_slots"] <= 256 * 256 and st["n_spilled"] == n and st["n_overflow"] == 0
    o = oracle_of(recs, weights, 2, threads=16)
    assert_same_as_oracle(agg, o, 2)


@pytest.mark.parametrize("max_keys", [23_000, 25_000, 31_500, 50_000])
def test_table_filled_exactly_to_max_keys(lib, max_keys):
    """A caller who stays within max_keys must never see ATREX_ERR_CAPACITY: a key can only live in
    its hash partition, so partitions are sized for the tail of their load.  These sizes sit where a
    flat 1.3 slots per key left the fullest partition of a random key set short in a third of the
    cases; both phases of every (operator, shape) are present, which widens the spread further."""
    rng = np.random.default_rng(max_keys)
    pairs = np.unique(rng.integers(0, 1 << 40, size=max_keys, dtype=np.uint64))[: max_keys // 2]
    recs = np.zeros(2 * len(pairs) * 2, dtype=RECORD_DTYPE)          # every key twice
    recs["op_id"] = np.tile((pairs >> np.uint64(24)).astype(np.uint16), 4)
    recs["shape_id"] = np.tile((pairs & np.uint64(0xFFFFFF)).astype(np.uint32) * np.uint32(2654435761), 4)
    recs["phase"] = np.repeat(np.array([0, 1, 0, 1], dtype=np.uint8), len(pairs))
    recs["app_id"] = rng.integers(0, 4, size=len(recs))
    recs["duration_ns"] = rng.integers(1, 1 << 28, size=len(recs))
    rng.shuffle(recs)
    weights = np.array([1, 7, 1000, (1 << 20) - 1], dtype=np.uint32)
    o = oracle_of(recs, weights, 2)
    n_keys = o.stats()["n_keys"]
    assert n_keys == 2 * len(pairs) and max_keys - 1 <= n_keys <= max_keys
    agg = gpu_aggregate(lib, recs, weights, 2, max_keys=n_keys)
    assert_same_as_oracle(agg, o, 2)


@pytest.mark.parametrize("max_keys,partitions", [(2_000_000, 256), (4_000_000, 512), (9_000_000, 1024), (18_000_000, 2048),
                                                 (1 << 25, 4096)])
@pytest.mark.parametrize("hot", [True, False])
def test_every_partition_count_with_full_range_keys(lib, max_keys, partitions, hot):
    """A spill entry carries (phase, operator, hash bits below the partition's) instead of the key, and
    the partition pass recovers a new key's shape by inverting the hash: every partition count the
    library can choose (2^8 .. 2^12, i.e. 24 .. 20 stored hash bits), operators over all 16 bits, shapes
    over all 32, eight phases, and two drains, so that keys written back by the first are found again
    by the second."""
    rng = np.random.default_rng(partitions + (1 if hot else 0))
    n = 600_011
    recs = np.zeros(n, dtype=RECORD_DTYPE)
    pool_op = rng.integers(0, 1 << 16, size=200_000).astype(np.uint16)
    pool_shape = rng.integers(0, 1 << 32, size=200_000, dtype=np.uint64).astype(np.uint32)
    pool_shape[:64] = np.array([0, 1, 0xFFFFFFFF, 0x80000000] * 16, dtype=np.uint32)   # the corners too
    pick = rng.integers(0, 200_000, size=n)
    pick[: n // 4] = rng.integers(0, 500, size=n // 4)            # a few keys frequent enough for the directory
    recs["op_id"], recs["shape_id"] = pool_op[pick], pool_shape[pick]
    recs["phase"] = rng.integers(0, 8, size=n)
    recs["app_id"] = rng.integers(0, 16, size=n)
    recs["duration_ns"] = rng.integers(0, 1 << 28, size=n)
    rng.shuffle(recs)
    weights = rng.integers(1, 1 << 20, size=16).astype(np.uint32)
    o = oracle_of(recs, weights, 8)
    agg = lib.Aggregator(weights, 8, max_keys, flags=0 if hot else lib.ATREX_FLAG_NO_HOT_DIRECTORY)
    half = n // 2
    agg.ingest(to_dev(recs[:half]), n=half)
    first = agg.stats()                                            # forces the first drain
    assert first["table_slots"] % partitions == 0 and first["table_slots"] // partitions <= 11520
    assert first["table_slots"] // partitions >= 8192 or partitions == 256
    agg.ingest(to_dev(recs[half:]), n=n - half)
    assert_same_as_oracle(agg, o, 8, ks=(5,))
    st = agg.stats()
    assert st["n_spilled"] > n // 2 and st["n_drains"] >= 2 and st["n_overflow"] == 0
