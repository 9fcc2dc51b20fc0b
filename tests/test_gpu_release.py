"""GPU parity for the release artefacts: the entry list in key order and the per-phase ranking
with running share and coverage cut (the construction behind Table 2), compared bit for bit with
the CPU oracle on the same seeded inputs; plus the refresh round trip (a stored entry list folded
into a new handle before more records arrive)."""
import ctypes as C

import numpy as np
import pytest

import oracle
import tracegen as tg
from tracegen.configs import make_spec
from tests.helpers import load_golden

pytestmark = pytest.mark.gpu

PEAK_BW = 8.0e12
PEAK_FLOPS = [1.0e15, 2.0e15, 4.0e15, 5.0e14, 2.5e14, 1.0e15, 1.0e15, 1.0e15]
PPMS = (0, 1, 250_000, 800_000, 999_999, 1_000_000)


@pytest.fixture(scope="module")
def lib():
    import paper_2607_14541_b200 as p
    return p


def dev(entries: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(entries).view(np.uint8).reshape(-1)).cuda()


def host(t, dtype):
    return t.cpu().numpy().view(dtype)


def synthetic_entries(seed: int, n: int, n_phases: int, wt_kind: str) -> np.ndarray:
    """Seeded entry list with unique keys in shuffled order.  wt_kind: 'wide' = up to 88 bits,
    'ties' = a handful of distinct values, 'zero', 'narrow' = below 2^20 (many skipped digits)."""
    rng = np.random.default_rng(seed)
    e = np.zeros(n, dtype=oracle.ENTRY_DTYPE)
    body = rng.permutation(np.arange(n, dtype=np.uint64) * np.uint64(2654435761) % np.uint64(1 << 40))
    # unique (op, shape) bodies need distinct values: multiplication by an odd constant mod 2^40 is a bijection
    assert len(np.unique(body)) == n
    op = (body >> np.uint64(28)) & np.uint64(0xFFF)
    shape = (body & np.uint64(0xFFFFFFF)) | (rng.integers(0, 8, n, dtype=np.uint64) << np.uint64(28))
    phase = rng.integers(0, n_phases, n, dtype=np.uint64)
    e["key"] = (phase << np.uint64(48)) | (op << np.uint64(32)) | shape
    assert len(np.unique(e["key"])) == n
    e["count"] = rng.integers(1, 1 << 40, n, dtype=np.uint64)
    if wt_kind == "wide":
        bits = rng.integers(0, 88, n)
        lo = rng.integers(0, 1 << 63, n, dtype=np.uint64) * np.uint64(2) + rng.integers(0, 2, n, dtype=np.uint64)
        hi = rng.integers(0, 1 << 24, n, dtype=np.uint64)
        for i in range(n):                      # clip each value to `bits[i]` significant bits
            b = int(bits[i])
            v = ((int(hi[i]) << 64) | int(lo[i])) & ((1 << b) - 1) if b else 0
            lo[i], hi[i] = v & (2**64 - 1), v >> 64
        e["wt_lo"], e["wt_hi"] = lo, hi
    elif wt_kind == "ties":
        vals = np.array([0, 1, 5, 1 << 33, (1 << 64) - 1], dtype=np.uint64)
        pick = rng.integers(0, len(vals), n)
        e["wt_lo"] = vals[pick]
        e["wt_hi"] = (pick == 2).astype(np.uint64) * np.uint64(3)
    elif wt_kind == "narrow":
        e["wt_lo"] = rng.integers(0, 1 << 20, n, dtype=np.uint64)
    e["phase_weight"] = rng.random(n)
    e["roofline_s"] = rng.random(n)
    return e


def check_rank(lib, entries_host, entries_dev, n, phases, ppms=PPMS, out_cap=None):
    for phase in phases:
        for ppm in ppms:
            exp_r, exp_c, exp_res = oracle.rank_phase(entries_host, phase, ppm, out_cap=out_cap)
            got_r, got_c, got_res = lib.rank_entries(entries_dev, n, phase, ppm, out_cap=out_cap)
            assert got_res == exp_res, (phase, ppm, got_res, exp_res)
            assert host(got_r, lib.ENTRY_DTYPE).tobytes() == exp_r.tobytes(), (phase, ppm)
            assert host(got_c, np.float64).tobytes() == exp_c.tobytes(), (phase, ppm)


@pytest.mark.parametrize("index,n", [(0, 200_000), (1, 400_000), (2, 300_000), (4, 300_000)])
def test_sorted_and_ranked_artefacts_from_a_trace(lib, index, n):
    import torch
    spec = make_spec(index, small=True, n=n)
    recs = tg.generate(spec)
    work = spec.work_table()
    o = oracle.Oracle(spec.app_weights, spec.n_phases)
    o.set_work(work)
    o.ingest(recs, threads=4)
    exp_entries = o.finalize(PEAK_BW, PEAK_FLOPS)             # the oracle's own list, in key order
    agg = lib.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys, max_work_rows=len(work))
    agg.set_work_table(work)
    agg.ingest(torch.from_numpy(recs.view(np.uint8).reshape(-1)).cuda(), n=len(recs))
    entries, n_ent = agg.finalize(PEAK_BW, PEAK_FLOPS)        # table order
    assert n_ent == len(exp_entries)
    got = lib.sort_entries_by_key(entries, n_ent)
    assert host(got, lib.ENTRY_DTYPE).tobytes() == oracle.sort_by_key(exp_entries).tobytes()
    check_rank(lib, exp_entries, entries, n_ent, range(spec.n_phases + 1), ppms=(0, 500_000, 900_000, 1_000_000))
    # the head of the ranking is what the handle's top-k returns
    for phase in range(spec.n_phases):
        head, _, _ = lib.rank_entries(entries, n_ent, phase, 0, out_cap=10)
        assert host(head, lib.ENTRY_DTYPE).tobytes() == agg.topk(phase, 10).tobytes()


@pytest.mark.parametrize("n", [1, 31, 8191, 8192, 8193, 100_003])
@pytest.mark.parametrize("wt_kind", ["wide", "ties"])
def test_synthetic_lists_across_tile_boundaries(lib, n, wt_kind):
    e = synthetic_entries(100 + n, n, 3, wt_kind)
    d = dev(e)
    assert host(lib.sort_entries_by_key(d, n), lib.ENTRY_DTYPE).tobytes() == oracle.sort_by_key(e).tobytes()
    check_rank(lib, e, d, n, (0, 1, 2, 7))


def test_large_list_with_every_word_in_play(lib):
    n = (1 << 21) + 4099
    e = synthetic_entries(9, n, 2, "wide")
    d = dev(e)
    assert host(lib.sort_entries_by_key(d, n), lib.ENTRY_DTYPE).tobytes() == oracle.sort_by_key(e).tobytes()
    check_rank(lib, e, d, n, (0, 1), ppms=(0, 700_000, 1_000_000))
    check_rank(lib, e, d, n, (1,), ppms=(950_000,), out_cap=1000)     # truncated output, same cut


def test_degenerate_lists(lib):
    n = 50_000
    z = synthetic_entries(4, n, 2, "zero")
    check_rank(lib, z, dev(z), n, (0, 1), ppms=(0, 600_000, 1_000_000))     # T = 0: shares +0.0, nothing kept
    nar = synthetic_entries(5, n, 1, "narrow")                               # most digits constant: passes skipped
    d = dev(nar)
    assert host(lib.sort_entries_by_key(d, n), lib.ENTRY_DTYPE).tobytes() == oracle.sort_by_key(nar).tobytes()
    check_rank(lib, nar, d, n, (0,))
    same = nar.copy()                                                        # one weight for all: order = key order
    same["wt_lo"] = 77
    check_rank(lib, same, dev(same), n, (0,), ppms=(1, 500_000, 1_000_000))
    # already sorted and reverse-sorted inputs
    asc = oracle.sort_by_key(nar)
    for arr in (asc, asc[::-1].copy()):
        assert host(lib.sort_entries_by_key(dev(arr), n), lib.ENTRY_DTYPE).tobytes() == asc.tobytes()


def test_worked_example_and_printed_column_on_gpu(lib, golden_dir):
    g = load_golden(golden_dir, "rank_example.json")
    e = np.zeros(len(g["entries"]), dtype=oracle.ENTRY_DTYPE)
    for i, r in enumerate(g["entries"]):
        e[i]["key"] = (r["phase"] << 48) | (r["key_op"] << 32) | r["key_shape"]
        e[i]["wt_lo"], e[i]["wt_hi"] = int(r["wt"]) & (2**64 - 1), int(r["wt"]) >> 64
    d = dev(e)
    ranked, cum, res = lib.rank_entries(d, len(e), g["phase"], 0)
    keys = host(ranked, lib.ENTRY_DTYPE)["key"]
    assert [[int(k >> 32) & 0xFFFF, int(k) & 0xFFFFFFFF] for k in keys] == g["ranked_ops_shapes"]
    assert list(host(cum, np.float64)) == g["cum"] and res["total"] == int(g["total"])
    for c in g["cuts"]:
        res = lib.rank_entries(d, len(e), g["phase"], c["coverage_ppm"])[2]
        assert res["n_keep"] == c["n_keep"] and res["covered"] == int(c["covered"]), c
    t2 = load_golden(golden_dir, "table2_cumulative.json")
    wts = [10 * s for s in t2["score_milli"]] + [10 * t2["tail_score_milli"] // t2["tail_operators"]] * t2["tail_operators"]
    e = np.zeros(len(wts), dtype=oracle.ENTRY_DTYPE)
    e["key"] = np.arange(len(wts), dtype=np.uint64)[::-1] + np.uint64(1 << 32)
    e["wt_lo"] = wts
    d = dev(e)
    _, cum, _ = lib.rank_entries(d, len(e), 0, 0)
    cum = host(cum, np.float64)
    for i, printed in enumerate(t2["cum_printed"]):
        assert abs(cum[i] - printed) <= (i + 1) * 0.0005 + 0.0005 + 0.001
    for c in t2["cuts"]:
        assert lib.rank_entries(d, len(e), 0, c["coverage_ppm"])[2]["n_keep"] == c["n_keep"], c


def test_argument_checks(lib):
    import torch
    n = 1000
    e = synthetic_entries(1, n, 2, "narrow")
    d = dev(e)
    out = torch.empty(n * 48, dtype=torch.uint8, device="cuda:0")
    cum = torch.empty(n, dtype=torch.float64, device="cuda:0")
    nbytes = lib.atrex_release_scratch_bytes(n)
    scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda:0")
    base = (scratch.data_ptr() + 255) // 256 * 256
    res = lib.atrex_rank_result_t()
    big = lib.ATREX_RELEASE_MAX_ENTRIES + 1
    assert lib.atrex_release_scratch_bytes(big) == 0 and nbytes > 24 * n
    assert lib.atrex_entries_sort_by_key(d.data_ptr(), big, out.data_ptr(), base, nbytes, None) == lib.ATREX_ERR_TOO_LARGE
    assert lib.atrex_entries_sort_by_key(d.data_ptr(), n, out.data_ptr(), base, nbytes - 1, None) == lib.ATREX_ERR_NOMEM
    assert lib.atrex_entries_sort_by_key(d.data_ptr(), n, out.data_ptr(), base + 8, nbytes, None) == lib.ATREX_ERR_INVALID
    assert lib.atrex_entries_sort_by_key(d.data_ptr(), n, d.data_ptr(), base, nbytes, None) == lib.ATREX_ERR_INVALID
    assert lib.atrex_entries_sort_by_key(None, n, out.data_ptr(), base, nbytes, None) == lib.ATREX_ERR_INVALID
    assert lib.atrex_entries_sort_by_key(None, 0, None, None, 0, None) == lib.ATREX_OK
    args = (out.data_ptr(), cum.data_ptr(), n, C.byref(res), base, nbytes, None)
    assert lib.atrex_entries_rank(d.data_ptr(), n, 8, 0, *args) == lib.ATREX_ERR_INVALID
    assert lib.atrex_entries_rank(d.data_ptr(), n, 0, 1_000_001, *args) == lib.ATREX_ERR_INVALID
    assert lib.atrex_entries_rank(d.data_ptr(), big, 0, 0, *args) == lib.ATREX_ERR_TOO_LARGE
    assert lib.atrex_entries_rank(d.data_ptr(), n, 0, 0, None, None, n, C.byref(res), base, nbytes, None) \
        == lib.ATREX_ERR_INVALID
    assert lib.atrex_entries_rank(d.data_ptr(), n, 0, 0, out.data_ptr(), cum.data_ptr(), n, C.byref(res), base, 100, None) \
        == lib.ATREX_ERR_NOMEM
    # counts and cut only, no output buffers
    assert lib.atrex_entries_rank(d.data_ptr(), n, 0, 500_000, None, None, 0, C.byref(res), base, nbytes, None) == lib.ATREX_OK
    exp = oracle.rank_phase(e, 0, 500_000)[2]
    assert (res.n_phase, res.n_keep, res.total_lo, res.covered_lo) == (exp["n_phase"], exp["n_keep"], exp["total"], exp["covered"])
    # a phase total of 2^108 or more cannot be scaled by 10^6 in 128 bits: refused
    huge = e.copy()
    huge["wt_hi"][0] = 1 << 44
    assert lib.atrex_entries_rank(dev(huge).data_ptr(), n, int(huge["key"][0]) >> 48, 10, *args) == lib.ATREX_ERR_TOO_LARGE


def test_refresh_round_trip(lib):
    """A stored artefact (the key-sorted entry list) is folded into a fresh handle before a new batch of
    records arrives; the result equals aggregating old and new records together."""
    import torch
    spec = make_spec(1, small=True, n=600_000)
    recs = tg.generate(spec)
    old, new = recs[:350_000], recs[350_000:]
    a = lib.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys)
    a.ingest(torch.from_numpy(old.view(np.uint8).reshape(-1)).cuda(), n=len(old))
    ent, n_ent = a.finalize(PEAK_BW, PEAK_FLOPS)
    stored = lib.sort_entries_by_key(ent, n_ent).cpu()               # the artefact leaves the device
    b = lib.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys)
    b.merge(stored.cuda(), n_ent)
    b.ingest(torch.from_numpy(new.view(np.uint8).reshape(-1)).cuda(), n=len(new))
    o = oracle.Oracle(spec.app_weights, spec.n_phases)
    o.ingest(recs, threads=4)
    exp = o.finalize(PEAK_BW, PEAK_FLOPS)
    ent2, n2 = b.finalize(PEAK_BW, PEAK_FLOPS)
    assert host(lib.sort_entries_by_key(ent2, n2), lib.ENTRY_DTYPE).tobytes() == exp.tobytes()
