"""The allocation-free ranking call, checked against the regular one and against the CPU oracle.

Some callers of this library cannot allocate device memory (their budget was split up at
start-up, or they are handed buffers but no allocator).  For them the library has one entry
point whose scratch space is a fixed array inside the library instead of a workspace.  This
test calls it through the C ABI on a finalize output and expects exactly what the handle-based
ranking returns -- and what the oracle's ranking of the same records gives -- on two calls in a
row: the second must not see anything the first left in the shared array.  It also checks the
one property the call exists for: the device's free memory does not move across the calls.  The
file name sorts last so that a failure here cannot hide other tests.
"""
import ctypes as C

import numpy as np
import pytest

import oracle
import tracegen as tg
from tracegen.configs import make_spec

pytestmark = pytest.mark.gpu


def test_static_scratch_topk_matches_the_workspace_topk_twice_in_a_row():
    import torch
    import paper_2607_14541_b200 as p

    spec = make_spec(1, small=True, n=300_000, n_dtypes=2)   # ~16k keys: well inside the fixed buffer
    recs = tg.generate(spec)
    work = spec.work_table()
    agg = p.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys, max_work_rows=len(work))
    agg.set_work_table(work)
    agg.ingest(torch.from_numpy(recs.view(np.uint8).reshape(-1)).cuda(), n=len(recs))
    entries, n = agg.finalize(spec.peak_bw, spec.peak_flops)
    assert 0 < n <= p.ATREX_STATIC_TOPK_MAX_ENTRIES
    out = torch.empty(4096 * 48, dtype=torch.uint8, device="cuda:0")      # the caller's output buffer
    ref = oracle.Oracle(spec.app_weights, spec.n_phases)
    ref.set_work(work)
    ref.ingest(recs)
    requests = ((1, 4096), (0, 7), (1, 1), (0, 4096))
    expected_lib = {r: agg.topk(*r) for r in requests}                    # the handle-based call may allocate; do it first
    n_out = C.c_uint32(0)                                                 # first call on this device: resolves the array's address
    assert p.atrex_topk_entries_static(entries.data_ptr(), n, 0, 1, out.data_ptr(), C.byref(n_out), None) == p.ATREX_OK
    torch.cuda.synchronize()

    # two calls in a row with different phases and sizes: a large selection first, then a
    # small one that would be polluted by leftovers if the shared array were not cleared
    host = torch.empty(4096 * 48, dtype=torch.uint8).pin_memory()
    free_before = torch.cuda.mem_get_info()[0]
    results = {}
    for phase, k in requests:
        n_out = C.c_uint32(0)
        rc = p.atrex_topk_entries_static(entries.data_ptr(), n, phase, k, out.data_ptr(), C.byref(n_out), None)
        assert rc == p.ATREX_OK
        host.copy_(out)                                                    # into memory that already exists
        results[(phase, k)] = host[: n_out.value * 48].numpy().view(p.ENTRY_DTYPE).copy()
    assert torch.cuda.mem_get_info()[0] == free_before                     # nothing was allocated on the device
    for (phase, k), got in results.items():
        assert got.tobytes() == expected_lib[(phase, k)].tobytes(), (phase, k)
        assert got.tobytes() == ref.topk(spec.peak_bw, spec.peak_flops, phase, k).tobytes(), (phase, k)

    # sizes beyond the fixed array are refused up front, and nothing is written
    n_out = C.c_uint32(123)
    too_many = p.ATREX_STATIC_TOPK_MAX_ENTRIES + 1
    assert p.atrex_topk_entries_static(entries.data_ptr(), too_many, 0, 1, out.data_ptr(), C.byref(n_out), None) \
        == p.ATREX_ERR_TOO_LARGE
    assert p.atrex_topk_entries_static(entries.data_ptr(), n, 0, too_many, out.data_ptr(), C.byref(n_out), None) \
        == p.ATREX_ERR_TOO_LARGE
    assert n_out.value == 0
    # an empty input or k == 0 is fine and writes nothing
    assert p.topk_entries_static(entries, 0, 0, 5, out) == 0
    assert p.topk_entries_static(entries, n, 0, 0, out) == 0
    # a phase with no entries
    assert p.topk_entries_static(entries, n, 5, 5, out) == 0
