"""The multi-rank path on CPU: two gloo ranks shard a trace, exchange their partial aggregates
by key owner, and the union must equal the single-rank result.  Per-rank aggregation, the fold
of received entries and the ranking use the CPU oracle here (no GPU on this machine); what is under
test is the product's host-side plumbing in ``paper_2607_14541_b200.distributed`` and the
library's host-callable pieces (owner function, exact combination of the totals)."""
import os
import socket

import numpy as np
import pytest
import torch.multiprocessing as mp

import oracle
import tracegen as tg
from tracegen.configs import make_spec

PEAK_BW, PEAK_FLOPS = 8.0e12, [1.0e15] * 8


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _fold(parts):
    """Exact fold of entry arrays by key (test-side stand-in for the merge kernel)."""
    acc = {}
    for part in parts:
        for e in part:
            k = int(e["key"])
            c, w = acc.get(k, (0, 0))
            acc[k] = (c + int(e["count"]), w + (int(e["wt_lo"]) | (int(e["wt_hi"]) << 64)))
    return acc


def _worker(rank, world, port, n, out_dir):
    import torch.distributed as dist
    from paper_2607_14541_b200 import distributed as D
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = make_spec(3, small=True, n=n)
    start, count = D.shard_range(n, rank, world)
    recs = tg.generate(spec, start, count)
    o = oracle.Oracle(spec.app_weights, spec.n_phases)
    o.ingest(recs)
    local = o.finalize(PEAK_BW, PEAK_FLOPS)
    received = D.exchange_entries_host(D.bucket_entries_by_owner_host(local, world))
    owned = _fold(received)
    assert all(D.owner_of_keys(np.array([k], dtype=np.uint64), world)[0] == rank for k in list(owned)[:200])
    mine_t = o.stats()["totals"]
    lo, hi = D.gather_totals_host(np.array([t & (2**64 - 1) for t in mine_t], dtype=np.uint64),
                                  np.array([t >> 64 for t in mine_t], dtype=np.uint64))
    totals = [int(lo[q]) | (int(hi[q]) << 64) for q in range(8)]
    # local top-k of the owned keys -> global top-k
    ent = np.zeros(len(owned), dtype=local.dtype)
    for i, (k, (c, w)) in enumerate(sorted(owned.items())):
        ent[i] = (k, c, w & (2**64 - 1), w >> 64, 0.0, 0.0)
    tops = []
    for phase in range(spec.n_phases):                    # every owner's local top-10, gathered, ranked again
        mine = oracle.rank_phase(ent, phase, 0)[0][:10]
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        tops.append(oracle.rank_phase(np.concatenate(gathered), phase, 0)[0][:10])
    np.save(os.path.join(out_dir, f"owned_{rank}.npy"), ent)
    if rank == 0:
        np.save(os.path.join(out_dir, "totals.npy"), np.array([str(t) for t in totals]))
        np.save(os.path.join(out_dir, "tops.npy"), np.concatenate(tops)["key"])
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_exchange_and_merge_equal_one_rank(tmp_path):
    from paper_2607_14541_b200 import distributed as D
    n, world = 60_001, 2
    mp.spawn(_worker, args=(world, _free_port(), n, str(tmp_path)), nprocs=world, join=True)
    spec = make_spec(3, small=True, n=n)
    o = oracle.Oracle(spec.app_weights, spec.n_phases)
    o.ingest(tg.generate(spec))
    whole = o.finalize(PEAK_BW, PEAK_FLOPS)
    parts = [np.load(os.path.join(tmp_path, f"owned_{r}.npy")) for r in range(world)]
    assert sum(len(p) for p in parts) == len(whole)                    # every key has exactly one owner
    union = np.concatenate(parts)
    union = union[np.argsort(union["key"], kind="stable")]
    for f in ("key", "count", "wt_lo", "wt_hi"):
        assert np.array_equal(union[f], whole[f]), f
    totals = [int(t) for t in np.load(os.path.join(tmp_path, "totals.npy"))]
    assert totals == o.stats()["totals"]
    expect = np.concatenate([o.topk(PEAK_BW, PEAK_FLOPS, ph, 10) for ph in range(spec.n_phases)])["key"]
    assert np.array_equal(np.load(os.path.join(tmp_path, "tops.npy")), expect)


def test_shard_ranges_and_owners_are_a_partition():
    from paper_2607_14541_b200 import distributed as D
    for n, world in ((10, 3), (1 << 30, 8), (7, 8)):
        spans = [D.shard_range(n, r, world) for r in range(world)]
        assert spans[0][0] == 0 and sum(c for _, c in spans) == n
        assert all(spans[i][0] + spans[i][1] == spans[i + 1][0] for i in range(world - 1))
    keys = np.arange(100_000, dtype=np.uint64) * np.uint64(2654435761)
    own = D.owner_of_keys(keys, 8)
    assert own.min() == 0 and own.max() == 7 and np.bincount(own).min() > 100_000 / 8 * 0.9
    # the owner function is the same whether asked one key at a time or in bulk
    import paper_2607_14541_b200 as p
    assert [p.atrex_key_owner(int(k), 8) for k in keys[:100]] == [int(x) for x in own[:100]]
    # 128-bit totals survive the combination with carries out of the low words
    a, b, c = (1 << 127) + (1 << 64) - 1, (1 << 64) - 1, 3
    lo = np.zeros((3, 8), dtype=np.uint64)
    hi = np.zeros((3, 8), dtype=np.uint64)
    for r, t in enumerate((a, b, c)):
        lo[r, 2], hi[r, 2] = t & (2**64 - 1), t >> 64
    out_lo, out_hi = p.combine_totals(lo, hi)
    assert (int(out_lo[2]) | (int(out_hi[2]) << 64)) == (a + b + c) % (1 << 128)
    assert not out_lo[[0, 1, 3, 4, 5, 6, 7]].any() and not out_hi[[0, 1, 3, 4, 5, 6, 7]].any()
