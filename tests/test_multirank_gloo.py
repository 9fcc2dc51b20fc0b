"""The multi-rank path on CPU: two gloo ranks shard a trace, exchange their partial aggregates
by key owner, and the union must equal the single-rank result.  Per-rank aggregation and the
fold of received entries use the CPU oracle here (no GPU on this machine); what is under test is the
product's host-side plumbing in ``paper_2607_14541_b200.distributed``."""
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
    received = D.exchange_entries(D.bucket_entries_by_owner(local, world))
    owned = _fold(received)
    assert all(D.owner_of_keys(np.array([k], dtype=np.uint64), world)[0] == rank for k in list(owned)[:200])
    totals = D.combine_phase_totals(o.stats()["totals"])
    # local top-k of the owned keys -> global top-k
    ent = np.zeros(len(owned), dtype=local.dtype)
    for i, (k, (c, w)) in enumerate(sorted(owned.items())):
        ent[i] = (k, c, w & (2**64 - 1), w >> 64, 0.0, 0.0)
    tops = []
    for phase in range(spec.n_phases):
        sel = ent[(ent["key"] >> np.uint64(48)) == phase]
        mine = D.merge_ranked([sel], 10)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        tops.append(D.merge_ranked(gathered, 10))
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
    # 128-bit totals survive the combination with carries out of every 32-bit piece
    big = (1 << 127) + (1 << 64) - 1
    halves = [big & 0xFFFFFFFF, (big >> 32) & 0xFFFFFFFF, (big >> 64) & 0xFFFFFFFF, (big >> 96) & 0xFFFFFFFF]
    assert sum(h << (32 * i) for i, h in enumerate(halves)) == big
