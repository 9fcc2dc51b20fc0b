"""The multi-GPU flow on one GPU, ranks run one after the other: each "rank" aggregates its slice
of the trace, the partial entries are bucketed by key owner, every owner folds what it would
receive (atrex_agg_merge) and finalizes against the exactly combined totals.  The union of the
owners' outputs must equal the single-handle result, and the oracle, bit for bit -- including the
per-phase weights, which depend on the totals over ALL shards.  (The NCCL exchange itself moves
bytes only; its host logic is covered by the 2-rank gloo test.)"""
import numpy as np
import pytest

import oracle
import tracegen as tg
from tracegen.configs import make_spec

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_aggregation_equals_single_handle(world):
    import torch
    import paper_2607_14541_b200 as p
    from paper_2607_14541_b200 import distributed as D

    spec = make_spec(3, small=True, n=(1 << 21) + 3, n_dtypes=3)
    recs, work = tg.generate(spec), spec.work_table()
    peaks = (spec.peak_bw, spec.peak_flops)
    dev = torch.from_numpy(recs.view(np.uint8).reshape(-1)).cuda()

    def new_handle():
        a = p.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys, max_work_rows=len(work))
        a.set_work_table(work)
        return a

    whole = new_handle()
    whole.ingest(dev, n=len(recs))
    expect = whole.finalize_numpy(*peaks)
    expect = expect[np.argsort(expect["key"], kind="stable")]

    # every rank aggregates its own slice
    locals_ = []
    for rank in range(world):
        start, count = D.shard_range(len(recs), rank, world)
        a = new_handle()
        a.ingest(dev[start * 16:(start + count) * 16], n=count)
        locals_.append(a)
    buckets = [D.bucket_entries_by_owner_torch(*a.finalize(*peaks), world) for a in locals_]
    totals = [sum(a.stats()["totals"][ph] for a in locals_) for ph in range(8)]
    assert totals == whole.stats()["totals"]

    # every owner folds the parts addressed to it and finalizes against the global totals
    owned, owners = [], []
    for dst in range(world):
        owner = new_handle()
        ent, n = D.merge_and_finalize_owned(owner, [buckets[src][dst] for src in range(world)], *peaks, totals)
        part = ent[: n * 48].cpu().numpy().view(p.ENTRY_DTYPE)
        assert (D.owner_of_keys(part["key"], world) == dst).all()
        owned.append(part)
        owners.append(owner)
    union = np.concatenate(owned)
    union = union[np.argsort(union["key"], kind="stable")]
    assert union.tobytes() == expect.tobytes()

    o = oracle.Oracle(spec.app_weights, spec.n_phases)
    o.set_work(work)
    o.ingest(recs, threads=4)
    assert union.tobytes() == o.finalize(*peaks).tobytes()

    # global ranking = merge of the owners' local rankings
    for phase in range(spec.n_phases):
        merged = D.merge_ranked([ow.topk(phase, 10) for ow in owners], 10)
        assert merged.tobytes() == whole.topk(phase, 10).tobytes()
