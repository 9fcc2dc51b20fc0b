"""The multi-GPU step on one GPU, two ways, both through the functions a real multi-GPU run uses
(``distributed.prepare_outgoing`` / ``fold_incoming`` / ``rank_candidates``):

* ranks run one after the other in one process, the collectives replaced by local copies
  (``distributed.Loopback``): each "rank" aggregates its slice of the trace, groups its entries by
  key owner on the device, every owner folds what it would receive and finalizes against the exactly
  combined totals.  The union of the owners' outputs must equal the single-handle result, and the
  oracle, bit for bit -- including the per-phase weights, which depend on the totals over ALL shards;
* ``distributed.aggregate_sharded`` and ``global_topk`` end to end under ``torch.distributed`` with
  the NCCL backend and a world of one rank (the all-to-all, all-gather and ranking code paths as they
  run on several GPUs), again bit-equal to the oracle.
"""
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

    # every rank aggregates its own slice and prepares what it would send
    outgoing = []
    for rank in range(world):
        start, count = D.shard_range(len(recs), rank, world)
        a = new_handle()
        a.ingest(dev[start * 16:(start + count) * 16], n=count)
        out = D.prepare_outgoing(a, *peaks, world)
        assert sum(out.counts) == a.stats()["n_keys"]
        for dst in range(world):                          # grouped by owner, as the library's host function says
            part = out.part_for(dst).cpu().numpy().view(p.ENTRY_DTYPE)
            assert (D.owner_of_keys(part["key"], world) == dst).all()
        outgoing.append(out)
    wire = D.Loopback(outgoing)

    # every owner folds the parts addressed to it and finalizes against the global totals
    owned, owners = [], []
    for dst in range(world):
        owner = new_handle()
        received, lo_rows, hi_rows = wire.deliver(dst)
        ent, n = D.fold_incoming(owner, received, *peaks, lo_rows, hi_rows)
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

    # global ranking = the owners' local rankings, gathered and ranked again on the device
    for phase in range(spec.n_phases):
        cands = [torch.from_numpy(ow.topk(phase, 10).view(np.uint8).reshape(-1).copy()).cuda() for ow in owners]
        merged = D.rank_candidates(cands, phase, 10)
        assert merged.tobytes() == whole.topk(phase, 10).tobytes()
        assert merged.tobytes() == o.topk(*peaks, phase, 10).tobytes()


def test_aggregate_sharded_under_nccl_with_one_rank():
    """The exchange itself -- all_to_all_single of counts and payload, all_gather of the totals' words
    and of the ranking candidates -- under the NCCL backend, world size 1, on this GPU."""
    import socket
    import torch
    import torch.distributed as dist
    import paper_2607_14541_b200 as p
    from paper_2607_14541_b200 import distributed as D

    spec = make_spec(1, small=True, n=(1 << 20) + 17, n_dtypes=2)
    recs, work = tg.generate(spec), spec.work_table()
    peaks = (spec.peak_bw, spec.peak_flops)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda:0"))
    try:
        def new_handle():
            a = p.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys, max_work_rows=len(work))
            a.set_work_table(work)
            return a
        local, owner = new_handle(), new_handle()
        local.ingest(torch.from_numpy(recs.view(np.uint8).reshape(-1)).cuda(), n=len(recs))
        ent, n = D.aggregate_sharded(local, owner, *peaks)
        got = ent[: n * 48].cpu().numpy().view(p.ENTRY_DTYPE)
        got = got[np.argsort(got["key"], kind="stable")]
        o = oracle.Oracle(spec.app_weights, spec.n_phases)
        o.set_work(work)
        o.ingest(recs, threads=4)
        assert got.tobytes() == o.finalize(*peaks).tobytes()
        for phase in range(spec.n_phases):
            assert D.global_topk(owner, phase, 10).tobytes() == o.topk(*peaks, phase, 10).tobytes()
    finally:
        dist.destroy_process_group()
