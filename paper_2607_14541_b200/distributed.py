"""Host-side plumbing for running the path on several GPUs (one process per GPU).

The aggregation shards by records: Eq. 2 is a plain sum over independent invocations and every
accumulator is an exact integer, so each rank aggregates its own slice of the trace with the
single-GPU kernels and no data-path collective.  One exchange step makes the partial results
global: every aggregated entry is sent to the rank that owns its key, and the owner folds what
it receives into its table with ``atrex_agg_merge`` (exact); Eq. 3's denominators become the sums
of the shards' per-phase totals.

Only plumbing lives here -- tensors handed to ``torch.distributed`` and to the C ABI.  Every piece
of arithmetic on keys, weights and totals is a library call: the owner function
(``atrex_key_owner``), the grouping of entries by owner (``atrex_entries_bucket_by_owner``), the
128-bit combination of totals (``atrex_totals_combine``; an element-wise reduction of 64-bit halves
by the collective would lose carries), the fold (``atrex_agg_merge``), the normalisation
(``atrex_agg_finalize_with_totals``) and the ranking of the gathered candidates
(``atrex_topk_entries_static``).  Received entries land in this GPU's own memory through plain NCCL
receives; no kernel is handed another GPU's memory.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import binding as B

ENTRY_BYTES = 48


def shard_range(n_total: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous slice [start, start + count) of the trace that ``rank`` ingests."""
    start = n_total * rank // world
    return start, n_total * (rank + 1) // world - start


def owner_of_keys(keys: np.ndarray, world: int) -> np.ndarray:
    """Rank that owns each packed key (``atrex_keys_owner``, the library's host-side owner function)."""
    k = np.ascontiguousarray(keys, dtype=np.uint64)
    out = np.zeros(k.shape[0], dtype=np.uint32)
    B.atrex_keys_owner(k.ctypes.data, k.shape[0], int(world), out.ctypes.data)
    return out.astype(np.int64)


# ---------------------------------------------------------------- one rank's two halves of the step

class Outgoing:
    """What one rank contributes to the exchange: its entries grouped by owner (a CUDA byte tensor),
    the entry count per destination rank, and its per-phase totals as (lo[8], hi[8]) words."""

    def __init__(self, grouped, counts, totals_lo, totals_hi):
        self.grouped, self.counts, self.totals_lo, self.totals_hi = grouped, counts, totals_lo, totals_hi

    def part_for(self, dst: int):
        begin = sum(self.counts[:dst]) * ENTRY_BYTES
        return self.grouped[begin: begin + self.counts[dst] * ENTRY_BYTES]


def prepare_outgoing(local_agg, peak_bw: float, peak_flops, world: int, out=None) -> Outgoing:
    """Sender side: finalize this rank's partial aggregate and group its entries by owner on the device.
    ``out``: an optional CUDA byte tensor with room for every key's 48-byte entry; with it the finalize
    is one pass (without it, a counting pass sizes the output first)."""
    local, n = local_agg.finalize(peak_bw, peak_flops, out=out)
    lo, hi = local_agg.totals_words()                 # the totals the finalize just computed: no second pass
    grouped, counts = B.bucket_entries_by_owner(local, n, world)
    return Outgoing(grouped, counts, lo, hi)


def fold_incoming(owner_agg, received, peak_bw: float, peak_flops, totals_lo_rows, totals_hi_rows, out=None):
    """Owner side: fold the received entries (a CUDA byte tensor, any order) into ``owner_agg``, combine the
    shards' totals exactly and finalize the owned keys against them (into ``out`` when given).  Returns
    (entries, n)."""
    n = received.numel() // ENTRY_BYTES
    if n:
        owner_agg.merge(received, n)
    lo, hi = B.combine_totals(totals_lo_rows, totals_hi_rows)
    return owner_agg.finalize(peak_bw, peak_flops, out=out, global_totals=(lo, hi))


# ---------------------------------------------------------------- the exchange over torch.distributed

def exchange(outgoing: Outgoing, group=None):
    """All-to-all of the grouped entries (``all_to_all_single``: NCCL over NVLink on GPUs) and all-gather of
    the totals' words.  Returns (received CUDA byte tensor, lo rows [world, 8], hi rows [world, 8])."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    dev = outgoing.grouped.device
    send_counts = torch.tensor([c * ENTRY_BYTES for c in outgoing.counts], dtype=torch.int64, device=dev)
    recv_counts = torch.empty_like(send_counts)
    dist.all_to_all_single(recv_counts, send_counts, group=group)
    recv_list = recv_counts.tolist()
    received = torch.empty(sum(recv_list), dtype=torch.uint8, device=dev)
    dist.all_to_all_single(received, outgoing.grouped, recv_list, send_counts.tolist(), group=group)
    words = torch.from_numpy(np.concatenate([outgoing.totals_lo, outgoing.totals_hi]).view(np.int64).copy()).to(dev)
    rows = [torch.empty_like(words) for _ in range(world)]
    dist.all_gather(rows, words, group=group)
    table = torch.stack(rows).cpu().numpy().view(np.uint64)
    return received, table[:, :B.ATREX_MAX_PHASES].copy(), table[:, B.ATREX_MAX_PHASES:].copy()


def aggregate_sharded(local_agg, owner_agg, peak_bw: float, peak_flops, group=None, out_local=None, out_owner=None):
    """Full multi-GPU step for one rank, after ``local_agg`` has ingested this rank's slice: group the
    local entries by owner, exchange, fold what arrives into ``owner_agg`` and finalize the owned keys
    against the totals over all shards.  Returns (entries, n) of the keys this rank owns.  ``out_local`` /
    ``out_owner``: optional output buffers for the two finalize calls (one pass each instead of two)."""
    import torch.distributed as dist
    out = prepare_outgoing(local_agg, peak_bw, peak_flops, dist.get_world_size(group), out=out_local)
    received, lo_rows, hi_rows = exchange(out, group)
    return fold_incoming(owner_agg, received, peak_bw, peak_flops, lo_rows, hi_rows, out=out_owner)


def global_topk(owner_agg, phase: int, k: int, group=None):
    """Table 2's ranking over all shards: every owner's local top-k is gathered and the candidates are
    ranked on the device (``atrex_topk_entries_static``: weighted time descending as exact integers,
    key ascending).  Returns a numpy array of entries; world * k may be at most 65 536."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    dev = f"cuda:{owner_agg.device}"
    mine = owner_agg.topk(phase, k)
    padded = np.zeros(k * ENTRY_BYTES + 8, dtype=np.uint8)
    padded[:8] = np.array([len(mine)], dtype=np.uint64).view(np.uint8)
    padded[8: 8 + mine.nbytes] = mine.view(np.uint8).reshape(-1)
    send = torch.from_numpy(padded).to(dev)
    rows = [torch.empty_like(send) for _ in range(world)]
    dist.all_gather(rows, send, group=group)
    return rank_candidates([r[8: 8 + int(r[:8].view(torch.int64).item()) * ENTRY_BYTES] for r in rows], phase, k)


def rank_candidates(parts, phase: int, k: int) -> np.ndarray:
    """The best ``k`` of the candidate entries in ``parts`` (CUDA byte tensors), ranked on the device."""
    import torch
    parts = [p for p in parts if p.numel()]
    if not parts or k == 0:
        return np.zeros(0, dtype=B.ENTRY_DTYPE)
    cand = torch.cat(parts).contiguous()
    out = torch.empty(k * ENTRY_BYTES, dtype=torch.uint8, device=cand.device)
    m = B.topk_entries_static(cand, cand.numel() // ENTRY_BYTES, phase, k, out)
    return out[: m * ENTRY_BYTES].cpu().numpy().view(B.ENTRY_DTYPE).copy()


# ---------------------------------------------------------------- ranks run in turn inside one process

class Loopback:
    """Stands in for the collectives when several ranks are run one after the other in a single process
    (one GPU): it is handed every rank's ``Outgoing`` and gives each destination what the all-to-all
    would deliver, as local copies."""

    def __init__(self, outgoing: list[Outgoing]):
        self.outgoing = outgoing

    def deliver(self, dst: int):
        import torch
        received = torch.cat([o.part_for(dst) for o in self.outgoing])
        lo_rows = np.stack([o.totals_lo for o in self.outgoing])
        hi_rows = np.stack([o.totals_hi for o in self.outgoing])
        return received, lo_rows, hi_rows


# ---------------------------------------------------------------- CPU tensors (gloo), for the host-logic tests

def bucket_entries_by_owner_host(entries: np.ndarray, world: int) -> list[np.ndarray]:
    """Split a structured array of entries into one array per destination rank (host memory; the
    device path uses ``atrex_entries_bucket_by_owner``)."""
    owner = owner_of_keys(entries["key"], world)
    order = np.argsort(owner, kind="stable")
    bounds = np.searchsorted(owner[order], np.arange(world + 1))
    return [entries[order[bounds[r]:bounds[r + 1]]] for r in range(world)]


def exchange_entries_host(buckets: list[np.ndarray], group=None) -> list[np.ndarray]:
    """All-to-all of per-destination entry arrays as CPU tensors (every backend supports the all-gather
    it is built from).  Returns what each source rank sent to this rank."""
    import torch
    import torch.distributed as dist
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    assert len(buckets) == world
    dtype = buckets[0].dtype
    counts = torch.tensor([len(b) for b in buckets], dtype=torch.int64)
    all_counts = [torch.zeros(world, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(all_counts, counts, group=group)
    incoming = [int(all_counts[src][rank]) for src in range(world)]
    width = int(max(int(c.sum()) for c in all_counts))
    mine = np.zeros(width * ENTRY_BYTES, dtype=np.uint8)
    payload = np.concatenate(buckets).view(np.uint8).reshape(-1)
    mine[: payload.shape[0]] = payload
    everyone = [torch.zeros(width * ENTRY_BYTES, dtype=torch.uint8) for _ in range(world)]
    dist.all_gather(everyone, torch.from_numpy(mine), group=group)
    out = []
    for src in range(world):
        begin = int(all_counts[src][:rank].sum()) * ENTRY_BYTES
        raw = everyone[src].numpy()[begin: begin + incoming[src] * ENTRY_BYTES]
        out.append(raw.view(dtype).copy())
    return out


def gather_totals_host(totals_lo: np.ndarray, totals_hi: np.ndarray, group=None):
    """All-gather of one rank's totals' words as CPU tensors, combined exactly by the library.
    Returns (lo[8], hi[8])."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    words = torch.from_numpy(np.concatenate([totals_lo, totals_hi]).astype(np.uint64).view(np.int64).copy())
    rows = [torch.empty_like(words) for _ in range(world)]
    dist.all_gather(rows, words, group=group)
    table = torch.stack(rows).numpy().view(np.uint64)
    return B.combine_totals(table[:, :B.ATREX_MAX_PHASES].copy(), table[:, B.ATREX_MAX_PHASES:].copy())
