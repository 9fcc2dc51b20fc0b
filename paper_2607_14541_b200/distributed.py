"""Host-side plumbing for running the path on several GPUs (one process per GPU).

The aggregation shards by records: Eq. 2 is a plain sum over independent invocations and every
accumulator is an exact integer, so each rank aggregates its own slice of the trace with the
single-GPU kernels and no data-path collective.  One exchange step makes the partial results
global: every aggregated entry is sent to the rank that owns its key, and the owner folds what
it receives into its table with ``atrex_agg_merge`` (exact).  Per-phase totals are combined as
128-bit integers on the host: an element-wise reduction of the 64-bit halves would lose carries.

Only tensor plumbing lives here (torch.distributed for the exchange); all arithmetic on the
records stays in the CUDA kernels.  Works with the ``nccl`` backend on GPUs and with ``gloo`` on
CPU tensors (used by the multi-process tests).
"""
from __future__ import annotations

import numpy as np

ENTRY_BYTES = 48
_MIX = np.uint64(0x9E3779B97F4A7C15)


def shard_range(n_total: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous slice [start, start + count) of the trace that ``rank`` ingests."""
    start = n_total * rank // world
    return start, n_total * (rank + 1) // world - start


def owner_of_keys(keys: np.ndarray, world: int) -> np.ndarray:
    """Rank that owns each packed key (any fixed function of the key works; this one mixes the bits)."""
    with np.errstate(over="ignore"):
        h = np.asarray(keys, dtype=np.uint64) * _MIX
    return ((h >> np.uint64(33)) % np.uint64(world)).astype(np.int64)


def bucket_entries_by_owner(entries: np.ndarray, world: int) -> list[np.ndarray]:
    """Split a structured array of entries into one array per destination rank."""
    owner = owner_of_keys(entries["key"], world)
    order = np.argsort(owner, kind="stable")
    bounds = np.searchsorted(owner[order], np.arange(world + 1))
    return [entries[order[bounds[r]:bounds[r + 1]]] for r in range(world)]


def exchange_entries(buckets: list[np.ndarray], group=None, device=None) -> list[np.ndarray]:
    """All-to-all of per-destination entry arrays.  Returns what each source rank sent to this rank.

    With ``device`` set (a CUDA device) the payload travels as CUDA tensors over ``all_to_all_single``
    (NCCL over NVLink); otherwise as CPU tensors, gathered and filtered, which every backend supports.
    """
    import torch
    import torch.distributed as dist
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    assert len(buckets) == world
    dtype = buckets[0].dtype
    counts = torch.tensor([len(b) for b in buckets], dtype=torch.int64)
    all_counts = [torch.zeros(world, dtype=torch.int64) for _ in range(world)]
    if device is not None:
        counts_dev = counts.to(device)
        gathered = [torch.zeros(world, dtype=torch.int64, device=device) for _ in range(world)]
        dist.all_gather(gathered, counts_dev, group=group)
        all_counts = [g.cpu() for g in gathered]
    else:
        dist.all_gather(all_counts, counts, group=group)
    incoming = [int(all_counts[src][rank]) for src in range(world)]
    if device is not None:
        send = torch.from_numpy(np.concatenate(buckets).view(np.uint8).reshape(-1).copy()).to(device)
        recv = torch.empty(sum(incoming) * ENTRY_BYTES, dtype=torch.uint8, device=device)
        dist.all_to_all_single(recv, send, [c * ENTRY_BYTES for c in incoming],
                               [len(b) * ENTRY_BYTES for b in buckets], group=group)
        flat = recv.cpu().numpy()
        out, off = [], 0
        for c in incoming:
            out.append(flat[off:off + c * ENTRY_BYTES].view(dtype).copy())
            off += c * ENTRY_BYTES
        return out
    # portable path: every rank publishes all its buckets, each rank keeps the slices addressed to it
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


def combine_phase_totals(local_totals: list[int], group=None) -> list[int]:
    """Sum per-phase 128-bit totals over ranks exactly (gather the halves, add as integers)."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    halves = []
    for t in local_totals:
        halves += [t & 0xFFFFFFFF, (t >> 32) & 0xFFFFFFFF, (t >> 64) & 0xFFFFFFFF, (t >> 96) & 0xFFFFFFFF]
    mine = torch.tensor(halves, dtype=torch.int64)
    everyone = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(everyone, mine, group=group)
    out = [0] * len(local_totals)
    for t in everyone:
        v = t.tolist()
        for p in range(len(local_totals)):
            out[p] += v[4 * p] | (v[4 * p + 1] << 32) | (v[4 * p + 2] << 64) | (v[4 * p + 3] << 96)
    return out


def merge_ranked(candidates: list[np.ndarray], k: int) -> np.ndarray:
    """Global top-k from every rank's local top-k: weighted time descending (exact), key ascending."""
    allc = np.concatenate(candidates) if candidates else np.zeros(0)
    if len(allc) == 0:
        return allc
    wt = allc["wt_hi"].astype(object) * (1 << 64) + allc["wt_lo"].astype(object)
    order = sorted(range(len(allc)), key=lambda i: (-wt[i], int(allc["key"][i])))
    return allc[order[:k]]


def owner_of_keys_torch(keys):
    """``owner_of_keys`` on a CUDA int64 tensor of packed keys; ``world`` is applied by the caller."""
    import torch
    h = keys * torch.tensor(-7046029254386353131, dtype=torch.int64, device=keys.device)  # 0x9E3779B97F4A7C15
    return (h >> 33) & 0x7FFFFFFF  # logical shift of the product's top 31 bits


def bucket_entries_by_owner_torch(entries, n: int, world: int):
    """Split a CUDA uint8 tensor of ``n`` 48-byte entries into per-destination tensors (on the device)."""
    import torch
    e = entries[: n * ENTRY_BYTES].view(torch.int64).view(n, ENTRY_BYTES // 8)
    owner = owner_of_keys_torch(e[:, 0]) % world
    order = torch.argsort(owner, stable=True)
    counts = torch.bincount(owner, minlength=world).tolist()
    sorted_e = e[order].contiguous().view(torch.uint8).view(-1)
    out, off = [], 0
    for c in counts:
        out.append(sorted_e[off * ENTRY_BYTES:(off + c) * ENTRY_BYTES])
        off += c
    return out


def merge_and_finalize_owned(owner_agg, parts, peak_bw, peak_flops, global_totals):
    """Owner side of the exchange: fold the entry tensors received from every rank into
    ``owner_agg`` (``atrex_agg_merge``) and finalize against the totals over all shards."""
    for part in parts:
        if part.numel():
            owner_agg.merge(part, part.numel() // ENTRY_BYTES)
    return owner_agg.finalize(peak_bw, peak_flops, global_totals=global_totals)


def aggregate_sharded(local_agg, owner_agg, peak_bw, peak_flops, group=None):
    """Full multi-GPU flow for one rank, after ``local_agg`` has ingested this rank's slice:
    finalize locally, send every entry to its key's owner (NCCL all-to-all), fold what arrives into
    ``owner_agg``, combine the per-phase totals exactly, and finalize the owned keys against them.
    Returns (entries, n) of the keys this rank owns."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    local, n = local_agg.finalize(peak_bw, peak_flops)
    buckets = bucket_entries_by_owner_torch(local, n, world)
    send_counts = torch.tensor([b.numel() for b in buckets], dtype=torch.int64, device=local.device)
    recv_counts = torch.empty_like(send_counts)
    dist.all_to_all_single(recv_counts, send_counts, group=group)
    recv = torch.empty(int(recv_counts.sum()), dtype=torch.uint8, device=local.device)
    dist.all_to_all_single(recv, torch.cat(buckets) if buckets else local[:0], recv_counts.tolist(),
                           send_counts.tolist(), group=group)
    totals = combine_phase_totals(local_agg.stats()["totals"], group=group)
    return merge_and_finalize_owned(owner_agg, [recv], peak_bw, peak_flops, totals)
