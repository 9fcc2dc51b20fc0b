// Ingest, everything but the scatter pass (scatter.cu): Eq. 2's group-by sum, streamed, as a
// two-pass radix-partitioned aggregation.
//
// Random read-modify-write into a table far larger than L2 is bound by DRAM latency and by
// the L2's atomic rate, not by bandwidth, so the hot path avoids global atomics altogether:
//
// Pass 1  SCATTER  (scatter.cu) accumulates the records of hot keys in a shared-memory directory
//   and appends every other record as a 12-byte entry to the CTA's private buffer of the key's
//   partition.
//
// Pass 2  PARTITION  (persistent CTAs, one partition at a time each).  Runs lazily: only when a
//   buffer is filling up, or when results are about to be read.  The CTA copies its
//   partition's keys from HBM into shared memory, streams the partition's entries from all
//   scatter CTAs, finds or claims each key's slot in shared memory and accumulates there, then
//   adds the per-slot deltas back to the HBM table with coalesced read-modify-writes.  The CTA
//   is the only writer of its partition, so no global atomics are involved.
//
// All sums are integers, so the result does not depend on which route a record took, on
// scheduling, or on chunking.  Entries that do not fit a spill buffer, directory wraps and
// merges fall back to exact atomic updates of the HBM table.
#include <type_traits>

#include "atrex_dev.cuh"
#include "kernels.h"

namespace atrex {

constexpr int INGEST_THREADS = 1024;
constexpr uint32_t DIR_WAYS = 4;                   // slots per hot-directory bucket (32 bytes of keys)
constexpr uint32_t NEW_KEY_FLAG = 0x80000000u;     // partition pass: slot claimed in this launch

__device__ __forceinline__ uint32_t dir_bucket_of_key(ull key, uint32_t mult, uint32_t n_buckets) {
    return dir_bucket(hash32(key), (uint32_t)(key >> 48), mult, n_buckets);
}
__constant__ uint32_t DIR_MULTS[4] = {0xC2B2AE35u, 0x27D4EB2Fu, 0x165667B1u, 0x9E3779B9u};

// Shared memory is addressed explicitly through 32-bit shared-window addresses in the hot
// loops: one integer add per access instead of generic 64-bit pointer arithmetic.
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ ulonglong2 lds_v2u64(uint32_t a) {
    ulonglong2 v;
    asm volatile("ld.shared.v2.u64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t atoms_add(uint32_t a, uint32_t v) {
    uint32_t o;
    asm volatile("atom.shared.add.u32 %0, [%1], %2;" : "=r"(o) : "r"(a), "r"(v) : "memory");
    return o;
}
__device__ __forceinline__ void reds_add(uint32_t a, uint32_t v) {
    asm volatile("red.shared.add.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void reds_or(uint32_t a, uint32_t v) {
    asm volatile("red.shared.or.b32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t atoms_exch(uint32_t a, uint32_t v) {
    uint32_t o;
    asm volatile("atom.shared.exch.b32 %0, [%1], %2;" : "=r"(o) : "r"(a), "r"(v) : "memory");
    return o;
}
__device__ __forceinline__ ull atoms_cas64(uint32_t a, ull expected, ull desired) {
    ull o;
    asm volatile("atom.shared.cas.b64 %0, [%1], %2, %3;" : "=l"(o) : "r"(a), "l"(expected), "l"(desired) : "memory");
    return o;
}

// Shared-memory accumulation uses native 32-bit atomics only (64-bit shared atomics are
// compare-and-swap loops).  A slot's weighted time is kept in two limbs: the returning add on
// the low limb tells the adder whether it wrapped, and the adder then adds the carry, with the
// value's high word, to the high limb (part_accumulate).  One add raises the high limb by at most 2^21 (a warp's
// combined 32 records of < 2^48 each), so the adder that takes it across 2^30 drains both
// limbs; the adds that can slip in before its exchange (one per thread of the CTA) stay below
// 2^31, so the high limb never wraps.
constexpr uint32_t DRAIN_BIT = 0x40000000u;

__device__ __forceinline__ ull limbs_drain(uint32_t a0, uint32_t a1, ull* hi_out) {
    // the two exchanges need not be simultaneous: whatever lands between them stays in the
    // limbs for the next drain or the final flush
    const ull lo = atoms_exch(a0, 0u);
    const ull hi = atoms_exch(a1, 0u);
    const ull v = lo + (hi << 32);
    *hi_out = v < lo ? 1ull : 0ull;
    return v;
}

// Adds every CTA's directory image row into the table and clears the rows.  A CTA handles 32
// directory slots: warp w sums rows w, w + 8, ... of those slots (exact: 128-bit sum, count), the
// eight partial sums meet in shared memory and warp 0 does one table update per slot.
constexpr int FOLD_WARPS = 8;

__global__ void __launch_bounds__(FOLD_WARPS * 32) hot_fold_kernel(const ull* hot_keys, ulonglong2* hot_img,
                                                                   uint32_t n_groups, uint32_t hot_slots, TableRef t) {
    __shared__ ull s_lo[FOLD_WARPS][32], s_hi[FOLD_WARPS][32], s_cnt[FOLD_WARPS][32];
    const uint32_t lane = threadIdx.x & 31u, w = threadIdx.x >> 5;
    const uint32_t i = blockIdx.x * 32u + lane;
    ull lo = 0, hi = 0, count = 0;
    if (i < hot_slots) {
        for (uint32_t g = w; g < n_groups; g += FOLD_WARPS) {
            ulonglong2* at = hot_img + (size_t)g * hot_slots + i;
            const ulonglong2 v = *at;
            if ((v.x | v.y) == 0) continue;
            const ull s = lo + v.x;
            hi += (v.y >> HI_SHIFT) + (s < lo ? 1ull : 0ull);
            lo = s;
            count += v.y & COUNT_MASK;
            *at = make_ulonglong2(0, 0);
        }
    }
    s_lo[w][lane] = lo;
    s_hi[w][lane] = hi;
    s_cnt[w][lane] = count;
    __syncthreads();
    if (w == 0 && i < hot_slots) {
#pragma unroll
        for (int k = 1; k < FOLD_WARPS; ++k) {
            const ull s = lo + s_lo[k][lane];
            hi += s_hi[k][lane] + (s < lo ? 1ull : 0ull);
            lo = s;
            count += s_cnt[k][lane];
        }
        if ((lo | hi | count) != 0) {
            const ull key = ~hot_keys[i];
            table_accumulate(t, key, hash32(key), lo, hi, count);
        }
    }
}

// --------------------------------------------------------------------------------------
// Pass 2: a CTA aggregates one partition at a time entirely in shared memory.  CTAs are
// persistent and take partitions blockIdx.x, blockIdx.x + gridDim.x, ...; while one partition
// is processed, the next one's keys and spill entries are pulled into L2.  Per partition: copy the
// keys in, each in the pass's own 64-bit form (phase, operator, 32-bit hash: unique inside a
// partition, and what a spill entry carries); stream the entries of all scatter CTAs, four per lane,
// and settle each with one look at the first pair of its probe sequence (hit, or a new key with room
// there); entries that need more than that wait in the warp's segment of a per-CTA queue in global
// memory and are settled, 32 per round, once the warp's share of the stream is through (or earlier,
// when the segment could not take another batch); then write the deltas back.
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Shared-window addresses of the partition pass's arrays: keys ull[C] (the pass's own key form, 0 =
// empty), acc {u32 low limb, u32 count | NEW_KEY_FLAG}[C], a1 u32[C] (high limb).
struct PartSmem {
    uint32_t keys, acc, a1;
};

__device__ __forceinline__ uint4 lds_v4u32(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}

// General probe, one entry per lane (busy = this lane has one): walks the key's probe sequence from
// the pair at `slot`, claims the first free slot if the key is not there.  Warp-convergent.  Returns
// the key's slot, or PROBE_FAILED when the partition has no room.
constexpr uint32_t PROBE_FAILED = 0xFFFFFFFFu;

__device__ __forceinline__ uint32_t probe_general(const PartSmem& m, ull skey, uint32_t slot, uint32_t advance, bool busy,
                                                  uint32_t C, Control* ctl) {
    uint32_t steps = 0;
    while (__any_sync(0xFFFFFFFFu, busy)) {
        if (busy) {
            const ulonglong2 kk = lds_v2u64(m.keys + ATREX_INDEX(slot, C - 1u, ctl) * 8);
            const bool hit1 = kk.y == skey;
            if (kk.x == skey || hit1) {
                slot += hit1 ? 1u : 0u;
                busy = false;
            } else if (kk.x == 0 || kk.y == 0) {
                // claim the first empty slot of the pair; a lost race re-reads the pair
                const uint32_t at = slot + (kk.x == 0 ? 0u : 1u);
                const ull old = atoms_cas64(m.keys + at * 8, 0ull, skey);
                if (old == 0) reds_or(m.acc + at * 8 + 4, NEW_KEY_FLAG);
                if (old == 0 || old == skey) {
                    slot = at;
                    busy = false;
                }
            } else {
                slot += advance;
                if (slot >= C) slot -= C;
            }
            if (busy && ++steps > 2 * C) {  // partition full (bounded; counts lost races too)
                busy = false;
                slot = PROBE_FAILED;
                atomicOr(&ctl->status, ST_TABLE_FULL);
                atomicAdd(&ctl->n_dropped, 1ull);
            }
        }
    }
    return slot;
}

// A slot whose high limb filled up: its sums move to HBM (this CTA owns the slot, so those adds are
// exact; the write-back adds on top).  Rare, hence not inlined.
__device__ __noinline__ void part_drain_slot(uint32_t acc, uint32_t a1, ulonglong2* val) {
    ull hi, lo = limbs_drain(acc, a1, &hi);
    ull* vp = reinterpret_cast<ull*>(val);
    ull old = atomicAdd(vp, lo);
    hi += (old + lo < old) ? 1ull : 0ull;
    if (hi) atomicAdd(vp + 1, hi << HI_SHIFT);
}

// One entry's product (vlo + 2^32 vhi, vhi < 2^16) and count into its slot's limbs: a returning add on
// the low limb, whose wrap is the carry; the high limb is touched only when there is something to add.
__device__ __forceinline__ void part_accumulate(const PartSmem& m, uint32_t slot, uint32_t vlo, uint32_t vhi,
                                                ulonglong2* vals_of_partition, uint32_t C, Control* ctl) {
    slot = ATREX_INDEX(slot, C, ctl);
    const uint32_t acc = m.acc + slot * 8;
    const uint32_t o0 = atoms_add(acc, vlo);
    reds_add(acc + 4, 1u);
    const uint32_t x = vhi + ((o0 + vlo < o0) ? 1u : 0u);
    if (x != 0) {
        const uint32_t o1 = atoms_add(m.a1 + slot * 4, x);
        if (((o1 + x) & ~o1 & DRAIN_BIT) != 0) part_drain_slot(acc, m.a1 + slot * 4, vals_of_partition + slot);
    }
}

// The first 256 entries (24 lines) of sub-buffer `sb` towards L2, as far as it holds that many.
__device__ __forceinline__ void prefetch_entries(const PartitionParams& q, ull sb, uint32_t lane) {
    const uint32_t bytes = q.spill_cnt[sb] * SPILL_ENTRY_BYTES;
    if (lane < 24 && lane * 128u < bytes) prefetch_l2(q.spill + sb * q.cap * SPILL_ENTRY_BYTES + lane * 128u);
}

// Settles a warp's queued entries, one per lane and round, by the general probe.  Other warps may
// still be streaming: the probe copes with keys that appear meanwhile.  Called once the warp's share of
// the partition's stream is through, and before a batch that might not fit the queue (a crowded
// partition of new keys).  Not inlined: it runs a few times per partition and warp.
__device__ __noinline__ void settle_queue(const TableRef t, const PartSmem m, const ulonglong2* my_queue, uint32_t qn_w, uint32_t C,
                                          ull base, uint32_t lane);

// A queued entry: {key, product}; bit 63 of the product word says that the key's first pair was full
// of other keys when the entry was looked up, so its probe may start at the second pair.
constexpr ull QUEUED_SKIP_FIRST = 1ull << 63;

// One batch of 128 entries of a sub-buffer, four consecutive ones (48 bytes) per lane.  FULL: the
// batch is complete (no masks).  Keys are handled as their two 32-bit halves (kh: mark, phase,
// operator; kl: hash).  Entry state is bit sets per lane -- `open` (present, slot not known yet), `hit`
// (slot known), `room` (the first pair of the probe sequence had a free slot when it was read).
// part_bits = the partition's index in the hash's top bits, hmask = the hash bits below them.
template <bool FULL>
__device__ __forceinline__ void stream_batch(const PartitionParams& q, const PartSmem& m, const unsigned char* src,
                                             uint32_t part_bits, uint32_t hmask, uint32_t e0, uint32_t n_e, uint32_t C, ull base,
                                             ulonglong2* my_queue, uint32_t queue_cap_w, uint32_t& qn_w, uint32_t lane) {
    uint32_t kh[4], kl[4], vlo[4], vhi[4], slot[4];
    uint32_t open = 0;
    {
        // the lane's entries e, e + 1, e + 2, e + 3 (e a multiple of 4) as twelve words; in an even
        // entry the 8-byte word comes first, in an odd one last.  A buffer's capacity is a multiple
        // of 4, so a lane that holds any entry may read all 48 bytes.
        const uint32_t e = e0 + 4u * lane;
        uint4 w[3];
        if (FULL || e < n_e) {
            const uint4* at = reinterpret_cast<const uint4*>(src + (size_t)e * SPILL_ENTRY_BYTES);
#pragma unroll
            for (int j = 0; j < 3; ++j) w[j] = __ldcs(at + j);
            open = FULL ? 0xFu : (0xFu >> (4u - min(n_e - e, 4u)));
        } else {
#pragma unroll
            for (int j = 0; j < 3; ++j) w[j] = make_uint4(0, 0, 0, 0);
        }
        const uint32_t alo[4] = {w[0].x, w[1].x, w[1].z, w[2].z}, ahi[4] = {w[0].y, w[1].y, w[1].w, w[2].w};
        const uint32_t b[4] = {w[0].z, w[0].w, w[2].x, w[2].y};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            kh[u] = 0x80000000u | ((b[u] >> 8) & 0x00FF0000u) | (ahi[u] >> 16);
            kl[u] = part_bits | (b[u] & hmask);
            vlo[u] = alo[u];
            vhi[u] = ahi[u] & 0xFFFFu;
            slot[u] = local_of(kl[u], b[u] >> 24, C) & ~1u;  // first pair of the probe sequence
        }
    }
    // First look, straight-line for all four entries: most keys sit in the first pair of slots of
    // their probe sequence.  (Pairs fill from the even slot, and slots never empty again.)
    uint32_t hit = 0, room = 0, even_taken = 0;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const uint4 kk = lds_v4u32(m.keys + ATREX_INDEX(slot[u], C - 1u, q.t.ctl) * 8);
        const bool h0 = kk.x == kl[u] && kk.y == kh[u];
        const bool h1 = kk.z == kl[u] && kk.w == kh[u];
        if (h1) slot[u] |= 1u;
        if (h0 || h1) hit |= 1u << u;
        if (kk.w == 0) room |= 1u << u;
        if (kk.y != 0) even_taken |= 1u << u;
    }
    hit &= open;     // (an absent entry is a well-formed key too)
    open &= ~hit;
    // A new key whose first pair has room is inserted at once, so that its later occurrences find it
    // there; a slot lost to another key defers the entry.
    if (__any_sync(0xFFFFFFFFu, (open & room) != 0)) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (open & room & (1u << u)) {
                const uint32_t at = slot[u] + ((even_taken >> u) & 1u);
                const ull skey = ((ull)kh[u] << 32) | kl[u];
                const ull old = atoms_cas64(m.keys + at * 8, 0ull, skey);
                if (old == 0) reds_or(m.acc + at * 8 + 4, NEW_KEY_FLAG);
                if (old == 0 || old == skey) {
                    slot[u] = at;
                    hit |= 1u << u;
                    open &= ~(1u << u);
                }
            }
        }
    }
    if (__any_sync(0xFFFFFFFFu, open != 0)) {
        // The rest (keys further down their probe sequence, lost races: a few per batch) is not settled
        // here, where the fixed cost of a general probe round would be paid for a handful of entries: it
        // goes to this warp's queue and is settled by settle_queue, 32 entries per warp round.
        uint32_t before[4], total = 0;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t pend = __ballot_sync(0xFFFFFFFFu, (open >> u) & 1u);
            before[u] = total + __popc(pend & ((1u << lane) - 1u));
            total += __popc(pend);
        }
        // (the caller settles the queue before a batch that might not fit: there is room for all 128)
        const uint32_t qbase = qn_w;
        qn_w += total;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (open & (1u << u)) {
                const ull v = vlo[u] | ((ull)vhi[u] << 32) | ((room >> u) & 1u ? 0ull : QUEUED_SKIP_FIRST);
                my_queue[ATREX_INDEX(qbase + before[u], queue_cap_w, q.t.ctl)] = make_ulonglong2(((ull)kh[u] << 32) | kl[u], v);
            }
        }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
        if (hit & (1u << u)) part_accumulate(m, slot[u], vlo[u], vhi[u], q.t.vals + base, C, q.t.ctl);
}

__device__ __noinline__ void settle_queue(const TableRef t, const PartSmem m, const ulonglong2* my_queue, uint32_t qn_w, uint32_t C,
                                          ull base, uint32_t lane) {
    __syncwarp();   // the queue was written by other lanes of this warp
    for (uint32_t i0 = 0; i0 < qn_w; i0 += 32u) {
        const bool serving = i0 + lane < qn_w;
        const ulonglong2 ent = serving ? __ldcg(my_queue + i0 + lane) : make_ulonglong2(0, 0);
        const uint32_t hh = (uint32_t)ent.x;
        const uint32_t advance = 2u * stride_of(t, stride_index(hh));
        uint32_t start = local_of(hh, ckey_phase(ent.x), C) & ~1u;
        if (ent.y & QUEUED_SKIP_FIRST) {
            start += advance;
            if (start >= C) start -= C;
        }
        const uint32_t found = probe_general(m, ent.x, start, advance, serving, C, t.ctl);
        if (serving && found != PROBE_FAILED)
            part_accumulate(m, found, (uint32_t)ent.y, (uint32_t)(ent.y >> 32) & 0xFFFFu, t.vals + base, C, t.ctl);
    }
    __syncwarp();   // the queue may be overwritten from here on
}

__global__ void __launch_bounds__(INGEST_THREADS, 1) partition_kernel(PartitionParams q) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t C = q.t.C;
    ull* s_keys = reinterpret_cast<ull*>(smem_raw);
    uint2* s_acc = reinterpret_cast<uint2*>(s_keys + C);      // {low limb, count | NEW_KEY_FLAG}
    uint32_t* s_a1 = reinterpret_cast<uint32_t*>(s_acc + C);  // high limb
    PartSmem m;
    m.keys = smem_addr(s_keys);
    m.acc = smem_addr(s_acc);
    m.a1 = smem_addr(s_a1);
    __shared__ uint32_t s_total;
    // each warp owns a segment of the CTA's queue: no shared counter, and a warp can settle its own
    // leftovers as soon as its share of the stream is through
    const uint32_t queue_cap_w = q.queue_cap / (INGEST_THREADS / 32);
    ulonglong2* const my_queue = q.queue + (size_t)blockIdx.x * q.queue_cap + (size_t)(threadIdx.x >> 5) * queue_cap_w;
    const uint32_t n_parts = 1u << q.t.lp;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u, n_warps = blockDim.x >> 5;
    // the spill buffers are drained lazily: unless forced, only when the scatter launch just
    // before this one found a buffer filling up
    if (!q.force && ld_relaxed(&q.t.ctl->drain_seq) != q.seq) return;
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicAdd(&q.t.ctl->n_drains, 1ull);

    // Partitions are handed out by a counter (their entry counts differ by a few per cent, and a static
    // split leaves the kernel waiting for its slowest CTA); a CTA always holds its next partition as
    // well, so that it can pull that one's keys and entries towards L2 early.
    __shared__ uint32_t s_next;
    if (blockIdx.x >= n_parts) return;                             // (never: at least 256 partitions)
    if (threadIdx.x == 0) s_next = (uint32_t)atomicAdd(&q.t.ctl->part_cursor, 1ull);
    uint32_t part = blockIdx.x;                                     // the first round is the static one
    while (part < n_parts) {
        __syncthreads();  // s_next is set; the previous partition's write-back has finished reading shared memory
        const uint32_t next = gridDim.x + s_next;                   // the counter starts at 0: partitions >= gridDim
        __syncthreads();
        if (threadIdx.x == 0) {
            s_total = 0;
            s_next = (uint32_t)atomicAdd(&q.t.ctl->part_cursor, 1ull);
        }
        __syncthreads();
        uint32_t local_total = 0;
        for (uint32_t g = threadIdx.x; g < q.n_used; g += blockDim.x) local_total += q.spill_cnt[((ull)g << q.t.lp) + part];
        local_total = __reduce_add_sync(0xFFFFFFFFu, local_total);
        if (lane == 0 && local_total) atomicAdd(&s_total, local_total);

        __syncthreads();
        if (s_total == 0) {  // nothing was spilled to this partition (uniform)
            part = next;
            continue;
        }

        const ull base = (ull)part * C;
        for (uint32_t i0 = threadIdx.x; i0 < C; i0 += 4 * blockDim.x) {  // four key loads per thread in flight
            ull k[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) k[u] = i0 + u * blockDim.x < C ? q.t.keys[base + i0 + u * blockDim.x] : 0ull;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t i = i0 + u * blockDim.x;
                if (i < C) {
                    s_keys[i] = k[u] == 0 ? 0ull : ckey_of_key(~k[u]);   // the table stores complemented keys, 0 = empty
                    s_acc[i] = make_uint2(0, 0);
                    s_a1[i] = 0;
                }
            }
        }
        {   // the accumulators of this partition are read back at the end: start them towards L2 now
            const unsigned char* vb = reinterpret_cast<const unsigned char*>(q.t.vals + base);
            for (uint32_t off = threadIdx.x * 128u; off < C * 16u; off += blockDim.x * 128u) prefetch_l2(vb + off);
        }
        __syncthreads();

        const uint32_t part_bits = part << (32 - q.t.lp), hmask = 0xFFFFFFFFu >> q.t.lp;
        uint32_t qn_w = 0;  // entries in this warp's queue segment (warp-uniform)
        for (uint32_t g = warp; g < q.n_used; g += n_warps) {
            const ull sb = ((ull)g << q.t.lp) + part;
            const uint32_t n_e = q.spill_cnt[sb];
            const unsigned char* buf = q.spill + sb * q.cap * SPILL_ENTRY_BYTES;
            // Short-distance L2 prefetch, a fixed window of 256 entries per warp (a longer reach gets
            // evicted before use: all warps of all CTAs together must stay well inside L2): the head of
            // this warp's next sub-buffer now, and inside the loop the lines two batches ahead.
            if (g + n_warps < q.n_used) prefetch_entries(q, ((ull)(g + n_warps) << q.t.lp) + part, lane);
            for (uint32_t e0 = 0; e0 < n_e; e0 += 128) {
                if (lane < 12 && (e0 + 256u) * SPILL_ENTRY_BYTES + lane * 128u < n_e * SPILL_ENTRY_BYTES)
                    prefetch_l2(buf + (e0 + 256u) * SPILL_ENTRY_BYTES + lane * 128u);
                if (qn_w + 128u > queue_cap_w) {   // (warp-uniform) the next batch might not fit the queue
                    settle_queue(q.t, m, my_queue, qn_w, C, base, lane);
                    qn_w = 0;
                }
                if (e0 + 128u <= n_e)
                    stream_batch<true>(q, m, buf, part_bits, hmask, e0, n_e, C, base, my_queue, queue_cap_w, qn_w, lane);
                else
                    stream_batch<false>(q, m, buf, part_bits, hmask, e0, n_e, C, base, my_queue, queue_cap_w, qn_w, lane);
            }
        }
        settle_queue(q.t, m, my_queue, qn_w, C, base, lane);
        __syncthreads();
        {   // while the deltas are written back, pull the next partition's keys and each warp's
            // first sub-buffer towards L2 (used within microseconds, so they are still there)
            if (next < n_parts) {
                const unsigned char* nk = reinterpret_cast<const unsigned char*>(q.t.keys + (ull)next * C);
                for (uint32_t off = threadIdx.x * 128u; off < C * 8u; off += blockDim.x * 128u) prefetch_l2(nk + off);
                if (warp < q.n_used) prefetch_entries(q, ((ull)warp << q.t.lp) + next, lane);
            }
        }
        // read-modify-write of the touched slots, four per thread in flight (the loads miss L1 by
        // design and mostly come from L2, where the prefetch at the start of the partition put them)
        for (uint32_t i0 = threadIdx.x; i0 < C; i0 += 4 * blockDim.x) {
            uint2 c[4];   // {low limb, count | NEW_KEY_FLAG}
            ulonglong2 old[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t i = i0 + u * blockDim.x;
                c[u] = i < C ? s_acc[i] : make_uint2(0, 0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                old[u] = make_ulonglong2(0, 0);
                if (c[u].y) {
                    const ull* vp = reinterpret_cast<const ull*>(q.t.vals + base + i0 + u * blockDim.x);
                    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(old[u].x), "=l"(old[u].y) : "l"(vp));
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (c[u].y == 0) continue;
                const uint32_t i = i0 + u * blockDim.x;
                const ull nlo = old[u].x + ((ull)c[u].x | ((ull)s_a1[i] << 32));
                const ull cnthi = old[u].y + (ull)(c[u].y & ~NEW_KEY_FLAG) + ((nlo < old[u].x ? 1ull : 0ull) << HI_SHIFT);
                q.t.vals[base + i] = make_ulonglong2(nlo, cnthi);
                if (c[u].y & NEW_KEY_FLAG) q.t.keys[base + i] = ~key_of_ckey(s_keys[i]);
            }
        }
        // this partition's buffers are empty again
        for (uint32_t g = threadIdx.x; g < q.n_used; g += blockDim.x) q.spill_cnt[((ull)g << q.t.lp) + part] = 0;
        part = next;
    }
}

// --------------------------------------------------------------------------------------
// Hot-directory construction, three small kernels over a strided sample of the records:
//   1. count   every sampled key bumps one of 2^20 counters chosen by its hash;
//   2. admit   sampled keys whose counter reached ADMIT_MIN are inserted, with exact counts,
//              into a candidate table (colliding cold keys may slip in; harmless);
//   3. select  one CTA picks the count threshold that fills the directory and installs the
//              candidates, most frequent classes first, into 4-slot buckets.
// Which keys end up in the directory only affects speed, never results.
constexpr uint32_t SKETCH_BITS = 20;   // as many counters as samples, so that cold keys stay below ADMIT_MIN
constexpr uint32_t ADMIT_MIN = 3;
constexpr uint32_t CAND_PROBES = 16;

__device__ __forceinline__ bool sample_key(const HotBuildParams& p, uint32_t j, ull* key) {
    uint4 v = p.recs[(ull)j * p.stride];
    uint32_t khi = v.y & 0x00FFFFFFu;
    *key = ((ull)khi << 32) | v.z;
    return v.x < p.n_apps && (khi >> 16) < p.n_phases;
}

// Lanes of a warp that target the same counter are combined first, so that a trace dominated
// by one key does not serialise on one address.
__device__ __forceinline__ void combined_count(uint32_t* counters, uint32_t index, bool active) {
    unsigned act = __ballot_sync(0xFFFFFFFFu, active);
    if (!active) return;
    unsigned same = __match_any_sync(act, index);
    if ((threadIdx.x & 31u) == (unsigned)(__ffs(same) - 1)) atomicAdd(&counters[index], (uint32_t)__popc(same));
}

__global__ void __launch_bounds__(256) hot_count_kernel(HotBuildParams p) {
    const uint32_t stride = gridDim.x * blockDim.x;
    const uint32_t rounds = (p.n_sample + stride - 1) / stride;  // uniform trip count: warp collectives inside
    for (uint32_t r = 0; r < rounds; ++r) {
        uint32_t j = r * stride + blockIdx.x * blockDim.x + threadIdx.x;
        ull key = 0;
        bool ok = j < p.n_sample && sample_key(p, j, &key);
        combined_count(p.sketch, hash32(key) >> (32 - SKETCH_BITS), ok);
    }
}

__global__ void __launch_bounds__(256) hot_admit_kernel(HotBuildParams p) {
    const uint32_t stride = gridDim.x * blockDim.x;
    const uint32_t rounds = (p.n_sample + stride - 1) / stride;
    for (uint32_t r = 0; r < rounds; ++r) {
        uint32_t j = r * stride + blockIdx.x * blockDim.x + threadIdx.x;
        ull key = 0;
        bool ok = j < p.n_sample && sample_key(p, j, &key);
        uint32_t h = hash32(key);
        ok = ok && p.sketch[h >> (32 - SKETCH_BITS)] >= ADMIT_MIN;
        const ull skey = ~key;
        uint32_t s = (h * 0x9E3779B1u) >> (32 - p.cand_bits);
        bool found = false;
        if (ok) {
            for (uint32_t probe = 0; probe < CAND_PROBES && !found; ++probe) {
                ull k = ld_relaxed(&p.cand_keys[s]);
                if (k == 0) {
                    k = atomicCAS(&p.cand_keys[s], 0ull, skey);
                    if (k == 0) k = skey;
                }
                if (k == skey)
                    found = true;
                else
                    s = (s + 1) & ((1u << p.cand_bits) - 1);
            }
        }
        combined_count(p.cand_cnt, s, found);
    }
}

constexpr uint32_t SELECT_MAX = 14336;  // candidates kept for installation (directory <= 11.6K slots, x1.25)
constexpr uint32_t OCC_MAX = 3072;      // directory buckets (<= 11.6K / 4)
constexpr size_t SELECT_SMEM = (size_t)SELECT_MAX * 12 + (size_t)OCC_MAX * 4;

__global__ void __launch_bounds__(1024, 1) hot_select_kernel(HotBuildParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ull* c_key = reinterpret_cast<ull*>(smem_raw);                        // [SELECT_MAX]
    uint32_t* c_cnt = reinterpret_cast<uint32_t*>(c_key + SELECT_MAX);    // [SELECT_MAX]
    __shared__ uint32_t hist[1024];
    __shared__ uint32_t s_thr, s_inserted, s_max, s_n;
    const uint32_t n_cand = 1u << p.cand_bits;
    hist[threadIdx.x] = 0;
    for (uint32_t i = threadIdx.x; i < p.hot_slots; i += blockDim.x) p.hot_keys[i] = 0;
    if (threadIdx.x == 0) s_inserted = s_max = s_n = 0;
    __syncthreads();
    // one CTA walks the candidate table: eight independent loads per thread at a time, or the scan
    // is a chain of dependent memory round trips
    constexpr int SCAN_ILP = 8;
    for (uint32_t i0 = threadIdx.x; i0 < n_cand; i0 += SCAN_ILP * blockDim.x) {
        uint32_t c[SCAN_ILP];
#pragma unroll
        for (int u = 0; u < SCAN_ILP; ++u) c[u] = i0 + u * blockDim.x < n_cand ? p.cand_cnt[i0 + u * blockDim.x] : 0u;
#pragma unroll
        for (int u = 0; u < SCAN_ILP; ++u) {
            if (c[u] != 0) atomicAdd(&hist[min(c[u], 1023u)], 1u);
            if (c[u] >= 1023u) atomicMax(&s_max, c[u]);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        // smallest threshold >= 2 whose class fits the directory with some over-subscription
        uint32_t budget = min(p.hot_slots + p.hot_slots / 4, SELECT_MAX), cum = 0, thr = 1024;
        for (int c = 1023; c >= 2; --c) {
            if (cum + hist[c] > budget) break;
            cum += hist[c];
            thr = (uint32_t)c;
        }
        s_thr = thr;
        // a key holding more than 1/32 of the sample makes same-slot collisions inside a warp
        // common: tell the scatter pass to combine equal lanes first
        p.ctl->hot_skew = ((ull)s_max * 32u >= p.n_sample) ? 1ull : 0ull;
    }
    __syncthreads();
    const uint32_t thr = s_thr;
    // compact the selected candidates into shared memory, then install them class by class
    for (uint32_t i0 = threadIdx.x; i0 < n_cand; i0 += SCAN_ILP * blockDim.x) {
        uint32_t c[SCAN_ILP];
        ull k[SCAN_ILP];
#pragma unroll
        for (int u = 0; u < SCAN_ILP; ++u) c[u] = i0 + u * blockDim.x < n_cand ? p.cand_cnt[i0 + u * blockDim.x] : 0u;
#pragma unroll
        for (int u = 0; u < SCAN_ILP; ++u) k[u] = c[u] >= thr ? p.cand_keys[i0 + u * blockDim.x] : 0ull;
#pragma unroll
        for (int u = 0; u < SCAN_ILP; ++u) {
            if (c[u] >= thr) {
                uint32_t at = atomicAdd(&s_n, 1u);
                if (at < SELECT_MAX) {
                    c_key[at] = k[u];
                    c_cnt[at] = c[u];
                }
            }
        }
    }
    __syncthreads();
    const uint32_t n_sel = min(s_n, SELECT_MAX);
    // pick the bucket-hash multiplier that loses the least sampled weight: a key is lost when
    // its bucket's slots are already taken (approximated by arrival order among the keys that
    // matter, which is close to what the class-ordered installation below does)
    __shared__ uint32_t s_lost[4];
    uint32_t* occupancy = c_cnt + SELECT_MAX;  // [OCC_MAX] bucket counters behind the compact lists
    const uint32_t n_buckets = p.hot_slots / DIR_WAYS;
    if (threadIdx.x < 4) s_lost[threadIdx.x] = 0;
    for (uint32_t m = 0; m < 4; ++m) {
        for (uint32_t i = threadIdx.x; i < n_buckets; i += blockDim.x) occupancy[i] = 0;
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < n_sel; i += blockDim.x) {
            uint32_t c = c_cnt[i];
            if (c < 16) continue;
            uint32_t b = dir_bucket_of_key(~c_key[i], DIR_MULTS[m], n_buckets);
            if (atomicAdd(&occupancy[b], 1u) >= DIR_WAYS) atomicAdd(&s_lost[m], c);
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        uint32_t best = 0;
        for (uint32_t m = 1; m < 4; ++m)
            if (s_lost[m] < s_lost[best]) best = m;
        p.ctl->dir_mult = DIR_MULTS[best];
        s_thr = DIR_MULTS[best];  // broadcast (the threshold is already in registers)
    }
    __syncthreads();
    const uint32_t mult = s_thr;
    for (uint32_t i = threadIdx.x; i < n_buckets; i += blockDim.x) occupancy[i] = 0;
    __syncthreads();
    // install from the most to the least frequent class (counts within a class differ < 2x), so
    // that a key can only lose its bucket to keys about as frequent as itself; a bucket's ways are
    // handed out by its shared-memory counter
    for (int round = 0; round < 11; ++round) {
        uint32_t hi = round == 0 ? 0xFFFFFFFFu : (2048u >> round), lo = max(1024u >> round, thr);
        if (lo < hi) {
            for (uint32_t i = threadIdx.x; i < n_sel; i += blockDim.x) {
                uint32_t c = c_cnt[i];
                if (c >= lo && c < hi) {
                    ull skey = c_key[i];
                    const uint32_t b = dir_bucket_of_key(~skey, mult, n_buckets);
                    const uint32_t way = atomicAdd(&occupancy[b], 1u);
                    if (way < DIR_WAYS) {
                        p.hot_keys[b * DIR_WAYS + way] = skey;
                        atomicAdd(&s_inserted, 1u);
                    }
                }
            }
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) p.ctl->hot_n = s_inserted;
}

// --------------------------------------------------------------------------------------
// Merge of already aggregated units into the table.
__global__ void __launch_bounds__(256) merge_kernel(const atrex_entry_t* in, ull n, TableRef t) {
    for (ull i = (ull)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (ull)gridDim.x * blockDim.x) {
        atrex_entry_t e = in[i];
        table_accumulate(t, e.key, hash32(e.key), e.wt_lo, e.wt_hi, e.count);
    }
}

// --------------------------------------------------------------------------------------
// host launchers

cudaError_t ingest_prepare() {
    cudaError_t e = scatter_prepare();
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(partition_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448 - 2048);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(hot_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SELECT_SMEM);
}

cudaError_t launch_partition(const PartitionParams& q, int n_sms, cudaStream_t stream) {
    int grid = (int)(1u << q.t.lp) < n_sms ? (int)(1u << q.t.lp) : n_sms;
    partition_kernel<<<grid, INGEST_THREADS, (size_t)q.t.C * 20, stream>>>(q);
    return cudaGetLastError();
}

cudaError_t launch_hot_build(const HotBuildParams& p, int n_sms, cudaStream_t stream) {
    // the caller has zeroed the sketch and the candidate table on this stream
    int grid = (int)((p.n_sample + 255) / 256);
    if (grid > n_sms * 8) grid = n_sms * 8;
    hot_count_kernel<<<grid, 256, 0, stream>>>(p);
    hot_admit_kernel<<<grid, 256, 0, stream>>>(p);
    hot_select_kernel<<<1, 1024, SELECT_SMEM, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_hot_fold(const ull* hot_keys, ulonglong2* hot_img, uint32_t n_groups, uint32_t hot_slots,
                            const TableRef& t, cudaStream_t stream) {
    if (hot_slots == 0) return cudaSuccess;
    hot_fold_kernel<<<(hot_slots + 31) / 32, FOLD_WARPS * 32, 0, stream>>>(hot_keys, hot_img, n_groups, hot_slots, t);
    return cudaGetLastError();
}

cudaError_t launch_merge(const atrex_entry_t* in, ull n, const TableRef& t, int grid, cudaStream_t stream) {
    merge_kernel<<<grid, 256, 0, stream>>>(in, n, t);
    return cudaGetLastError();
}

}  // namespace atrex
