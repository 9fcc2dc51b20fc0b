// Pass 1 of the ingest (Eq. 2's group-by sum, streamed): SCATTER, one persistent CTA per SM.
//
// Each thread pulls records with 32-byte vector loads (two 16-byte records per load, three loads
// rotating per thread so that two are in flight while one is consumed, streaming cache policy),
// validates, packs the key and multiplies the application's card-hour weight by the duration.
//   * Keys found in the shared-memory HOT DIRECTORY (the most frequent keys of a sample of the
//     trace, identical in every CTA, read-only during the pass) are accumulated on the spot with
//     32-bit shared-memory atomics in limbs with explicit carries.
//   * Every other record becomes a 12-byte entry {product, operator, phase, hash bits} appended to
//     the CTA's private buffer of the key's partition (see spill_append).
// At the end the CTA adds its directory accumulators to its own row of a directory image
// ([CTA][slot], plain coalesced read-modify-writes; hot_fold_kernel adds the rows into the table
// before results are read) and stores its per-partition cursors: the buffers persist across launches
// until the partition pass drains them.
//
// The kernel runs out of issue slots, shared-memory pipe cycles and latency-hiding warps long before
// it runs out of DRAM bandwidth, so the hot loop is written for a low instruction count: the shared-memory layout is a compile-time function
// of the partition count (every array address is a register plus an immediate), rarely taken
// branches (products of 2^48 and more, a full buffer, a drain of a directory slot) are calls to functions that are not inlined, and the three load buffers rotate by
// name instead of being copied.
#include "atrex_dev.cuh"
#include "kernels.h"

namespace atrex {

namespace {

#ifndef ATREX_SCATTER_THREADS
#define ATREX_SCATTER_THREADS 1024
#endif
constexpr int SCATTER_THREADS = ATREX_SCATTER_THREADS;
constexpr uint32_t NO_SLOT = 0xFFFFFFFFu;
constexpr uint32_t DIR_WAYS = 4;

// Shared-memory map of the scatter pass for 2^LP partitions (byte offsets into the dynamic shared memory).
template <uint32_t LP>
struct Smem {
    static constexpr uint32_t P = 1u << LP;
    static constexpr uint32_t SLOTS = scatter_hot_slots(LP);   // directory slots, whole 4-way buckets
    static constexpr uint32_t NB = SLOTS / DIR_WAYS;
    static constexpr uint32_t RING = 0;                         // record ring: SCATTER_RING_STAGES tiles
    static constexpr uint32_t CUR = RING + SCATTER_RING_STAGES * SCATTER_RING_TILE;   // u32[P]  entries appended to this CTA's buffer of each partition
    static constexpr uint32_t APPW = CUR + 4u * P;              // u32[APPW_SMEM_MAX]  card-hour weights
    static constexpr uint32_t TAG = APPW + 4u * APPW_SMEM_MAX;  // u32[NB + 1]  four 8-bit tags per bucket (+ one pad bucket)
    static constexpr uint32_t KEYS = (TAG + 4u * (NB + 1u) + 7u) & ~7u;   // ull[SLOTS + 4]  key, all ones = empty
    static constexpr uint32_t ACC = KEYS + 8u * (SLOTS + DIR_WAYS);       // {u32 lo, u32 hi, u32 count}[SLOTS + 4]
    static constexpr uint32_t TOTAL = ACC + 12u * (SLOTS + DIR_WAYS);
    static_assert(TOTAL <= SCATTER_SMEM_BYTES, "scatter pass shared memory");
    static_assert(SLOTS % 32 == 0, "whole buckets");
};

__device__ __forceinline__ void ld_stream_256(const void* p, uint32_t (&w)[8]) {
    asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(p));
}
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// Loads of the directory's tags and keys and of the weights: these arrays are read-only during the
// pass, so the loads are not volatile and the compiler may overlap the look-ups of several records.
__device__ __forceinline__ uint32_t lds_u32(uint32_t a) {
    uint32_t v;
    asm("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ ull lds_u64(uint32_t a) {
    ull v;
    asm("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(a));
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
__device__ __forceinline__ uint32_t atoms_exch(uint32_t a, uint32_t v) {
    uint32_t o;
    asm volatile("atom.shared.exch.b32 %0, [%1], %2;" : "=r"(o) : "r"(a), "r"(v) : "memory");
    return o;
}
// What the hot loop keeps in registers (everything else is read from the kernel's parameter block,
// i.e. straight from the constant bank).
struct Ctx {
    uint32_t sb;              // shared-window address of the dynamic shared memory
    uint32_t mult;            // bucket-hash multiplier of this directory image
    unsigned char* my_spill;  // this CTA's buffers
    ull keep;                 // L2 cache policy of the spill stores: evict last
};

// (rare) counters of invalid records and of records that found their buffer full
__device__ __noinline__ void count_one(ull* counter) { atomicAdd(counter, 1ull); }

// Shared-memory accumulation uses native 32-bit atomics only (64-bit shared atomics are
// compare-and-swap loops).  A slot's weighted time is kept in two limbs: the returning add on the
// low limb tells the adder whether it wrapped, and the adder then adds the carry, with the value's
// high word, to the high limb.  One add raises the high limb by at most 2^21 (a warp's combined 32
// records of < 2^48 each), so the adder that takes it across 2^30 drains both limbs; the adds that
// can slip in before its exchange (one per thread of the CTA) stay below 2^31, so the high limb
// never wraps.
constexpr uint32_t DRAIN_BIT = 0x40000000u;

// (rare) Moves a directory slot's limbs to the table.  The two exchanges need not be simultaneous:
// whatever lands between them stays in the limbs for the next drain or the final flush.
__device__ __noinline__ void drain_slot(TableRef t, uint32_t acc, ull key, uint32_t h) {
    const ull lo = atoms_exch(acc, 0u);
    const ull hi = atoms_exch(acc + 4, 0u);
    const ull v = lo + (hi << 32);
    table_accumulate(t, key, h, v, v < lo ? 1ull : 0ull, 0);
}

// (rare) A record that cannot take the limb route: straight to the table with full 64-bit adds.
__device__ __noinline__ void table_route(TableRef t, ull key, uint32_t h, ull prod) { table_accumulate(t, key, h, prod, 0, 1); }
// (rare) An invalid record is counted; a valid one whose product has bits at or above 2^48 goes to the table.
__device__ __noinline__ void rare_record(TableRef t, bool valid, ull key, uint32_t h, ull prod) {
    if (valid)
        table_accumulate(t, key, h, prod, 0, 1);
    else
        atomicAdd(&t.ctl->n_rejected, 1ull);
}

// Add (count, v) to a directory slot, v < 2^53, count <= 32.  Most products fit 32 bits and most
// low-limb adds do not wrap: the high limb is then left alone (one returning atomic and one reduction
// per hit instead of two and one).
template <uint32_t LP>
__device__ __forceinline__ void dir_add(const IngestParams& p, const Ctx& c, uint32_t slot, ull v, uint32_t count, ull key,
                                        uint32_t h) {
    const uint32_t acc = c.sb + Smem<LP>::ACC + ATREX_INDEX(slot, Smem<LP>::SLOTS, p.t.ctl) * 12u;
    const uint32_t v0 = (uint32_t)v;
    const uint32_t o0 = atoms_add(acc, v0);
    reds_add(acc + 8, count);
    const uint32_t x1 = (uint32_t)(v >> 32) + ((o0 + v0 < o0) ? 1u : 0u);
    if (x1 != 0) {
        const uint32_t o1 = atoms_add(acc + 4, x1);
        if ((o1 + x1) & ~o1 & DRAIN_BIT) drain_slot(p.t, acc, key, h);
    }
}

// (rare) The buffer is full: the ticket is handed back and the record takes the exact slow path.
template <uint32_t LP>
__device__ __noinline__ void spill_overflow(TableRef t, uint32_t cw, ull key, ull prod, uint32_t h) {
    reds_add(cw, 0xFFFFFFFFu);
    table_accumulate(t, key, h, prod, 0, 1);
    atomicAdd(&t.ctl->n_overflow, 1ull);
}

// Spill: the record becomes a 12-byte entry in this CTA's buffer of the key's partition -- an 8-byte
// word {product (48 bits), operator} and a 4-byte word {phase, the hash bits below the partition's}.
// Inside its partition (the hash's top bits) the triple (phase, operator, hash) identifies the key:
// for a given operator the hash is a bijection of the shape (shape_of_hash).
template <uint32_t LP>
__device__ __forceinline__ void spill_append(const IngestParams& p, Ctx& c, bool todo, uint32_t khi, uint32_t shape, ull prod,
                                             uint32_t h) {
    if (!todo) return;
    const uint32_t part = ATREX_INDEX(h >> (32 - LP), Smem<LP>::P, p.t.ctl);
    const uint32_t cw = c.sb + Smem<LP>::CUR + part * 4u;
    const uint32_t tk = atoms_add(cw, 1u);
    if (tk < p.cap) {
        // Entry tk occupies bytes [12 tk, 12 tk + 12) of the buffer; its 8-byte word sits at whichever
        // end is 8-byte aligned.  Two or three entries before the buffer reaches its next 128-byte
        // line, that line is pulled into L2 (a partial store into a line that is not cached stalls on a
        // fill), and the stores ask the L2 to evict their lines last: a buffer's current line is
        // written to some 20 times over ~40 K cycles while 16 GiB of records stream through the same cache.
        // (a CTA's buffers together stay below 4 GB: 2^12 partitions x 2^15 entries x 12 bytes)
        const uint32_t off = (part * p.cap + ATREX_INDEX(tk, p.cap, p.t.ctl)) * SPILL_ENTRY_BYTES;
        const uint32_t odd = tk & 1u;
        // word a = product | operator << 48, word b = phase << 24 | low hash bits, put together bytewise
        const uint32_t a_hi = __byte_perm((uint32_t)(prod >> 32), khi, 0x5410);
        const uint32_t b = __byte_perm(h & (0xFFFFFFFFu >> LP), khi, 0x6210);
        {   // one address: the entry's parity picks between two pairs of stores at immediate offsets (the
            // 8-byte word goes to the 8-byte aligned end), which is cheaper than computing two addresses
            unsigned char* at = c.my_spill + off;
            asm volatile(
                "{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %5, 0;\n\t"
                "@q  st.global.L2::cache_hint.u32 [%0], %3, %4;\n\t"
                "@q  st.global.L2::cache_hint.v2.u32 [%0+4], {%1, %2}, %4;\n\t"
                "@!q st.global.L2::cache_hint.v2.u32 [%0], {%1, %2}, %4;\n\t"
                "@!q st.global.L2::cache_hint.u32 [%0+8], %3, %4;\n\t}"
                ::"l"(at), "r"((uint32_t)prod), "r"(a_hi), "r"(b), "l"(c.keep), "r"(odd) : "memory");
            if ((off & 127u) - 96u < 12u) asm volatile("prefetch.global.L2 [%0+64];" ::"l"(at));
        }
    } else {
        spill_overflow<LP>(p.t, cw, ((ull)khi << 32) | shape, prod, h);
    }
}

// One record, start to finish (the register-staged loop has no registers to spare for working on
// two records at once).  Called by all lanes of a warp together (absent records masked by `present`).
template <uint32_t LP, bool HOT, bool DEDUPE, bool FULL>
__device__ __forceinline__ void one_record(const IngestParams& p, Ctx& c, uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3,
                                           bool present) {
    using L = Smem<LP>;
    const uint32_t khi = w1 & 0x00FFFFFFu;                  // phase << 16 | op_id: the key's high word
    bool ok = w0 < p.n_apps && khi < p.phase_lim;
    if (!FULL) ok = ok && present;
    // card-hour weight: from shared memory when the table fits there (an out-of-range index reads
    // some other weight, which is not used), else from global memory
    const uint32_t wgt = (p.appw_in_smem != 0) ? lds_u32(c.sb + L::APPW + (w0 & (APPW_SMEM_MAX - 1u)) * 4u) : __ldg(p.app_w + (ok ? w0 : 0u));
    const ull prod = (ull)wgt * (ull)w3;
    const uint32_t h = hash32(khi & 0xFFFFu, w2);
    const ull key = ((ull)khi << 32) | w2;
    // The limb arithmetic and the 12-byte spill entries assume products below 2^48 (e.g. weights
    // < 2^20, durations < 2^28).  Anything larger is still exact: straight to the table.  That and
    // the count of invalid records share one rarely taken branch (two separate ones cost the
    // configurations whose records mostly hit the directory 4-9 %).
    const bool todo_in = ok && (uint32_t)(prod >> 32) < 0x10000u;
    bool todo = todo_in;
    if ((FULL || present) && !todo_in) rare_record(p.t, ok, key, h, prod);
    if (HOT) {
        // Directory look-up: one 32-bit word per 4-slot bucket holds an 8-bit tag per slot (hash bits
        // the bucket choice does not use); the lowest slot whose tag matches is confirmed against the
        // 8-byte key.  A wrong tag match (1 in 64 look-ups) fails the confirmation and the record takes
        // the spill path: slower, still exact.
        const uint32_t x = dir_mix(h, khi >> 16, c.mult);
        const uint32_t b = ATREX_INDEX(__umulhi(x, L::NB), L::NB, p.t.ctl);
        const uint32_t t = lds_u32(c.sb + L::TAG + b * 4u) ^ __byte_perm(x, 0, 0);   // 0 in the bytes that match
        const uint32_t m = (t - 0x01010101u) & ~t & 0x80808080u;                      // lowest flagged byte is exact
        const uint32_t at = ATREX_INDEX(b * DIR_WAYS + ((uint32_t)__clz((int)__brev(m)) >> 3), L::SLOTS + DIR_WAYS, p.t.ctl);
        bool hit = todo && m != 0 && lds_u64(c.sb + L::KEYS + at * 8u) == key;
        if (DEDUPE) {
            // one key dominates the trace: combine the lanes that share the first hitting lane's slot
            const unsigned hits = __ballot_sync(0xFFFFFFFFu, hit);
            if (hits != 0) {
                const int lead = __ffs(hits) - 1;
                const uint32_t slot = hit ? at : NO_SLOT;
                const uint32_t ls = __shfl_sync(0xFFFFFFFFu, slot, lead);
                const unsigned same = __ballot_sync(0xFFFFFFFFu, slot == ls);
                if (__popc(same) >= 2 && slot == ls) {
                    const uint32_t s_lo = __reduce_add_sync(same, (uint32_t)prod & 0xFFFFFFu);
                    const uint32_t s_hi = __reduce_add_sync(same, (uint32_t)(prod >> 24));
                    if ((threadIdx.x & 31u) == (unsigned)lead)
                        dir_add<LP>(p, c, ls, (ull)s_lo + ((ull)s_hi << 24), (uint32_t)__popc(same), key, h);
                    hit = false;
                    todo = false;
                }
            }
        }
        if (hit) {
            dir_add<LP>(p, c, at, prod, 1u, key, h);
            todo = false;
        }
    }
    spill_append<LP>(p, c, todo, khi, w2, prod, h);
}

// The same for R records per lane at once (used with the shared-memory record ring, where the
// registers allow it; w[r] = the record's four words).  Called by all lanes of a
// warp together (absent records masked by `present`).  Written in stages over the R records so that
// their shared-memory round trips overlap: all look-ups are issued before the first result is used.
template <uint32_t LP, bool HOT, bool DEDUPE, bool FULL, int R>
__device__ __forceinline__ void process(const IngestParams& p, Ctx& c, const uint32_t (&w)[R][4], bool present) {
    using L = Smem<LP>;
    uint32_t khi[R], h[R], wgt[R], x[R], tags[R];
    bool todo[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        khi[r] = w[r][1] & 0x00FFFFFFu;                  // phase << 16 | op_id: the key's high word
        bool ok = w[r][0] < p.n_apps && khi[r] < p.phase_lim;
        if (!FULL) ok = ok && present;
        if ((FULL || present) && !ok) count_one(&p.t.ctl->n_rejected);
        todo[r] = ok;
        // card-hour weight: from shared memory when the table fits there (an out-of-range index reads
        // some other weight, which is not used), else from global memory
        wgt[r] = (p.appw_in_smem != 0) ? lds_u32(c.sb + L::APPW + (w[r][0] & (APPW_SMEM_MAX - 1u)) * 4u) : __ldg(p.app_w + (ok ? w[r][0] : 0u));
        h[r] = hash32(khi[r] & 0xFFFFu, w[r][2]);
        if (HOT) {
            // Directory look-up: one 32-bit word per 4-slot bucket holds an 8-bit tag per slot (hash
            // bits the bucket choice does not use)
            x[r] = dir_mix(h[r], khi[r] >> 16, c.mult);
            tags[r] = lds_u32(c.sb + L::TAG + __umulhi(x[r], L::NB) * 4u);
        }
    }
    ull prod[R];
    uint32_t at[R];
    ull found[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        prod[r] = (ull)wgt[r] * (ull)w[r][3];
        if (HOT) {
            // the lowest slot whose tag matches is confirmed against the 8-byte key; a wrong tag match
            // (1 in 64 look-ups) fails the confirmation and the record takes the spill path: slower,
            // still exact
            const uint32_t t = tags[r] ^ __byte_perm(x[r], 0, 0);                     // 0 in the bytes that match
            const uint32_t m = (t - 0x01010101u) & ~t & 0x80808080u;                  // lowest flagged byte is exact
            at[r] = __umulhi(x[r], L::NB) * DIR_WAYS + ((uint32_t)__clz((int)__brev(m)) >> 3);
            found[r] = ~0ull;
            if (m != 0) found[r] = lds_u64(c.sb + L::KEYS + at[r] * 8u);
        }
    }
    bool hit[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const ull key = ((ull)khi[r] << 32) | w[r][2];
        // The limb arithmetic and the 12-byte spill entries assume products below 2^48 (e.g. weights
        // < 2^20, durations < 2^28).  Anything larger is still exact: straight to the table.
        if (todo[r] && (uint32_t)(prod[r] >> 32) >= 0x10000u) {
            table_route(p.t, key, h[r], prod[r]);
            todo[r] = false;
        }
        hit[r] = HOT && todo[r] && found[r] == key;
    }
    if (HOT && DEDUPE) {
        // one key dominates the trace: combine the lanes that share the first hitting lane's slot
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const unsigned hits = __ballot_sync(0xFFFFFFFFu, hit[r]);
            if (hits == 0) continue;
            const int lead = __ffs(hits) - 1;
            const uint32_t slot = hit[r] ? at[r] : NO_SLOT;
            const uint32_t ls = __shfl_sync(0xFFFFFFFFu, slot, lead);
            const unsigned same = __ballot_sync(0xFFFFFFFFu, slot == ls);
            if (__popc(same) >= 2 && slot == ls) {
                const uint32_t s_lo = __reduce_add_sync(same, (uint32_t)prod[r] & 0xFFFFFFu);
                const uint32_t s_hi = __reduce_add_sync(same, (uint32_t)(prod[r] >> 24));
                if ((threadIdx.x & 31u) == (unsigned)lead)
                    dir_add<LP>(p, c, ls, (ull)s_lo + ((ull)s_hi << 24), (uint32_t)__popc(same), ((ull)khi[r] << 32) | w[r][2], h[r]);
                hit[r] = false;
                todo[r] = false;
            }
        }
    }
    if (HOT) {
        // hits: the returning low-limb adds of all R records first, then the rest
        uint32_t o0[R];
#pragma unroll
        for (int r = 0; r < R; ++r)
            if (hit[r]) o0[r] = atoms_add(c.sb + L::ACC + at[r] * 12u, (uint32_t)prod[r]);
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (hit[r]) {
                const uint32_t acc = c.sb + L::ACC + at[r] * 12u;
                const uint32_t v0 = (uint32_t)prod[r];
                reds_add(acc + 8, 1u);
                const uint32_t x1 = (uint32_t)(prod[r] >> 32) + ((o0[r] + v0 < o0[r]) ? 1u : 0u);
                if (x1 != 0) {
                    const uint32_t o1 = atoms_add(acc + 4, x1);
                    if ((o1 + x1) & ~o1 & DRAIN_BIT) drain_slot(p.t, acc, ((ull)khi[r] << 32) | w[r][2], h[r]);
                }
                todo[r] = false;
            }
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) spill_append<LP>(p, c, todo[r], khi[r], w[r][2], prod[r], h[r]);
}

template <uint32_t LP, bool HOT, bool DEDUPE>
__device__ __forceinline__ void scatter_body(const IngestParams& p, Ctx& c) {
    // CTA b handles record pairs (b + k * gridDim) * 1024 + tid, k = 0, 1, ...  Three 32-byte loads
    // rotate per thread: while one is consumed the next two are in flight.  Rounds in which every
    // CTA's tile is complete need no bounds checks; the last (ragged) ones are predicated.
    const unsigned char* body = reinterpret_cast<const unsigned char*>(p.body);
    const uint32_t stride = gridDim.x * SCATTER_THREADS;                  // pairs per round
    const uint32_t full_rounds = (uint32_t)(p.n_pairs / stride);
    const uint32_t rounds = (uint32_t)((p.n_pairs + stride - 1) / stride);
    const uint32_t first = blockIdx.x * SCATTER_THREADS + threadIdx.x;
    uint32_t bufA[8], bufB[8], bufC[8];
    auto fetch = [&](uint32_t round, uint32_t (&raw)[8]) {                // any round, bounds checked
        const ull i = first + (ull)round * stride;
        if (round < rounds && i < p.n_pairs) {
            ld_stream_256(body + i * 32, raw);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) raw[j] = 0;
        }
    };
    auto consume_full = [&](const uint32_t (&raw)[8]) {
        one_record<LP, HOT, DEDUPE, true>(p, c, raw[0], raw[1], raw[2], raw[3], true);
        one_record<LP, HOT, DEDUPE, true>(p, c, raw[4], raw[5], raw[6], raw[7], true);
    };
    auto consume_tail = [&](uint32_t round, const uint32_t (&raw)[8]) {
        const bool present = round < rounds && first + (ull)round * stride < p.n_pairs;
        one_record<LP, HOT, DEDUPE, false>(p, c, raw[0], raw[1], raw[2], raw[3], present);
        one_record<LP, HOT, DEDUPE, false>(p, c, raw[4], raw[5], raw[6], raw[7], present);
    };
    fetch(0, bufA);
    fetch(1, bufB);
    uint32_t round = 0;
    {
        // main part: every round fetched here is complete for every CTA, so the loads need no checks
        const unsigned char* next = body + (first + 2ull * stride) * 32;
        for (; round + 5 <= full_rounds; round += 3) {
            ld_stream_256(next, bufC);
            next += gridDim.x * (SCATTER_THREADS * 32u);
            consume_full(bufA);
            ld_stream_256(next, bufA);
            next += gridDim.x * (SCATTER_THREADS * 32u);
            consume_full(bufB);
            ld_stream_256(next, bufB);
            next += gridDim.x * (SCATTER_THREADS * 32u);
            consume_full(bufC);
        }
    }
    for (; round < rounds; round += 3) {
        fetch(round + 2, bufC);
        consume_tail(round, bufA);
        fetch(round + 3, bufA);
        consume_tail(round + 1, bufB);
        fetch(round + 4, bufB);
        consume_tail(round + 2, bufC);
    }
    // records that do not form an aligned pair (at most one before and one after the body)
    if (blockIdx.x == 0 && threadIdx.x < 32) {
        uint4 v = make_uint4(0, 0, 0, 0);
        const bool present = threadIdx.x < p.n_single;
        if (present) v = *reinterpret_cast<const uint4*>(threadIdx.x == 0 ? p.single[0] : p.single[1]);
        one_record<LP, HOT, DEDUPE, false>(p, c, v.x, v.y, v.z, v.w, present);
    }
}

// ---- shared-memory record ring (ATREX_SCATTER_RING stages) ----------------------------------------
// One warp of the CTA is the producer: a single lane issues one bulk asynchronous copy per tile of
// 992 records (this GPU's memory only, no multicast) into the next free stage and names the stage's
// "full" barrier as the copy's completion.  The other 31 warps are consumers: each thread reads its own
// record of two consecutive tiles (conflict-free 16-byte shared loads), the warp then releases the two
// stages on their "empty" barriers.  What the ring buys is registers: the records in flight live in
// shared memory, so a consumer thread holds only the two records it is working on.  Every wait is
// bounded; one that runs out latches ST_TIMEOUT, raises the CTA's abort flag and everybody leaves.
__device__ __forceinline__ void mbar_init(uint32_t a, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t a, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(a), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t a) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t a, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok)
                 : "r"(a), "r"(parity)
                 : "memory");
    return ok != 0;
}
constexpr uint32_t RING_WAIT_TRIES = 1u << 22;
__device__ __forceinline__ bool mbar_wait(uint32_t a, uint32_t parity, const volatile uint32_t* abort_flag) {
    for (uint32_t i = 0; i < RING_WAIT_TRIES; ++i) {
        if (mbar_try_wait(a, parity)) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t mbar, ull policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(mbar), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ uint4 lds_record(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
    return v;
}

template <uint32_t LP, bool HOT, bool DEDUPE>
__device__ __forceinline__ void ring_body(const IngestParams& p, Ctx& c, ull* full_bar, ull* empty_bar, volatile uint32_t* abort_flag) {
    constexpr uint32_t S = SCATTER_RING_STAGES > 0 ? SCATTER_RING_STAGES : 1;
    constexpr uint32_t TILE_RECS = SCATTER_CONSUMER_WARPS * 32;
    const unsigned char* recs = reinterpret_cast<const unsigned char*>(p.recs);
    // tile T covers records [T * 992, (T + 1) * 992); CTA b takes tiles b, b + G, b + 2 G, ...
    const ull n_tiles = (p.n_recs + TILE_RECS - 1) / TILE_RECS;
    const uint32_t mine = blockIdx.x < n_tiles ? (uint32_t)((n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0u;
    const uint32_t fb = smem_addr(full_bar), eb = smem_addr(empty_bar);
    if (threadIdx.x >= TILE_RECS) {
        // producer warp
        if (threadIdx.x == TILE_RECS) {
            ull policy;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
            uint32_t issued = 0;
            for (uint32_t k = 0; k < mine; ++k, ++issued) {
                const uint32_t s = k % S;
                if (k >= S && !mbar_wait(eb + s * 8, ((k / S) - 1u) & 1u, abort_flag)) {
                    if (!*abort_flag) atomicOr(&p.t.ctl->status, ST_TIMEOUT);
                    *abort_flag = 1;
                    break;
                }
                const ull T = (ull)k * gridDim.x + blockIdx.x;
                const ull first = T * TILE_RECS;
                const uint32_t n_here = (uint32_t)(p.n_recs - first < TILE_RECS ? p.n_recs - first : TILE_RECS);
                mbar_expect_tx(fb + s * 8, n_here * 16u);
                bulk_load(c.sb + Smem<LP>::RING + s * SCATTER_RING_TILE, recs + first * 16, n_here * 16u, fb + s * 8, policy);
            }
            if (*abort_flag) {
                // leaving early: give the copies still in flight a (bounded) chance to land first
                for (uint32_t k = issued > S ? issued - S : 0; k < issued; ++k) {
                    bool done = false;
                    for (uint32_t i = 0; i < 4096 && !done; ++i) done = mbar_try_wait(fb + (k % S) * 8, (k / S) & 1u);
                }
            }
        }
        return;
    }
    // consumers: two tiles (two records per thread) at a time
    const uint32_t lane_off = threadIdx.x * 16u;
    for (uint32_t k = 0; k < mine; k += 2) {
        const uint32_t s0 = k % S, s1 = (k + 1) % S;
        const bool second = k + 1 < mine;
        bool ok = mbar_wait(fb + s0 * 8, (k / S) & 1u, abort_flag);
        if (ok && second) ok = mbar_wait(fb + s1 * 8, ((k + 1) / S) & 1u, abort_flag);
        if (!ok) {
            if (!*abort_flag) atomicOr(&p.t.ctl->status, ST_TIMEOUT);
            *abort_flag = 1;
            return;
        }
        const ull first0 = ((ull)k * gridDim.x + blockIdx.x) * TILE_RECS, first1 = first0 + (ull)gridDim.x * TILE_RECS;
        const bool p0 = first0 + threadIdx.x < p.n_recs, p1 = second && first1 + threadIdx.x < p.n_recs;
        uint4 r0 = make_uint4(0, 0, 0, 0), r1 = make_uint4(0, 0, 0, 0);
        if (p0) r0 = lds_record(c.sb + Smem<LP>::RING + s0 * SCATTER_RING_TILE + lane_off);
        if (p1) r1 = lds_record(c.sb + Smem<LP>::RING + s1 * SCATTER_RING_TILE + lane_off);
        __syncwarp();
        if ((threadIdx.x & 31u) == 0) {   // the warp has its records in registers: hand the stages back
            mbar_arrive(eb + s0 * 8);
            if (second) mbar_arrive(eb + s1 * 8);
        }
        const uint32_t w[2][4] = {{r0.x, r0.y, r0.z, r0.w}, {r1.x, r1.y, r1.z, r1.w}};
        const bool full = second && first1 + TILE_RECS <= p.n_recs;     // both tiles complete (uniform)
        if (full) {
            process<LP, HOT, DEDUPE, true, 2>(p, c, w, true);
        } else {
            // ragged end: one record at a time, each with its own mask
            const uint32_t wa[1][4] = {{r0.x, r0.y, r0.z, r0.w}}, wb[1][4] = {{r1.x, r1.y, r1.z, r1.w}};
            process<LP, HOT, DEDUPE, false, 1>(p, c, wa, p0);
            process<LP, HOT, DEDUPE, false, 1>(p, c, wb, p1);
        }
    }
}

template <uint32_t LP, bool HOT>
__global__ void __launch_bounds__(SCATTER_THREADS, 1) scatter_kernel(IngestParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using L = Smem<LP>;
    uint32_t* g_cursor = reinterpret_cast<uint32_t*>(smem_raw + L::CUR);
    uint32_t* g_appw = reinterpret_cast<uint32_t*>(smem_raw + L::APPW);
    uint32_t* g_tag = reinterpret_cast<uint32_t*>(smem_raw + L::TAG);
    ull* g_keys = reinterpret_cast<ull*>(smem_raw + L::KEYS);
    uint32_t* g_acc = reinterpret_cast<uint32_t*>(smem_raw + L::ACC);

    __shared__ __align__(8) ull s_full[SCATTER_RING_STAGES ? SCATTER_RING_STAGES : 1], s_empty[SCATTER_RING_STAGES ? SCATTER_RING_STAGES : 1];
    __shared__ uint32_t s_abort;
    if (SCATTER_RING_STAGES > 0 && threadIdx.x == 0) {
        for (uint32_t i = 0; i < SCATTER_RING_STAGES; ++i) {
            mbar_init(smem_addr(&s_full[i]), 1);                          // the producer's arrive + the copy's bytes
            mbar_init(smem_addr(&s_empty[i]), SCATTER_CONSUMER_WARPS);    // one arrive per consumer warp
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }

    Ctx c;
    c.sb = smem_addr(smem_raw);
    c.mult = HOT ? (uint32_t)p.t.ctl->dir_mult : 1u;
    c.my_spill = p.spill + ((size_t)blockIdx.x << LP) * p.cap * SPILL_ENTRY_BYTES;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(c.keep));

    // The buffers persist across launches until the partition pass drains them: resume the cursors.
    for (uint32_t i = threadIdx.x; i < L::P; i += blockDim.x) g_cursor[i] = p.spill_cnt[((size_t)blockIdx.x << LP) + i];
    if (p.appw_in_smem != 0)
        for (uint32_t i = threadIdx.x; i < p.n_apps; i += blockDim.x) g_appw[i] = p.app_w[i];
    if (HOT) {
        for (uint32_t i = threadIdx.x; i < L::SLOTS + DIR_WAYS; i += blockDim.x) {
            const ull image = i < L::SLOTS ? p.hot_keys[i] : 0ull;   // ~key, 0 = empty
            g_keys[i] = ~image;
            reinterpret_cast<unsigned char*>(g_tag)[i] =
                image ? (unsigned char)(dir_mix(hash32(~image), (uint32_t)(~image >> 48) & 0xFFu, c.mult) & 0xFFu) : 0;
            g_acc[3 * i] = 0;
            g_acc[3 * i + 1] = 0;
            g_acc[3 * i + 2] = 0;
        }
    }
    __syncthreads();

    if (SCATTER_RING_STAGES > 0) {
        if (HOT && p.t.ctl->hot_skew != 0)
            ring_body<LP, HOT, true>(p, c, s_full, s_empty, &s_abort);
        else
            ring_body<LP, HOT, false>(p, c, s_full, s_empty, &s_abort);
    } else {
        if (HOT && p.t.ctl->hot_skew != 0)
            scatter_body<LP, HOT, true>(p, c);
        else
            scatter_body<LP, HOT, false>(p, c);
    }

    __syncthreads();
    uint32_t spilled = 0, fullest = 0;
    bool crowded = false;
    for (uint32_t i = threadIdx.x; i < L::P; i += blockDim.x) {
        const size_t at = ((size_t)blockIdx.x << LP) + i;
        const uint32_t before = p.spill_cnt[at], n = min(g_cursor[i], p.cap);
        p.spill_cnt[at] = n;
        spilled += n - before;
        crowded |= n > p.drain_above;
        fullest = max(fullest, n);
    }
    fullest = __reduce_max_sync(0xFFFFFFFFu, fullest);
    spilled = __reduce_add_sync(0xFFFFFFFFu, spilled);
    crowded = __any_sync(0xFFFFFFFFu, crowded);
    if ((threadIdx.x & 31u) == 0) {
        if (spilled) atomicAdd(&p.t.ctl->n_spilled, (ull)spilled);
        // a buffer is filling up: have the partition pass that follows this launch drain them
        if (crowded) atomicMax(&p.t.ctl->drain_seq, p.seq);
        atomicMax(&p.t.ctl->max_fill, (ull)fullest);
    }
    if (HOT) {
        // This launch's directory sums go to the CTA's own row of the directory image: plain coalesced
        // read-modify-writes, no atomics (148 CTAs adding the same few thousand keys into the table at
        // the end of every launch cost 59 us per launch).  hot_fold_kernel adds the rows into the table
        // before results are read.
        ulonglong2* img = p.hot_img + (size_t)blockIdx.x * L::SLOTS;
        for (uint32_t i0 = threadIdx.x; i0 < L::SLOTS; i0 += 4 * blockDim.x) {  // four slots per thread in flight
            uint32_t cn[4], lo[4], hi[4];
            ulonglong2 o[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t i = i0 + u * blockDim.x;
                const bool in = i < L::SLOTS;
                lo[u] = in ? g_acc[3 * i] : 0u;
                hi[u] = in ? g_acc[3 * i + 1] : 0u;
                cn[u] = in ? g_acc[3 * i + 2] : 0u;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) o[u] = (cn[u] | lo[u] | hi[u]) ? img[i0 + u * blockDim.x] : make_ulonglong2(0, 0);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if ((cn[u] | lo[u] | hi[u]) == 0) continue;
                const ull nlo = o[u].x + ((ull)lo[u] | ((ull)hi[u] << 32));
                img[i0 + u * blockDim.x] = make_ulonglong2(nlo, o[u].y + (ull)cn[u] + ((nlo < o[u].x ? 1ull : 0ull) << HI_SHIFT));
            }
        }
    }
}

template <uint32_t LP>
cudaError_t prepare_lp() {
    cudaError_t e = cudaFuncSetAttribute(scatter_kernel<LP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)SCATTER_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(scatter_kernel<LP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)SCATTER_SMEM_BYTES);
}

template <uint32_t LP>
void launch_lp(const IngestParams& p, bool hot, int grid, cudaStream_t stream) {
    if (hot)
        scatter_kernel<LP, true><<<grid, SCATTER_THREADS, Smem<LP>::TOTAL, stream>>>(p);
    else
        scatter_kernel<LP, false><<<grid, SCATTER_THREADS, Smem<LP>::TOTAL, stream>>>(p);
}

}  // namespace

cudaError_t scatter_prepare() {
    cudaError_t e = prepare_lp<8>();
    if (e == cudaSuccess) e = prepare_lp<9>();
    if (e == cudaSuccess) e = prepare_lp<10>();
    if (e == cudaSuccess) e = prepare_lp<11>();
    if (e == cudaSuccess) e = prepare_lp<12>();
    return e;
}

cudaError_t launch_scatter(const IngestParams& p, bool hot, int grid, cudaStream_t stream) {
    if (hot && p.hot_slots != scatter_hot_slots(p.t.lp)) return cudaErrorInvalidValue;
    switch (p.t.lp) {
        case 8: launch_lp<8>(p, hot, grid, stream); break;
        case 9: launch_lp<9>(p, hot, grid, stream); break;
        case 10: launch_lp<10>(p, hot, grid, stream); break;
        case 11: launch_lp<11>(p, hot, grid, stream); break;
        case 12: launch_lp<12>(p, hot, grid, stream); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace atrex
