// Device-side data layout and helpers shared by the library's kernels.
//
// HBM layout
//   key table   : P partitions (power of two) of C slots each, structure of arrays:
//                   keys[P*C]  ~key, so that 0 means EMPTY and reset is a memset
//                   vals[P*C]  {lo, cnthi}: lo = low 64 bits of the weighted time (wraps; wraps
//                              are counted), cnthi = count in bits 0..39, number of wraps of
//                              `lo` plus merged high words in bits 40..63
//                              (count < 2^40, weighted time < 2^88)
//                 A key lives in the partition given by the top log2 P bits of its 32-bit hash, at
//                 a slot found by double hashing over slot pairs inside that partition only (see
//                 find_or_claim below).  C is chosen so that one partition's
//                 keys and per-launch accumulators fit in one SM's shared memory: the
//                 aggregation pass owns a partition per CTA and needs no global atomics.
//   spill bufs  : [G][P][cap] 12-byte entries -- an 8-byte word {weighted duration, operator}
//                 and a 4-byte word {phase, low hash bits} -- and [G][P] counts,
//                 written by CTA g of the scatter pass (its buffers are contiguous, which keeps
//                 the scattered appends within a few pages), read by CTA p of the partition pass
//   work table  : the same P partitions (by the same hash of op_id and shape_id) of Cw 32-byte
//                 slots {~(op_id << 32 | shape_id), flops, bytes, dtype}, probed inside the partition
//   control     : counters, per-phase totals, top-k histogram
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/atrex_agg.h"

namespace atrex {

typedef unsigned long long ull;

struct WorkSlot {
    ull skey;      // ~(op_id << 32 | shape_id), 0 = EMPTY
    ull flops;
    ull bytes;
    ull dtype;
};
static_assert(sizeof(WorkSlot) == 32, "one slot per 32-byte sector");

constexpr ull COUNT_MASK = (1ull << 40) - 1;
constexpr int HI_SHIFT = 40;

// device status bits
constexpr ull ST_TABLE_FULL = 1;
constexpr ull ST_WORK_DUP = 2;
constexpr ull ST_WORK_FULL = 4;
constexpr ull ST_WORK_DTYPE = 8;
constexpr ull ST_TIMEOUT = 16;
constexpr ull ST_BOUNDS = 32;   // debug build: an index was outside its array

constexpr int TOPK_BINS = 4096;       // 12-bit digits
constexpr int TOPK_DIGITS = 12;       // 144-bit composite = 88-bit weighted time, 56-bit ~key
constexpr uint32_t TOPK_CAND_CAP = 65536;

struct Control {
    ull status;
    ull n_rejected;
    ull n_dropped;
    ull n_out;                 // entries emitted by the last finalize
    ull sel_count;             // top-k: selected candidates
    ull hot_n;                 // keys in the hot directory
    ull work_status;           // ST_WORK_* bits of the last work-table load
    ull hot_skew;              // 1 if one key dominates the sample: combine equal lanes per warp
    ull n_spilled;             // records routed through the spill buffers
    ull n_overflow;            // records that found their spill buffer full (slow exact path)
    ull drain_seq;             // sequence number of the last scatter launch that asked for a drain
    ull max_fill;              // fullest spill buffer seen since reset (entries)
    ull n_drains;              // partition passes that actually ran
    ull dir_mult;              // multiplier of the hot directory's bucket hash chosen at build time
    ull part_cursor;           // partition pass: next partition to hand out (zeroed before each launch)
    ull pad1[1];
    ull total_lo[ATREX_MAX_PHASES];
    ull total_hi[ATREX_MAX_PHASES];
    ull keys_per_phase[ATREX_MAX_PHASES];
    ull count_per_phase[ATREX_MAX_PHASES];
    ull sel_count_all[ATREX_MAX_PHASES];  // top-k: candidates collected per phase
    uint32_t hist[TOPK_BINS];
};

// 32-bit mixer of (op_id, shape_id) for the key table, the spill partitions, the hot directory
// and the work table: two multiplicative hashes of the two words, folded and multiplied once
// more.  The top bits pick the partition, the bits below them the start slot inside it.  The
// phase is deliberately left out: a key's partition is then also the partition of its
// (operator, shape) row in the work table, which keeps the roofline pass's look-ups local.
constexpr uint32_t HASH_A = 0x9E3779B1u, HASH_B = 0x85EBCA77u, HASH_C = 0x2C1B3C6Du;
__device__ __forceinline__ uint32_t hash32(uint32_t op, uint32_t shape) {
    uint32_t h = (shape * HASH_A) ^ (op * HASH_B);
    h ^= h >> 15;
    h *= HASH_C;
    h ^= h >> 13;
    return h;
}
// For a given operator the hash is a bijection of the shape (odd multipliers, xor-shifts), so inside a
// partition the triple (phase, operator, hash) identifies a key as well as (phase, operator, shape) does.
// The inverse: undo the xor-shifts, multiply by the multipliers' inverses modulo 2^32.
constexpr uint32_t mod_inverse_u32(uint32_t a) {   // a odd; Newton's iteration doubles the correct bits
    uint32_t x = a;
    for (int i = 0; i < 5; ++i) x *= 2u - a * x;
    return x;
}
constexpr uint32_t HASH_A_INV = mod_inverse_u32(HASH_A), HASH_C_INV = mod_inverse_u32(HASH_C);
static_assert(HASH_A * HASH_A_INV == 1u && HASH_C * HASH_C_INV == 1u, "modular inverses");
__host__ __device__ __forceinline__ uint32_t shape_of_hash(uint32_t h, uint32_t op) {
    uint32_t x = h ^ (h >> 13) ^ (h >> 26);
    x *= HASH_C_INV;
    x = x ^ (x >> 15) ^ (x >> 30);
    return (x ^ (op * HASH_B)) * HASH_A_INV;
}
__device__ __forceinline__ uint32_t hash32(ull key) { return hash32((uint32_t)(key >> 32) & 0xFFFFu, (uint32_t)key); }

// Placement of a key in the scatter pass's hot directory: the high bits of the mixed hash choose the
// bucket, its low byte is the slot's tag.  The odd multiplier is picked per directory build so that
// as little sampled weight as possible is lost to crowded buckets.  The table hash `h` leaves the
// phase out, the directory must not: the phases of a hot (operator, shape) are usually all hot and
// would otherwise fight over one bucket.
__device__ __forceinline__ uint32_t dir_mix(uint32_t h, uint32_t phase, uint32_t mult) {
    return (h + phase * 0x9E3779B9u) * mult;
}
__device__ __forceinline__ uint32_t dir_bucket(uint32_t h, uint32_t phase, uint32_t mult, uint32_t n_buckets) {
    return __umulhi(dir_mix(h, phase, mult), n_buckets);
}

// The partition pass's own form of a key, unique inside a partition: bit 63 set (so that 0 can mean
// an empty slot), phase << 16 | operator in bits 32..55, the 32-bit hash below.
constexpr ull CKEY_MARK = 1ull << 63;
__device__ __forceinline__ ull ckey_of(uint32_t khi24, uint32_t h) { return CKEY_MARK | ((ull)khi24 << 32) | h; }
__device__ __forceinline__ ull ckey_of_key(ull key) { return ckey_of((uint32_t)(key >> 32) & 0x00FFFFFFu, hash32((uint32_t)(key >> 32) & 0xFFFFu, (uint32_t)key)); }
__device__ __forceinline__ uint32_t ckey_phase(ull ckey) { return (uint32_t)(ckey >> 48) & 0xFFu; }
__device__ __forceinline__ ull key_of_ckey(ull ckey) {
    const uint32_t khi24 = (uint32_t)(ckey >> 32) & 0x00FFFFFFu;
    return ((ull)khi24 << 32) | shape_of_hash((uint32_t)ckey, khi24 & 0xFFFFu);
}
// The two words of a spill entry (12 bytes): a = product (48 bits) | operator << 48,
// b = phase << 24 | the hash bits below the partition's log2 P (at most 24: there are at least 2^8 partitions).
constexpr uint32_t SPILL_ENTRY_BYTES = 12;
__device__ __forceinline__ ull ckey_of_spill(ull a, uint32_t b, uint32_t part, uint32_t lp) {
    return ckey_of(((b >> 24) << 16) | (uint32_t)(a >> 48), (part << (32 - lp)) | (b & (0xFFFFFFFFu >> lp)));
}

__device__ __forceinline__ ull pack_key(uint32_t phase, uint32_t op, uint32_t shape) {
    return ((ull)phase << 48) | ((ull)op << 32) | (ull)shape;
}

// Debug build (-DATREX_DEBUG_BOUNDS): every index into the key table, the work table, the spill buffers
// and the kernels' shared-memory arrays goes through ATREX_INDEX, which latches ST_BOUNDS in the control
// block and substitutes index 0 when the index is outside [0, limit) -- the access then touches valid
// memory and the violation is reported as ATREX_ERR_BOUNDS by the next finalize / stats (nothing traps).
// In the regular build the macro is the index itself.
#ifdef ATREX_DEBUG_BOUNDS
template <typename I, typename L>
__device__ __forceinline__ I checked_index(I i, L limit, ull* status) {
    if ((ull)i < (ull)limit) return i;
    atomicOr(status, ST_BOUNDS);
    return (I)0;
}
#define ATREX_INDEX(i, limit, ctl) atrex::checked_index((i), (limit), &(ctl)->status)
#else
#define ATREX_INDEX(i, limit, ctl) (i)
#endif

__device__ __forceinline__ ull ld_relaxed(const ull* p) {
    ull v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p));
    return v;
}

struct TableRef {
    ull* keys;            // [P * C]
    ulonglong2* vals;     // [P * C] {lo, cnthi}
    uint32_t lp;          // log2(P)
    uint32_t C;           // slots per partition (even)
    Control* ctl;
    ull strides;          // eight probe strides in slot pairs, one byte each: odd primes that do not divide C / 2
};

constexpr ull NO_INDEX = ~0ull;

__device__ __forceinline__ uint32_t part_of(uint32_t h, uint32_t lp) { return h >> (32 - lp); }  // lp >= 1

// Probe sequence of a key inside its partition (double hashing over slot pairs): it starts at the
// pair holding local_of() and moves on by one of eight strides chosen by other hash bits; inside a
// pair the even slot comes first.  The strides are coprime to the number of pairs, so the sequence
// visits every pair once.  Every prober -- this file's global-memory path and the partition pass's
// shared-memory path -- follows the same order, and a key sits at the first slot of its sequence
// that was free when it arrived.  Clusters of linear probing, which at the load factors reached
// here (up to 0.7) made the slowest of a warp's probes several times the average, do not form.
// The phase, which the partition choice ignores, is mixed into the start so that the phases of one
// (operator, shape) do not pile up on the same pair.
__device__ __forceinline__ uint32_t local_of(uint32_t h, uint32_t phase, uint32_t C) {
    return __umulhi((h ^ (phase * 0x9E3779B9u)) * 0x85EBCA6Bu, C);
}
__device__ __forceinline__ uint32_t stride_index(uint32_t h) { return (h >> 3) & 7u; }
__device__ __forceinline__ uint32_t stride_of(const TableRef& t, uint32_t index) {
    return (uint32_t)(t.strides >> (8 * index)) & 0xFFu;
}

// Find (or claim) the slot of `key` directly in HBM.  Returns NO_INDEX when the key's
// partition has no free slot.  Used off the hot path: directory flush, buffer overflow,
// merge.
__device__ __forceinline__ ull find_or_claim(const TableRef& t, ull key, uint32_t h) {
    const ull skey = ~key;
    const ull base = (ull)part_of(h, t.lp) * t.C;
    uint32_t s = local_of(h, (uint32_t)(key >> 48), t.C) & ~1u;
    const uint32_t advance = 2u * stride_of(t, stride_index(h));
    for (uint32_t probe = 0; probe < t.C; ++probe) {
        ull* kp = t.keys + ATREX_INDEX(base + s, (ull)t.C << t.lp, t.ctl);
        ull k = ld_relaxed(kp);
        if (k == skey) return base + s;
        if (k == 0) {
            ull old = atomicCAS(kp, 0ull, skey);
            if (old == 0 || old == skey) return base + s;
        }
        if (s & 1u) {  // second slot of the pair done: on to the next pair
            s = (s & ~1u) + advance;
            if (s >= t.C) s -= t.C;
        } else {
            s |= 1u;
        }
    }
    return NO_INDEX;
}

// Exact, order-independent accumulation of (count, v_hi * 2^64 + v_lo) into a slot: the
// thread whose add wraps `lo` is unique, and it alone adds the carry.
__device__ __forceinline__ void slot_add(const TableRef& t, ull idx, ull v_lo, ull v_hi, ull count) {
    ull* v = reinterpret_cast<ull*>(t.vals + ATREX_INDEX(idx, (ull)t.C << t.lp, t.ctl));
    ull carry = 0;
    if (v_lo != 0) {
        ull old = atomicAdd(v, v_lo);
        carry = (old + v_lo < old) ? 1ull : 0ull;
    }
    ull inc = count + ((v_hi + carry) << HI_SHIFT);
    if (inc != 0) atomicAdd(v + 1, inc);
}

__device__ __forceinline__ void table_accumulate(const TableRef& t, ull key, uint32_t h, ull v_lo, ull v_hi, ull count) {
    ull idx = find_or_claim(t, key, h);
    if (idx == NO_INDEX) {
        atomicOr(&t.ctl->status, ST_TABLE_FULL);
        atomicAdd(&t.ctl->n_dropped, count);
        return;
    }
    slot_add(t, idx, v_lo, v_hi, count);
}

// One round-to-nearest-even conversion of hi * 2^64 + lo to binary64.  The top 64
// significant bits are kept with a sticky bit folded into bit 0 (far below the 53-bit cut),
// converted with a single rounding, then scaled by an exact power of two.
__device__ __forceinline__ double u128_to_f64_rn(ull hi, ull lo) {
    if (hi == 0) return __ull2double_rn(lo);
    int s = __clzll((long long)hi);
    ull m, rest;
    if (s == 0) {
        m = hi;
        rest = lo;
    } else {
        m = (hi << s) | (lo >> (64 - s));
        rest = lo << s;
    }
    if (rest != 0) m |= 1ull;
    double scale = __longlong_as_double((long long)(1023 + 64 - s) << 52);
    return __dmul_rn(__ull2double_rn(m), scale);
}

}  // namespace atrex
