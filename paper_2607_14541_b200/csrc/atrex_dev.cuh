// Device-side data layout and helpers shared by the library's kernels.
//
// HBM layout
//   key table   : open addressing, power-of-two capacity >= 2 * max_keys, one 32-byte slot
//                 (= one L2 sector) per key:
//                   skey  = ~key, so that 0 means EMPTY and reset is a memset
//                   lo    = low 64 bits of the weighted time (wraps; wraps are counted)
//                   cnthi = count in bits 0..39, number of wraps of `lo` plus merged high
//                           words in bits 40..63  (count < 2^40, weighted time < 2^88)
//                   spare
//   work table  : same scheme keyed by op_id << 32 | shape_id, holding flops, bytes, dtype
//   control     : counters, per-phase totals, top-k histogram
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/atrex_agg.h"

namespace atrex {

typedef unsigned long long ull;

struct Slot {
    ull skey;
    ull lo;
    ull cnthi;
    ull spare;
};
static_assert(sizeof(Slot) == 32, "one slot per 32-byte sector");

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
    ull pad0;
    ull total_lo[ATREX_MAX_PHASES];
    ull total_hi[ATREX_MAX_PHASES];
    ull keys_per_phase[ATREX_MAX_PHASES];
    ull count_per_phase[ATREX_MAX_PHASES];
    uint32_t hist[TOPK_BINS];
};

// 64-bit mixer for slot selection: multiply, fold, multiply; the top bits index the table.
__device__ __forceinline__ ull hash_key(ull key) {
    ull h = key * 0x9E3779B97F4A7C15ull;
    h ^= h >> 32;
    h *= 0xD6E8FEB86659FD93ull;
    return h;
}

__device__ __forceinline__ ull pack_key(uint32_t phase, uint32_t op, uint32_t shape) {
    return ((ull)phase << 48) | ((ull)op << 32) | (ull)shape;
}

__device__ __forceinline__ ull ld_relaxed(const ull* p) {
    ull v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p));
    return v;
}

// Find (or claim) the slot of `key`.  Returns nullptr after `max_probe` steps (table full).
__device__ __forceinline__ Slot* find_or_claim(Slot* table, ull mask, int shift, uint32_t max_probe,
                                               ull key, ull h) {
    const ull skey = ~key;
    ull s = h >> shift;
    for (uint32_t probe = 0; probe < max_probe; ++probe) {
        Slot* e = table + s;
        ull k = ld_relaxed(&e->skey);
        if (k == skey) return e;
        if (k == 0) {
            ull old = atomicCAS(&e->skey, 0ull, skey);
            if (old == 0 || old == skey) return e;
        }
        s = (s + 1) & mask;
    }
    return nullptr;
}

// Exact, order-independent accumulation of (count, v_hi * 2^64 + v_lo) into a slot: the
// thread whose add wraps `lo` is unique, and it alone adds the carry.
__device__ __forceinline__ void slot_add(Slot* e, ull v_lo, ull v_hi, ull count) {
    ull carry = 0;
    if (v_lo != 0) {
        ull old = atomicAdd(&e->lo, v_lo);
        carry = (old + v_lo < old) ? 1ull : 0ull;
    }
    ull inc = count + ((v_hi + carry) << HI_SHIFT);
    if (inc != 0) atomicAdd(&e->cnthi, inc);
}

struct TableRef {
    Slot* table;
    ull mask;
    int shift;            // 64 - log2(capacity)
    uint32_t max_probe;
    Control* ctl;
};

__device__ __forceinline__ void table_accumulate(const TableRef& t, ull key, ull h, ull v_lo, ull v_hi, ull count) {
    Slot* e = find_or_claim(t.table, t.mask, t.shift, t.max_probe, key, h);
    if (e == nullptr) {
        atomicOr(&t.ctl->status, ST_TABLE_FULL);
        atomicAdd(&t.ctl->n_dropped, count);
        return;
    }
    slot_add(e, v_lo, v_hi, count);
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
