// Kernel parameter blocks and host-side launchers (internal to the library).
#pragma once
#include "atrex_dev.cuh"

namespace atrex {

// Build-time variant of the scatter pass (the default is the fastest measured; the other is kept so
// that the comparison can be repeated):
//   ATREX_SCATTER_RING   stages of a shared-memory ring that a producer warp fills with bulk
//                        asynchronous copies of record tiles (0: records are loaded straight into
//                        registers, two 32-byte loads alternating per thread)
#ifndef ATREX_SCATTER_RING
#define ATREX_SCATTER_RING 0
#endif

// Shared memory of the scatter pass (dynamic, one CTA per SM) and what fits in it.  Per partition a
// cursor word, 16 KB of card-hour weights, the record ring if there
// is one, then the hot directory: a tag byte, an 8-byte key and 12 bytes of accumulators per slot, in
// whole 4-way buckets.
constexpr uint32_t APPW_SMEM_MAX = 4096;
constexpr uint32_t SCATTER_SMEM_BYTES = 232448 - 1024;
constexpr uint32_t SCATTER_RING_STAGES = ATREX_SCATTER_RING;
constexpr uint32_t SCATTER_CONSUMER_WARPS = SCATTER_RING_STAGES ? 31 : 32;
constexpr uint32_t SCATTER_RING_TILE = SCATTER_CONSUMER_WARPS * 32 * 16;   // one record per consumer thread
constexpr uint32_t scatter_fixed_bytes(uint32_t lp) {
    return (4u << lp) + 4u * APPW_SMEM_MAX + SCATTER_RING_STAGES * SCATTER_RING_TILE + 128u;
}
constexpr uint32_t scatter_hot_slots(uint32_t lp) { return ((SCATTER_SMEM_BYTES - scatter_fixed_bytes(lp)) / 21u) & ~31u; }

struct IngestParams {
    const void* recs;          // all records of this launch (16-byte aligned) ...
    ull n_recs;
    const void* body;          // ... and the same split up: first record of the 32-byte aligned run of record pairs
    ull n_pairs;               // pairs in the body
    const void* single[2];     // records outside the body (unaligned head, odd tail)
    uint32_t n_single;
    uint32_t n_apps, n_phases;
    uint32_t phase_lim;        // n_phases << 16: bound of (phase << 16 | op_id)
    uint32_t appw_in_smem;
    const uint32_t* app_w;     // device copy of the card-hour weights
    const ull* hot_keys;       // directory image, hot_slots entries of ~key (0 = empty)
    uint32_t hot_slots;        // multiple of 4
    uint32_t hot_buckets;      // hot_slots / 4
    ulonglong2* hot_img;       // [n_groups][hot_slots] each CTA's directory sums since the last fold, {lo, count | hi << 40}
    TableRef t;
    // spill buffers: entry i of scatter CTA g for partition p at spill + ((g * P + p) * cap + i) * 12 bytes: an 8-byte
    // word {product, operator} and a 4-byte word {phase, low hash bits}, the 8-byte word at the 8-byte aligned end
    unsigned char* spill;
    uint32_t* spill_cnt;       // [n_groups][P]
    uint32_t n_groups;         // G, row pitch of the buffers (= CTAs of the widest scatter launch)
    uint32_t cap;              // entries per (partition, CTA) buffer, a multiple of 32 (whole 128-byte lines)
    uint32_t drain_above;      // ask for a drain when a buffer holds more entries than this
    ull seq;                   // sequence number of this launch
};

struct PartitionParams {
    TableRef t;
    const unsigned char* spill;
    uint32_t* spill_cnt;
    uint32_t n_groups;         // row pitch G
    uint32_t n_used;           // scatter CTAs whose buffers are read (<= G)
    uint32_t cap;
    uint32_t force;            // 1: drain unconditionally; 0: only if the scatter launch `seq` asked for it
    ull seq;
    ulonglong2* queue;         // [gridDim][queue_cap] entries whose first look failed, settled after the partition's stream
    uint32_t queue_cap;
};

struct HotBuildParams {
    const uint4* recs;
    ull stride;
    uint32_t n_sample;
    uint32_t n_apps, n_phases;
    ull* hot_keys;
    uint32_t hot_slots;
    uint32_t* sketch;          // [2^20] sample counters by hash
    ull* cand_keys;            // [1 << cand_bits] candidate table: ~key, 0 = empty
    uint32_t* cand_cnt;        // [1 << cand_bits] exact sample counts of the candidates
    uint32_t cand_bits;
    Control* ctl;
};

struct WorkRef {
    WorkSlot* table;     // [P * Cw], nullptr when no work table was provisioned
    uint32_t lp;         // log2(P), same partitioning as the key table
    uint32_t Cw;         // slots per partition
    ull strides;         // eight probe strides, one byte each: odd primes that do not divide Cw (double hashing)
};

struct FinalizeParams {
    TableRef t;
    ull n_slots;
    Control* ctl;
    WorkRef work;
    atrex_hw_peaks_t peaks;
    atrex_entry_t* out;
    ull out_cap;
};

struct TopkParams {
    TableRef t;
    ull n_slots;
    Control* ctl;
    uint32_t phase;
    uint32_t n_prefix_digits;   // leading 12-bit digits of the ranking composite already fixed
    uint16_t prefix_digit[12];  // their values, most significant first
    uint32_t shift;             // leading zero bits of the composite dropped before digit extraction
    int collect_all;
    ull* sel;                   // [sel_cap][4]: composite words 2,1,0 and the slot index
    uint32_t sel_cap;
};

// Top-k over several phases in one pass over the table: phase q of `active_mask` has its own digit
// alignment, fixed prefix, histogram row and selection region.
struct TopkAllParams {
    TableRef t;
    ull n_slots;
    uint32_t active_mask;                              // phases taking part in this pass
    uint32_t collect_all_mask;                         // phases whose every entry is collected
    uint32_t shift[ATREX_MAX_PHASES];
    uint32_t n_prefix_digits[ATREX_MAX_PHASES];
    uint16_t prefix_digit[ATREX_MAX_PHASES][12];
    uint32_t* hist;                                    // [ATREX_MAX_PHASES][TOPK_BINS] next-digit counts
    ull* sel;                                          // [ATREX_MAX_PHASES][sel_cap][4]
    ull* sel_count;                                    // [ATREX_MAX_PHASES]
    uint32_t sel_cap;
};

cudaError_t ingest_prepare();
cudaError_t scatter_prepare();
cudaError_t launch_scatter(const IngestParams& p, bool hot, int grid, cudaStream_t stream);
cudaError_t launch_partition(const PartitionParams& p, int n_sms, cudaStream_t stream);
cudaError_t launch_hot_build(const HotBuildParams& p, int n_sms, cudaStream_t stream);
cudaError_t launch_hot_fold(const ull* hot_keys, ulonglong2* hot_img, uint32_t n_groups, uint32_t hot_slots,
                            const TableRef& t, cudaStream_t stream);
cudaError_t launch_merge(const atrex_entry_t* in, ull n, const TableRef& t, int grid, cudaStream_t stream);

cudaError_t finalize_prepare();
cudaError_t launch_totals(const TableRef& t, ull n_slots, int grid, cudaStream_t stream);
cudaError_t launch_emit(const FinalizeParams& p, int grid, cudaStream_t stream);
cudaError_t launch_work_insert(const atrex_work_t* rows, ull n, const WorkRef& w, Control* ctl, int grid,
                               cudaStream_t stream);
cudaError_t launch_topk_hist_all(const TopkAllParams& p, int n_sms, cudaStream_t stream);
cudaError_t launch_topk_collect_all(const TopkAllParams& p, int grid, cudaStream_t stream);
cudaError_t launch_topk_hist(const TopkParams& p, int grid, cudaStream_t stream);
cudaError_t launch_topk_sort(ull* sel, uint32_t n_pow2, cudaStream_t stream);
cudaError_t launch_topk_emit(const FinalizeParams& p, const ull* sel, uint32_t n, cudaStream_t stream);

}  // namespace atrex
