/*
 * atrex_agg.h -- C ABI of the B200 trace-aggregation library.
 *
 * The library turns production inference-trace records into per-problem importance
 * weights and roofline ceilings, as defined by the paper's benchmark construction:
 *
 *   Eq. 2  cumulative observed device time per (operator, phase), summed over kernel
 *          invocations; here kept per (operator, shape, phase) key and scaled by the
 *          application's card-hour weight (Eq. 3's p_a) as an exact 128-bit integer;
 *   Eq. 3  normalisation so that weights sum to 1, taken separately for each serving
 *          phase (Sec. 3.1: each serving phase gets its own set of weights);
 *   Eq. 1  roofline time max(F / P_dtype, M / beta) per (operator, shape) unit;
 *   Table 2  ranking of units by weight (deterministic top-k).
 *
 * Conventions
 *   - Plain C, no exceptions, no global state: every call takes the handle.
 *   - "DEVICE" pointers are CUDA device memory on the handle's device; "HOST" pointers are
 *     ordinary host memory.  `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - All integers are little-endian; structs are packed as declared (no padding occurs).
 *   - Every function returns ATREX_OK (0) or a negative atrex_status_t; nothing aborts,
 *     traps or waits without a bound.
 *   - A handle must not be used from two host threads at once.
 *
 * Arithmetic contract (what makes results unique, so they can be compared bit for bit)
 *   key          = phase << 48 | op_id << 32 | shape_id
 *   count[key]   = number of valid records with that key                      (u64)
 *   wt[key]      = sum of app_weight[app_id] * duration_ns over those records  (u128, exact,
 *                  independent of ingestion order and chunking)
 *   T[phase]     = sum of wt over the phase's keys                             (u128)
 *   phase_weight = fl(fl(wt) / fl(T[phase])), or +0.0 when T[phase] == 0, where fl() of an
 *                  integer is ONE round-to-nearest-even conversion to binary64 and the
 *                  division is IEEE-754 binary64
 *   roofline_s   = fmax(fl(flops) / peak_flops[dtype], fl(bytes) / peak_bw); a key whose
 *                  (op_id, shape_id) has no work-table row gets the quiet NaN 0x7FF8000000000000
 *   A record is valid iff app_id < n_apps and phase < n_phases; invalid records are skipped
 *   and counted.  The `pad` byte is ignored.
 *   Limits: fewer than 2^40 records per handle between resets, and wt < 2^88 per key (always true
 *   when app_weight * duration_ns < 2^48, e.g. weights < 2^20 and durations < 2^28; larger
 *   products are accepted and summed exactly, through a slower path, as long as the key's sum
 *   stays below 2^88).
 */
#ifndef ATREX_AGG_H
#define ATREX_AGG_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ATREX_MAX_PHASES 8
#define ATREX_MAX_DTYPES 8
#define ATREX_MAX_TOPK 65536u
#define ATREX_MAX_WORLD 1024u     /* GPUs an entry array can be split over (atrex_entries_bucket_by_owner) */

typedef enum {
    ATREX_OK = 0,
    ATREX_ERR_INVALID = -1,        /* bad argument: null/misaligned pointer, range, duplicate work row */
    ATREX_ERR_CAPACITY = -2,       /* more distinct keys than provisioned; results are not valid        */
    ATREX_ERR_OUT_TOO_SMALL = -3,  /* output buffer too small; *n_out holds the needed count            */
    ATREX_ERR_CUDA = -4,           /* a CUDA runtime call failed (see atrex_agg_last_cuda_error)        */
    ATREX_ERR_TIMEOUT = -5,        /* a bounded device-side wait gave up                                */
    ATREX_ERR_STATE = -6,          /* call order: topk before finalize, or > 2^40 records               */
    ATREX_ERR_NOMEM = -7,          /* workspace too small / allocation failed                           */
    ATREX_ERR_TOO_LARGE = -8,      /* input larger than a fixed-size internal buffer can take           */
    ATREX_ERR_BOUNDS = -9          /* checked build only: a kernel computed an index outside its array  */
} atrex_status_t;

/* One observed device-kernel invocation (Sec. 3.1; the d_{a,phi,r,l} of Eq. 2). 16 bytes. */
typedef struct {
    uint32_t app_id;       /* application index a                      */
    uint16_t op_id;        /* operator family i                        */
    uint8_t  phase;        /* serving phase phi: 0 = prefill, 1 = decode, ... < n_phases */
    uint8_t  pad;          /* ignored                                  */
    uint32_t shape_id;     /* shape bucket s                           */
    uint32_t duration_ns;  /* observed device time of this invocation  */
} atrex_record_t;

/* Semantic work of one (operator, shape) unit (Sec. 3.3: F_j, M_j and the dtype tau_j). 24 bytes. */
typedef struct {
    uint32_t shape_id;
    uint16_t op_id;
    uint16_t dtype;        /* index into atrex_hw_peaks_t.peak_flops, < ATREX_MAX_DTYPES */
    uint64_t flops;
    uint64_t bytes;
} atrex_work_t;

/* Calibrated accelerator peaks (Sec. 3.3: P_tau and beta). All must be finite and > 0. */
typedef struct {
    double peak_bw;                        /* bytes / s  */
    double peak_flops[ATREX_MAX_DTYPES];   /* FLOP / s per dtype index */
} atrex_hw_peaks_t;

/* One aggregated unit. 48 bytes. */
typedef struct {
    uint64_t key;           /* phase << 48 | op_id << 32 | shape_id */
    uint64_t count;
    uint64_t wt_lo;         /* weighted time, low and high 64 bits  */
    uint64_t wt_hi;
    double   phase_weight;
    double   roofline_s;
} atrex_entry_t;

typedef struct {
    uint32_t n_apps;              /* >= 1 */
    uint32_t n_phases;            /* 1 .. ATREX_MAX_PHASES */
    uint64_t max_keys;            /* distinct (op, shape, phase) keys to provision for, >= 1 */
    uint64_t max_work_rows;       /* rows atrex_agg_set_work_table may receive (0 = none)    */
    const uint32_t* app_weights;  /* HOST, n_apps card-hour weights; copied by create        */
    void*    workspace;           /* DEVICE memory owned by the caller, 256-byte aligned, or */
    uint64_t workspace_bytes;     /*   NULL/0: the library allocates and frees its own       */
    int32_t  device;              /* CUDA device ordinal */
    uint32_t flags;               /* ATREX_FLAG_* */
} atrex_agg_config_t;

#define ATREX_FLAG_NO_HOT_DIRECTORY 1u  /* disable the shared-memory hot-key stage (debug / A-B) */

typedef struct {
    uint64_t n_valid;                     /* valid records ingested since create/reset */
    uint64_t n_rejected;                  /* records skipped as invalid                */
    uint64_t n_dropped;                   /* records lost to a full table (ATREX_ERR_CAPACITY) */
    uint64_t n_keys;                      /* distinct keys                             */
    uint64_t total_lo[ATREX_MAX_PHASES];  /* T[phase], low / high 64 bits              */
    uint64_t total_hi[ATREX_MAX_PHASES];
    uint64_t keys_per_phase[ATREX_MAX_PHASES];
    uint64_t table_slots;                 /* capacity of the key table                 */
    uint64_t hot_slots;                   /* keys currently in the shared-memory hot directory */
    uint64_t n_spilled;                   /* records that went through the partition spill buffers */
    uint64_t n_overflow;                  /* records that found their spill buffer full (slow exact path) */
    uint64_t max_spill_fill;              /* fullest spill buffer seen since reset, in entries */
    uint64_t spill_cap;                   /* capacity of one spill buffer, in entries */
    uint64_t n_drains;                    /* partition passes that ran since reset */
} atrex_stats_t;

typedef struct atrex_agg atrex_agg_t;

/* Bytes of DEVICE workspace a handle with this configuration needs (0 on invalid config). */
uint64_t atrex_agg_workspace_bytes(const atrex_agg_config_t* cfg);

/* Create a handle.  The workspace (caller's or library-allocated) is cleared on the device's
 * default stream and the call returns after that completes.  The caller keeps ownership of
 * cfg->workspace and must keep it alive until atrex_agg_destroy. */
int atrex_agg_create(const atrex_agg_config_t* cfg, atrex_agg_t** out);

/* Install the per-(operator, shape) work table used by Eq. 1.  `host_rows` is HOST memory, read
 * before the call returns.  n <= max_work_rows.  Duplicate (op, shape) pairs or dtype >=
 * ATREX_MAX_DTYPES give ATREX_ERR_INVALID (the table is then empty).  Synchronises `stream`. */
int atrex_agg_set_work_table(atrex_agg_t*, const atrex_work_t* host_rows, uint64_t n, void* stream);

/* Eq. 2: fold n records into the per-key sums.  `d_records` is DEVICE memory, 16-byte aligned,
 * and must stay valid until `stream` has passed this call.  Asynchronous: returns after
 * enqueueing; device-side conditions (table full) are latched and reported by the next
 * finalize / stats.  May be called any number of times; the result is independent of how the
 * records are split into calls and of their order. */
int atrex_agg_ingest(atrex_agg_t*, const atrex_record_t* d_records, uint64_t n, void* stream);

/* Same, for records in HOST memory (pinned memory gives asynchronous copies): the records are
 * copied through two device staging buffers inside the workspace, each copy overlapping the
 * previous piece's aggregation.  Returns after enqueueing the last piece; `h_records` must
 * stay valid until `stream` has passed this call. */
int atrex_agg_ingest_host(atrex_agg_t*, const atrex_record_t* h_records, uint64_t n, void* stream);

/* Fold already aggregated units (for instance another GPU's partial result: key, count, wt_lo,
 * wt_hi are read; the two doubles are ignored) into the table.  DEVICE pointer, asynchronous.
 * Exact: merging partial aggregates in any order equals aggregating all records at once. */
int atrex_agg_merge(atrex_agg_t*, const atrex_entry_t* d_entries, uint64_t n, void* stream);

/* Eq. 3 (per phase) and Eq. 1 for every key.  Writes one entry per distinct key to `d_out`
 * (DEVICE, capacity out_cap entries, order unspecified) and the number of entries to *n_out
 * (HOST).  d_out may be NULL with out_cap 0 to only obtain the count, refresh the totals and
 * set the peaks used by atrex_agg_topk.  Synchronises `stream`.  Non-destructive: ingest may
 * continue afterwards and finalize may be repeated, e.g. with other peaks. */
int atrex_agg_finalize(atrex_agg_t*, const atrex_hw_peaks_t* peaks, atrex_entry_t* d_out,
                       uint64_t out_cap, uint64_t* n_out, void* stream);

/* atrex_agg_finalize for one shard of a trace that was split over several handles (GPUs).
 * Eq. 3 normalises by the phase total over ALL records; when every handle holds only the keys it
 * owns (after the partial aggregates were exchanged and folded with atrex_agg_merge), the caller
 * adds the handles' per-phase totals (atrex_agg_totals, combined by atrex_totals_combine) and passes
 * the sums here: total_lo / total_hi are HOST arrays of ATREX_MAX_PHASES low / high 64-bit words.  The
 * entries written, and those atrex_agg_topk returns afterwards, then carry
 * phase_weight = fl(fl(wt) / fl(global total)), bit-identical to a single handle that saw every
 * record.  Everything else is as in atrex_agg_finalize. */
int atrex_agg_finalize_with_totals(atrex_agg_t*, const atrex_hw_peaks_t* peaks, const uint64_t* total_lo,
                                   const uint64_t* total_hi, atrex_entry_t* d_out, uint64_t out_cap,
                                   uint64_t* n_out, void* stream);

/* The per-phase totals T[phase] the last successful finalize of this handle normalised by (Eq. 3's
 * denominators; after atrex_agg_finalize the handle's own sums, after atrex_agg_finalize_with_totals
 * the totals that were passed in).  h_lo / h_hi: HOST arrays of ATREX_MAX_PHASES low / high words.
 * No device work.  ATREX_ERR_STATE without a finalize since the last ingest, merge or reset. */
int atrex_agg_totals(const atrex_agg_t*, uint64_t* h_lo, uint64_t* h_hi);

/* ---- exchange step of the multi-GPU path ------------------------------------------------------
 * Eq. 2 is a sum over independent invocations and all accumulators are exact integers, so the
 * trace shards by records: each GPU aggregates its slice with the calls above.  To make the
 * partial results global, every entry is sent to the GPU that owns its key and folded in there
 * with atrex_agg_merge; Eq. 3's denominators are then the sums of the shards' totals.  The three
 * calls below are the arithmetic of that step (the bytes are moved by the caller's collective).
 *
 * atrex_key_owner: the rank in [0, world) that owns `key`; a fixed scramble of the packed key. */
uint32_t atrex_key_owner(uint64_t key, uint32_t world);
/* The same for `n` keys at once: h_keys and h_out are HOST arrays. */
void atrex_keys_owner(const uint64_t* h_keys, uint64_t n, uint32_t world, uint32_t* h_out);

/* Groups the `n` entries at d_entries (DEVICE, 16-byte aligned) by owner rank: d_out (DEVICE, room
 * for n entries, must not overlap d_entries) receives rank 0's entries first, then rank 1's, ...;
 * h_counts (HOST, `world` values) the size of each group.  The order inside a group is unspecified.
 * d_scratch: DEVICE, 2 * world 64-bit words, contents irrelevant.  world <= ATREX_MAX_WORLD,
 * n <= 2^32 (ATREX_ERR_TOO_LARGE).  Synchronises `stream`. */
int atrex_entries_bucket_by_owner(const atrex_entry_t* d_entries, uint64_t n, uint32_t world, atrex_entry_t* d_out,
                                  uint64_t* d_scratch, uint64_t* h_counts, void* stream);

/* Exact sum of the shards' per-phase totals: h_lo / h_hi are HOST arrays [n_ranks][ATREX_MAX_PHASES]
 * of low / high 64-bit words (one row per shard, as atrex_agg_totals returns them), h_out_lo /
 * h_out_hi receive the ATREX_MAX_PHASES 128-bit sums.  Host arithmetic only (a reduction of the
 * halves by a collective would lose the carries). */
int atrex_totals_combine(const uint64_t* h_lo, const uint64_t* h_hi, uint32_t n_ranks, uint64_t* h_out_lo,
                         uint64_t* h_out_hi);

/* 1 if this library was built with -DATREX_DEBUG_BOUNDS, else 0.  In that build every index the
 * ingest kernels form into the key table, the spill buffers and their shared-memory arrays is range
 * checked; a violation substitutes a valid index, latches a status bit and makes the next finalize /
 * stats return ATREX_ERR_BOUNDS (nothing traps).  The regular build has no such checks. */
int atrex_build_has_bounds_checks(void);

/* Table 2: the min(k, keys of `phase`) entries with the largest weighted time, compared as
 * exact 128-bit integers, ties broken by ascending key; written in that order to `h_out`
 * (HOST, capacity k).  k <= ATREX_MAX_TOPK.  Uses the totals and peaks of the last finalize
 * (ATREX_ERR_STATE if there was none since the last ingest).  Synchronises `stream`.
 * Cost: the first call after a finalize selects the best k of EVERY phase in two passes over the
 * table and keeps the selections; further calls with the same k (any phase) only copy their
 * answer out, a call with another k repeats the second pass. */
int atrex_agg_topk(atrex_agg_t*, uint32_t phase, uint32_t k, atrex_entry_t* h_out, uint32_t* n_out,
                   void* stream);

/* Counters and per-phase totals (HOST output).  Synchronises `stream`. */
int atrex_agg_stats(atrex_agg_t*, atrex_stats_t* h_out, void* stream);

/* Diagnostic: copy the keys currently in the shared-memory hot directory (built from a sample of
 * the first large ingest after create/reset) to `h_keys` (HOST, capacity `cap` keys, any order).
 * *n_out = number of keys in the directory, which may exceed `cap`.  Synchronises `stream`. */
int atrex_agg_hot_directory(atrex_agg_t*, uint64_t* h_keys, uint32_t cap, uint32_t* n_out, void* stream);

/* Forget all records (the work table and weights are kept).  Asynchronous on `stream`. */
int atrex_agg_reset(atrex_agg_t*, void* stream);

void atrex_agg_destroy(atrex_agg_t*);

const char* atrex_strerror(int status);

/* cudaError_t value of the last failed CUDA call on this handle (0 if none). */
int atrex_agg_last_cuda_error(const atrex_agg_t*);

/* Number of kernels this handle has launched so far (for launch accounting in benchmarks). */
uint64_t atrex_agg_launch_count(const atrex_agg_t*);

/* Operator importance weights exactly as Eq. 2-3 state them (per-application denominators).
 *
 * The main path above weights each record by its application's card-hour weight and normalises per
 * phase.  Eq. 3 proper first turns every application's time into shares of that application's own
 * phase total, averages an operator's shares over the phases it runs in, and only then weights by
 * the card-hour fractions:
 *   Eq. 2  D[i][a][phi] = summed duration_ns of operator i's records of application a in phase phi
 *          D_a[phi]     = sum over all operators of D[.][a][phi]
 *   Eq. 3  wtilde_i = sum_a p_a * (1/|Phi_i|) * sum_{phi in Phi_i} D[i][a][phi] / D_a[phi]
 *          w_i      = wtilde_i / sum of wtilde_j over the retained operators j;  sum_i w_i = 1
 *   with p_a = app_weights[a] / sum(app_weights) and Phi_i = the phases in which operator i has any time.
 * A record is valid iff app_id < n_apps, op_id < n_ops and phase < n_phases (others are counted as
 * rejected; shape_id is not used: the weights are per operator).  A phase in which an application has
 * no time contributes nothing for that application; operators without time or not retained get 0.
 * Sums run in ascending phase, application and operator order, each operation rounded once, so the
 * results are bit-reproducible.  n_apps * n_ops * n_phases <= 2^28 (else ATREX_ERR_TOO_LARGE).
 *
 * create     app_weights: HOST, copied.  The library allocates its own device memory.
 * ingest     d_records: DEVICE, 16-byte aligned; asynchronous; any number of calls; order-independent.
 * finalize   h_retained: HOST n_ops flags (NULL = all retained); h_w, h_wtilde (may be NULL): HOST
 *            n_ops doubles; h_rejected (may be NULL): HOST.  Synchronises `stream`; repeatable. */
typedef struct atrex_eq3 atrex_eq3_t;
int atrex_eq3_create(uint32_t n_apps, uint32_t n_ops, uint32_t n_phases, const uint32_t* app_weights, int32_t device,
                     atrex_eq3_t** out);
int atrex_eq3_ingest(atrex_eq3_t*, const atrex_record_t* d_records, uint64_t n, void* stream);
int atrex_eq3_finalize(atrex_eq3_t*, const uint8_t* h_retained, double* h_w, double* h_wtilde, uint64_t* h_rejected,
                       void* stream);
int atrex_eq3_reset(atrex_eq3_t*, void* stream);
void atrex_eq3_destroy(atrex_eq3_t*);

/* Roofline score aggregation (Sec. 3.6, Eq. 4-6), batched over candidates.  No handle.
 *   Eq. 4  S_j = roofline_s[j] / t_cand[c][j] for every unit j = (operator, shape) of candidate c with
 *          correct[c][j] != 0.  A value above 1 is an evaluation error: it is counted and NOT clipped.
 *          A correct unit whose time is not a finite positive number is counted as an error too and
 *          left out.
 *   Eq. 5  S_i = median of operator i's S_j (even count: mean of the two middle values), 0 if operator
 *          i has no usable correct shape.
 *   Eq. 6  S_agg = sum_i w[i] * S_i, accumulated in operator order.
 * All pointers are DEVICE memory:
 *   d_roofline_s [n_units] doubles (e.g. the roofline_s of finalize's entries), d_unit_op [n_units]
 *   operator index of each unit (any order; units with an index >= n_ops are ignored),
 *   d_t_cand [n_candidates][n_units] doubles, d_correct [n_candidates][n_units] bytes, d_w [n_ops];
 *   outputs d_s_agg [n_candidates], d_s_op [n_candidates][n_ops] (may be NULL), d_errors
 *   [n_candidates] u64 (may be NULL).
 * n_units <= ATREX_SCORE_MAX_UNITS, n_ops <= ATREX_SCORE_MAX_OPS (else ATREX_ERR_TOO_LARGE).
 * Asynchronous on `stream`.  Results are bit-reproducible: one round-to-nearest division per unit, an
 * exact median, and products and sums rounded one by one in operator order. */
#define ATREX_SCORE_MAX_UNITS 16384u
#define ATREX_SCORE_MAX_OPS 4096u
int atrex_score_aggregate(const double* d_roofline_s, const uint32_t* d_unit_op, uint64_t n_units,
                          const double* d_t_cand, const uint8_t* d_correct, uint64_t n_candidates,
                          const double* d_w, uint32_t n_ops, double* d_s_agg, double* d_s_op,
                          uint64_t* d_errors, void* stream);

/* ---- Release artefacts: the entry list in key order, and the ranked list of one phase with its
 * running share and coverage cut (Table 2: operators ordered by weight with a "Cum." column; Sec. 3.3:
 * the weights are shipped as an artefact of their own and recomputed on refresh).
 *
 * Both calls work on an array of entries on the DEVICE (atrex_agg_finalize's output, or the
 * concatenation of several shards' outputs), one entry per key, and on caller-provided DEVICE
 * scratch of at least atrex_release_scratch_bytes(n) bytes, 256-byte aligned, whose contents are
 * undefined afterwards.  n <= ATREX_RELEASE_MAX_ENTRIES (else ATREX_ERR_TOO_LARGE; the scratch
 * size query then returns 0).  Too little scratch gives ATREX_ERR_NOMEM.  Input and output must
 * not overlap.  Both synchronise `stream` and run on the device that holds d_entries. */
#define ATREX_RELEASE_MAX_ENTRIES (1u << 28)
uint64_t atrex_release_scratch_bytes(uint64_t n);

/* d_out[0..n) = the entries ordered by packed key ascending (phase, then operator, then shape):
 * a canonical order for a stored artefact, independent of table geometry and sharding.  Entries
 * with equal keys (not produced by this library) keep their input order. */
int atrex_entries_sort_by_key(const atrex_entry_t* d_entries, uint64_t n, atrex_entry_t* d_out,
                              void* d_scratch, uint64_t scratch_bytes, void* stream);

typedef struct {
    uint64_t n_phase;                  /* entries of the phase                                   */
    uint64_t n_keep;                   /* coverage cut: length of the shortest sufficient prefix */
    uint64_t total_lo, total_hi;       /* T: sum of the phase's weighted times                   */
    uint64_t covered_lo, covered_hi;   /* weighted time of the first n_keep ranked entries       */
} atrex_rank_result_t;

/* The entries of `phase` ranked by weighted time descending (exact 128-bit compare), equal times
 * by key ascending -- the order of atrex_agg_topk, for the whole phase.
 *   d_ranked, d_cum_share   DEVICE, capacity out_cap each (may be NULL with out_cap 0): the first
 *                           min(n_phase, out_cap) ranked entries, and beside each its running
 *                           share cum[i] = fl(fl(wt_0 + ... + wt_i) / fl(T)).  The running sum is an
 *                           exact integer, rounded once per row, so the column is bit-reproducible and
 *                           ends at exactly 1.0; T = 0 gives +0.0.
 *   coverage_ppm            target share in millionths (<= 10^6).  n_keep is the smallest k with
 *                           10^6 * (wt_0 + ... + wt_{k-1}) >= coverage_ppm * T in integers: the hot set
 *                           that covers the target.  0 when coverage_ppm = 0 or T = 0; entries of
 *                           weight zero are never needed.
 *   h_result                HOST.
 * T is computed from the entries passed in (it must be below 2^108, else ATREX_ERR_TOO_LARGE), so the
 * list has to hold the whole phase for the shares to be Eq. 3's. */
int atrex_entries_rank(const atrex_entry_t* d_entries, uint64_t n, uint32_t phase, uint32_t coverage_ppm,
                       atrex_entry_t* d_ranked, double* d_cum_share, uint64_t out_cap,
                       atrex_rank_result_t* h_result, void* d_scratch, uint64_t scratch_bytes, void* stream);

/* Ranked top-k over an array of entries, for callers that cannot allocate device memory.
 *
 * (The paper has no counterpart to this call; it exists for deployment reasons only.)
 *
 * Who this is for: code that runs where nobody may call cudaMalloc -- a service whose device
 * memory was divided up at start-up, a plugin that receives buffers but no allocator, a process
 * whose memory pool belongs to another component.  atrex_agg_topk ranks out of a handle's
 * workspace, and that workspace had to be allocated by someone.  This call takes no handle: it
 * ranks `n` entries the caller already holds on the device (for instance atrex_agg_finalize's
 * output, or entries received from elsewhere) and keeps its selection buffer in a fixed array
 * inside the library image.  It calls no cudaMalloc, cudaFree or other allocating routine.
 *
 *   d_entries  DEVICE, n entries (8-byte aligned); key, wt_lo, wt_hi decide the ranking, the
 *              whole 48-byte entry is copied to the output unchanged
 *   n, k       at most ATREX_STATIC_TOPK_MAX_ENTRIES each; larger values are refused with
 *              ATREX_ERR_TOO_LARGE and nothing runs
 *   d_out      DEVICE, capacity k entries: the min(k, entries of `phase`) best entries of that
 *              phase, by weighted time descending (exact 128-bit compare), then key ascending
 *   h_n_out    HOST, number of entries written
 *
 * The fixed array costs 2 MiB + 256 bytes of device memory on every GPU that loads the library,
 * until the process exits.  All calls on a device share it and it keeps the previous call's
 * contents, so the call clears it first; two calls whose GPU work overlaps (different streams
 * or threads) would race on it -- keep them ordered.  The first call on each device also looks
 * up the array's device address; make that first call outside any stream capture.  The call
 * synchronises `stream` before returning. */
#define ATREX_STATIC_TOPK_MAX_ENTRIES 65536u
int atrex_topk_entries_static(const atrex_entry_t* d_entries, uint64_t n, uint32_t phase, uint32_t k,
                              atrex_entry_t* d_out, uint32_t* h_n_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ATREX_AGG_H */
