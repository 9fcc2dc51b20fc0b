// C ABI of the trace-aggregation library: argument checks, workspace carving, launches.
// The declarations and their contracts are in include/atrex_agg.h.
#include <cmath>
#include <cstddef>
#include <cstdlib>
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "kernels.h"

using namespace atrex;

namespace {

constexpr size_t ALIGN = 256;
constexpr size_t STAGING_BYTES = 64ull << 20;          // per staging buffer (two of them)
constexpr uint32_t LP_MIN = 8, LP_MAX = 12;             // 256 .. 4096 partitions
constexpr ull MAX_KEYS = 1ull << 25;
constexpr ull MAX_RECORDS_TOTAL = 1ull << 40;
constexpr uint32_t HOT_MIN_RECORDS = 32768;             // smaller calls run without a directory
constexpr uint32_t HOT_SAMPLE = 1u << 20;
constexpr uint32_t CAND_BITS = 17;                     // candidate table of the directory build
constexpr size_t SKETCH_BYTES = (size_t)4 << 20;        // 2^20 counters (ingest.cu SKETCH_BITS)
constexpr size_t HOT_SCRATCH_BYTES = SKETCH_BYTES + ((size_t)12 << CAND_BITS);
constexpr uint32_t SEL_CAP = ATREX_MAX_TOPK + TOPK_CAND_CAP;

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// A named range around each entry point's host work, for timelines taken with a tracing tool (the
// header-only NVTX: a no-op costing one pointer check when no tool is attached).
struct TraceRange {
    explicit TraceRange(const char* name) { nvtxRangePushA(name); }
    ~TraceRange() { nvtxRangePop(); }
    TraceRange(const TraceRange&) = delete;
    TraceRange& operator=(const TraceRange&) = delete;
};

ull pow2_at_least(ull x) {
    ull p = 1;
    while (p < x) p <<= 1;
    return p;
}

struct Layout {
    size_t off_ctl, off_keys, off_vals, off_work, off_appw, off_hot, off_staging[2], off_sel, off_topk_out, off_hist_all,
        off_spill_cnt, off_spill, off_hot_scratch, off_queue, off_hot_img, total;
    ull n_slots, work_slots;
    uint32_t lp, C;              // partitions = 1 << lp, slots per partition
    uint32_t Cw;                 // work-table slots per partition
    uint32_t n_groups, cap;      // spill buffers: [P][n_groups][cap] entries
    ull sub_launch;              // records per scatter + partition launch pair
    uint32_t hot_slots;
    uint32_t queue_cap;        // deferred entries per CTA in the partition pass
    bool appw_in_smem;
};

bool config_ok(const atrex_agg_config_t* c) {
    if (!c) return false;
    if (c->n_apps == 0 || c->n_phases == 0 || c->n_phases > ATREX_MAX_PHASES) return false;
    if (c->max_keys == 0 || c->max_keys > MAX_KEYS) return false;
    if (c->max_work_rows > (1ull << 30)) return false;
    return true;
}

void compute_layout(const atrex_agg_config_t* c, size_t smem_optin, int n_sms, Layout* L) {
    // Partition geometry: one partition's keys + per-launch accumulators (20 B per slot) must fit one
    // SM's shared memory.  A key can only live in its hash partition, so a partition is sized for the
    // tail of its load, not for the mean: with m = max_keys / P keys expected, the keys of one
    // (operator, shape) -- up to n_phases of them -- always fall together, which bounds the standard
    // deviation by sqrt(n_phases * m); six of those plus a constant, and never less than 1.3 m.
    const uint32_t c_max = (uint32_t)((smem_optin - 2048) / 20) & ~127u;
    auto slots_for = [&](uint32_t lp) -> ull {
        const ull m = (c->max_keys + (1ull << lp) - 1) >> lp;
        const ull flat = m + m * 3 / 10 + 1;
        const ull tail = m + (ull)std::ceil(6.0 * std::sqrt((double)c->n_phases * (double)m)) + 32;
        return flat > tail ? flat : tail;
    };
    L->lp = LP_MIN;
    while (L->lp < LP_MAX && slots_for(L->lp) > c_max) ++L->lp;
    ull per = slots_for(L->lp);
    if (per > c_max || L->lp > LP_MIN) per = c_max;  // big tables: use all of shared memory, lower load factor
    if (per < 128) per = 128;
    L->C = (uint32_t)((per + 31) / 32 * 32);
    L->n_slots = (ull)L->C << L->lp;
    L->n_groups = (uint32_t)n_sms;
    L->sub_launch = c->max_keys >= (1ull << 21) ? (1ull << 27) : (c->max_keys >= (1ull << 16) ? (1ull << 25) : (1ull << 24));
    // room for 4.5 launches' worth of entries if every record spilled; a drain is requested when a
    // buffer passes 3/4 of that, which leaves more than one full launch of headroom.  At the bench
    // workload (half of the records spill) four launches accumulate between drains.
    ull per_buf = (L->sub_launch * 9 / 2) / (((ull)n_sms) << L->lp);
    if (per_buf < 64) per_buf = 64;
    if (per_buf > 32768) per_buf = 32768;   // the scatter pass counts a buffer's entries in 16 bits, with headroom
    L->cap = (uint32_t)((per_buf + 31) / 32 * 32);   // a buffer is a whole number of 128-byte lines
    // entries of one partition whose first look fails wait in a per-CTA queue, one segment per warp:
    // room for a quarter of the partition's worst-case stream, at most 32 K entries (a warp whose
    // segment could not take another batch of 128 settles it first), at least two batches per warp
    {
        ull q = (ull)L->cap * n_sms / 4;
        L->queue_cap = (uint32_t)(q < 8192 ? 8192 : (q > 32768 ? 32768 : q));
    }
    // work table: same partitions as the key table, 1.5 slots per row plus slack for uneven partitions
    L->Cw = c->max_work_rows ? (uint32_t)((((c->max_work_rows * 3 / 2) >> L->lp) + 64 + 31) / 32 * 32) : 0;
    L->work_slots = (ull)L->Cw << L->lp;
    L->appw_in_smem = c->n_apps <= APPW_SMEM_MAX;
    L->hot_slots = scatter_hot_slots(L->lp);   // what the scatter pass's shared memory holds for this partition count
    if (c->flags & ATREX_FLAG_NO_HOT_DIRECTORY) L->hot_slots = 0;
    size_t o = 0;
    L->off_ctl = o;            o += round_up(sizeof(Control), ALIGN);
    L->off_keys = o;           o += round_up(L->n_slots * 8, ALIGN);
    L->off_vals = o;           o += round_up(L->n_slots * 16, ALIGN);
    L->off_work = o;           o += round_up(L->work_slots * sizeof(WorkSlot), ALIGN);
    L->off_appw = o;           o += round_up((size_t)c->n_apps * 4, ALIGN);
    L->off_hot = o;            o += round_up((size_t)(L->hot_slots ? L->hot_slots : 2) * 8, ALIGN);
    L->off_hot_img = o;        o += round_up((size_t)L->n_groups * (L->hot_slots ? L->hot_slots : 2) * 16, ALIGN);
    L->off_staging[0] = o;     o += STAGING_BYTES;
    L->off_staging[1] = o;     o += STAGING_BYTES;
    L->off_sel = o;            o += round_up((size_t)SEL_CAP * 32 * c->n_phases, ALIGN);   // one region per phase
    L->off_hist_all = o;       o += round_up((size_t)ATREX_MAX_PHASES * TOPK_BINS * 4, ALIGN);
    L->off_topk_out = o;       o += round_up((size_t)ATREX_MAX_TOPK * sizeof(atrex_entry_t), ALIGN);
    L->off_hot_scratch = o;    o += round_up(HOT_SCRATCH_BYTES, ALIGN);
    L->off_queue = o;          o += round_up((size_t)L->n_groups * L->queue_cap * 16, ALIGN);
    L->off_spill_cnt = o;      o += round_up(((size_t)L->n_groups << L->lp) * 4, ALIGN);
    L->off_spill = o;          o += round_up(((size_t)L->n_groups << L->lp) * L->cap * SPILL_ENTRY_BYTES, ALIGN) + ALIGN;  // + prefetch overrun
    L->total = o;
}

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) cudaSetDevice(dev);
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

}  // namespace

// What one ranking request worked out for every phase, kept until the next finalize: the
// first-digit histograms (one pass over the table for all phases) and, for the last k asked for,
// each phase's selection (one more pass for all phases).  A second phase's top-k of the same k then
// costs no pass over the table at all.
struct TopkCache {
    ull hist_gen = 0;                       // finalize generation the histograms belong to (0 = none)
    ull sel_gen = 0;                        // ... and the selections
    uint32_t k = 0;                         // k the selections were made for
    ull total[ATREX_MAX_PHASES] = {};       // candidates collected per phase
};

struct atrex_agg {
    atrex_agg_config_t cfg;
    Layout L;
    int n_sms = 0;
    bool owns_workspace = false;
    unsigned char* ws = nullptr;
    Control* ctl = nullptr;
    ull* keys = nullptr;
    ulonglong2* vals = nullptr;
    uint32_t* spill_cnt = nullptr;
    unsigned char* spill = nullptr;
    ulonglong2* queue = nullptr;
    unsigned char* hot_scratch = nullptr;
    WorkSlot* work = nullptr;
    uint32_t* d_appw = nullptr;
    ull* hot_keys = nullptr;
    ulonglong2* hot_img = nullptr;   // [n_groups][hot_slots] per-CTA directory sums not yet in the table
    bool hot_dirty = false;          // the image rows may hold sums
    unsigned char* staging[2] = {nullptr, nullptr};
    ull* sel = nullptr;
    atrex_entry_t* topk_out = nullptr;
    Control* h_ctl = nullptr;  // pinned mirror
    uint32_t* hist_all = nullptr;     // [ATREX_MAX_PHASES][TOPK_BINS] first-digit histograms of all phases
    uint32_t* h_hist_all = nullptr;   // pinned mirror
    TopkCache topk;
    ull fin_gen = 0;                  // bumped by every successful finalize
    bool hot_ready = false;
    bool finalized = false;
    bool spill_pending = false;   // entries may sit in the spill buffers
    ull scatter_seq = 0;          // sequence number of the last scatter launch
    atrex_hw_peaks_t peaks;
    ull n_records = 0;
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_ready[2] = {nullptr, nullptr}, ev_free[2] = {nullptr, nullptr};
    int last_cuda_error = 0;
    uint64_t launches = 0;

    // eight odd primes, one per byte, that do not divide m (m even or a power of two times such a number:
    // the strides are then coprime to it)
    static ull strides_for(uint32_t m) {
        ull strides = 0;
        uint32_t n = 0;
        for (uint32_t c = 7; n < 8; c += 2) {
            bool prime = true;
            for (uint32_t d = 3; d * d <= c; d += 2) prime = prime && (c % d != 0);
            if (prime && m % c != 0) strides |= (ull)c << (8 * n++);
        }
        return strides;
    }
    TableRef table_ref() const {
        TableRef t;
        t.keys = keys;
        t.vals = vals;
        t.lp = L.lp;
        t.C = L.C;
        t.ctl = ctl;
        t.strides = strides_for(L.C / 2);   // in slot pairs
        return t;
    }
    WorkRef work_ref() const {
        WorkRef w;
        w.table = L.work_slots ? work : nullptr;
        w.lp = L.lp;
        w.Cw = L.Cw;
        w.strides = strides_for(L.Cw ? L.Cw : 1);
        return w;
    }
    int scan_grid(ull n_items, int threads) const {
        ull g = (n_items + threads - 1) / threads;
        ull cap = (ull)n_sms * 8;
        if (g > cap) g = cap;
        return g < 1 ? 1 : (int)g;
    }
};

#define CU(h, call)                                   \
    do {                                              \
        cudaError_t e_ = (call);                      \
        if (e_ != cudaSuccess) {                      \
            (h)->last_cuda_error = (int)e_;           \
            return ATREX_ERR_CUDA;                    \
        }                                             \
    } while (0)

static int device_status_to_error(const Control* c) {
    if (c->status & ST_BOUNDS) return ATREX_ERR_BOUNDS;
    if (c->status & ST_TIMEOUT) return ATREX_ERR_TIMEOUT;
    if (c->status & ST_TABLE_FULL) return ATREX_ERR_CAPACITY;
    return ATREX_OK;
}

static int query_sm_count(int device) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || v <= 0) {
        cudaGetLastError();
        return 148;  // B200
    }
    return v;
}

static int query_smem_optin(int device, size_t* out) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess) return -1;
    *out = (size_t)v;
    return 0;
}

extern "C" {

uint64_t atrex_agg_workspace_bytes(const atrex_agg_config_t* cfg) {
    if (!config_ok(cfg)) return 0;
    // the directory size depends on the device's shared memory; without a device, size for
    // the sm_100 maximum (the layout only grows with it)
    size_t smem = 232448;
    size_t q;
    if (query_smem_optin(cfg->device, &q) == 0 && q > 0) smem = q;
    Layout L;
    compute_layout(cfg, smem, query_sm_count(cfg->device), &L);
    return L.total;
}

int atrex_agg_create(const atrex_agg_config_t* cfg, atrex_agg_t** out) {
    if (!out) return ATREX_ERR_INVALID;
    *out = nullptr;
    if (!config_ok(cfg) || !cfg->app_weights) return ATREX_ERR_INVALID;
    if (cfg->workspace && ((uintptr_t)cfg->workspace % ALIGN) != 0) return ATREX_ERR_INVALID;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device < 0 || cfg->device >= n_dev) {
        cudaGetLastError();
        return ATREX_ERR_CUDA;
    }
    atrex_agg* h = new (std::nothrow) atrex_agg;
    if (!h) return ATREX_ERR_NOMEM;
    h->cfg = *cfg;
    h->cfg.app_weights = nullptr;
    DeviceGuard guard(cfg->device);
    size_t smem = 0;
    int rc = ATREX_OK;
    do {
        if (query_smem_optin(cfg->device, &smem) != 0) { rc = ATREX_ERR_CUDA; break; }
        if (cudaDeviceGetAttribute(&h->n_sms, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess) { rc = ATREX_ERR_CUDA; break; }
        compute_layout(cfg, smem, h->n_sms, &h->L);
        if (cfg->workspace) {
            if (cfg->workspace_bytes < h->L.total) { rc = ATREX_ERR_NOMEM; break; }
            h->ws = (unsigned char*)cfg->workspace;
        } else {
            if (cudaMalloc((void**)&h->ws, h->L.total) != cudaSuccess) { cudaGetLastError(); rc = ATREX_ERR_NOMEM; break; }
            h->owns_workspace = true;
        }
        const Layout& L = h->L;
        h->ctl = (Control*)(h->ws + L.off_ctl);
        h->keys = (ull*)(h->ws + L.off_keys);
        h->vals = (ulonglong2*)(h->ws + L.off_vals);
        h->spill_cnt = (uint32_t*)(h->ws + L.off_spill_cnt);
        h->spill = h->ws + L.off_spill;
        h->queue = (ulonglong2*)(h->ws + L.off_queue);
        h->hot_scratch = h->ws + L.off_hot_scratch;
        h->work = (WorkSlot*)(h->ws + L.off_work);
        h->d_appw = (uint32_t*)(h->ws + L.off_appw);
        h->hot_keys = (ull*)(h->ws + L.off_hot);
        h->hot_img = (ulonglong2*)(h->ws + L.off_hot_img);
        h->staging[0] = h->ws + L.off_staging[0];
        h->staging[1] = h->ws + L.off_staging[1];
        h->sel = (ull*)(h->ws + L.off_sel);
        h->topk_out = (atrex_entry_t*)(h->ws + L.off_topk_out);
        h->hist_all = (uint32_t*)(h->ws + L.off_hist_all);
        cudaError_t e = cudaSuccess;
        if (e == cudaSuccess) e = cudaMemset(h->ws + L.off_ctl, 0, L.off_appw - L.off_ctl);  // control, table, work
        if (e == cudaSuccess) e = cudaMemcpy(h->d_appw, cfg->app_weights, (size_t)cfg->n_apps * 4, cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemset(h->hot_keys, 0, (size_t)(L.hot_slots ? L.hot_slots : 2) * 8);
        if (e == cudaSuccess) e = cudaMemset(h->hot_img, 0, (size_t)L.n_groups * (L.hot_slots ? L.hot_slots : 2) * 16);
        if (e == cudaSuccess) e = cudaMemset(h->spill_cnt, 0, ((size_t)L.n_groups << L.lp) * 4);
        if (e == cudaSuccess) e = cudaHostAlloc((void**)&h->h_ctl, sizeof(Control), cudaHostAllocDefault);
        if (e == cudaSuccess)
            e = cudaHostAlloc((void**)&h->h_hist_all, (size_t)ATREX_MAX_PHASES * TOPK_BINS * 4, cudaHostAllocDefault);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking);
        for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
            e = cudaEventCreateWithFlags(&h->ev_ready[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_free[i], cudaEventDisableTiming);
        }
        if (e == cudaSuccess) e = ingest_prepare();
        if (e == cudaSuccess) e = finalize_prepare();
        if (e == cudaSuccess) e = cudaDeviceSynchronize();
        if (e != cudaSuccess) { h->last_cuda_error = (int)e; rc = ATREX_ERR_CUDA; break; }
    } while (0);
    if (rc != ATREX_OK) {
        atrex_agg_destroy(h);
        return rc;
    }
    *out = h;
    return ATREX_OK;
}

void atrex_agg_destroy(atrex_agg_t* h) {
    if (!h) return;
    DeviceGuard guard(h->cfg.device);
    cudaDeviceSynchronize();
    for (int i = 0; i < 2; ++i) {
        if (h->ev_ready[i]) cudaEventDestroy(h->ev_ready[i]);
        if (h->ev_free[i]) cudaEventDestroy(h->ev_free[i]);
    }
    if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
    if (h->h_ctl) cudaFreeHost(h->h_ctl);
    if (h->h_hist_all) cudaFreeHost(h->h_hist_all);
    if (h->owns_workspace && h->ws) cudaFree(h->ws);
    delete h;
}

int atrex_agg_reset(atrex_agg_t* h, void* stream) {
    TraceRange range("atrex_agg_reset");
    if (!h) return ATREX_ERR_INVALID;
    DeviceGuard guard(h->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    CU(h, cudaMemsetAsync(h->ctl, 0, sizeof(Control), s));
    CU(h, cudaMemsetAsync(h->keys, 0, h->L.off_work - h->L.off_keys, s));  // keys and vals
    CU(h, cudaMemsetAsync(h->spill_cnt, 0, ((size_t)h->L.n_groups << h->L.lp) * 4, s));  // discard undrained entries
    if (h->hot_dirty) CU(h, cudaMemsetAsync(h->hot_img, 0, (size_t)h->L.n_groups * (h->L.hot_slots ? h->L.hot_slots : 2) * 16, s));
    h->hot_dirty = false;
    h->spill_pending = false;
    h->hot_ready = false;
    h->finalized = false;
    h->n_records = 0;
    return ATREX_OK;
}

int atrex_agg_set_work_table(atrex_agg_t* h, const atrex_work_t* rows, uint64_t n, void* stream) {
    TraceRange range("atrex_agg_set_work_table");
    if (!h || (n && !rows) || n > h->cfg.max_work_rows) return ATREX_ERR_INVALID;
    DeviceGuard guard(h->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    if (h->L.work_slots == 0) return ATREX_OK;
    CU(h, cudaMemsetAsync(h->work, 0, h->L.work_slots * sizeof(WorkSlot), s));
    CU(h, cudaMemsetAsync(&h->ctl->work_status, 0, sizeof(ull), s));
    const uint64_t per_piece = STAGING_BYTES / sizeof(atrex_work_t);
    for (uint64_t off = 0; off < n; off += per_piece) {
        uint64_t m = n - off < per_piece ? n - off : per_piece;
        CU(h, cudaMemcpyAsync(h->staging[0], rows + off, m * sizeof(atrex_work_t), cudaMemcpyHostToDevice, s));
        CU(h, launch_work_insert((const atrex_work_t*)h->staging[0], m, h->work_ref(), h->ctl, h->scan_grid(m, 256), s));
        h->launches++;
        CU(h, cudaStreamSynchronize(s));  // the staging buffer and the host rows are reused
    }
    CU(h, cudaMemcpyAsync(h->h_ctl, h->ctl, sizeof(Control), cudaMemcpyDeviceToHost, s));
    CU(h, cudaStreamSynchronize(s));
    h->finalized = false;
    if (h->h_ctl->work_status != 0) {
        CU(h, cudaMemsetAsync(h->work, 0, h->L.work_slots * sizeof(WorkSlot), s));
        CU(h, cudaStreamSynchronize(s));
        return ATREX_ERR_INVALID;
    }
    return ATREX_OK;
}

// Partition pass over the spill buffers.  Unforced, the kernel exits at once unless the scatter
// launch just before it saw a buffer more than 3/4 full; forced (before results are read), it
// drains whatever is there.
static int drain_spill(atrex_agg* h, bool force, cudaStream_t s) {
    if (force && !h->spill_pending) return ATREX_OK;
    PartitionParams q;
    q.t = h->table_ref();
    q.spill = h->spill;
    q.spill_cnt = h->spill_cnt;
    q.n_groups = h->L.n_groups;
    q.n_used = h->L.n_groups;
    q.cap = h->L.cap;
    q.queue = h->queue;
    q.queue_cap = h->L.queue_cap;
    q.force = force ? 1u : 0u;
    q.seq = h->scatter_seq;
    CU(h, cudaMemsetAsync(&h->ctl->part_cursor, 0, sizeof(ull), s));
    CU(h, launch_partition(q, h->n_sms, s));
    h->launches++;
    if (force && h->hot_dirty) {
        // results are about to be read: the directory sums kept per scatter CTA join the table
        CU(h, launch_hot_fold(h->hot_keys, h->hot_img, h->L.n_groups, h->L.hot_slots, h->table_ref(), s));
        h->launches++;
        h->hot_dirty = false;
    }
    if (force) h->spill_pending = false;
    return ATREX_OK;
}

static int ingest_launch(atrex_agg* h, const atrex_record_t* recs, uint64_t n, cudaStream_t s) {
    // hot directory from a sample of the first sufficiently large call after create/reset
    if (h->L.hot_slots && !h->hot_ready && n >= HOT_MIN_RECORDS) {
        HotBuildParams b;
        b.recs = (const uint4*)recs;
        b.n_sample = (uint32_t)(n < HOT_SAMPLE ? n : HOT_SAMPLE);
        b.stride = n / b.n_sample;
        b.n_apps = h->cfg.n_apps;
        b.n_phases = h->cfg.n_phases;
        b.hot_keys = h->hot_keys;
        b.hot_slots = h->L.hot_slots;
        b.ctl = h->ctl;
        b.sketch = (uint32_t*)h->hot_scratch;
        b.cand_keys = (ull*)(h->hot_scratch + SKETCH_BYTES);
        b.cand_cnt = (uint32_t*)(h->hot_scratch + SKETCH_BYTES + ((size_t)8 << CAND_BITS));
        b.cand_bits = CAND_BITS;
        CU(h, cudaMemsetAsync(h->hot_scratch, 0, HOT_SCRATCH_BYTES, s));
        CU(h, launch_hot_build(b, h->n_sms, s));
        h->launches += 3;
        h->hot_ready = true;
    }
    IngestParams p;
    memset(&p, 0, sizeof(p));
    const unsigned char* base = (const unsigned char*)recs;
    uint64_t head = (((uintptr_t)base & 31u) != 0 && n > 0) ? 1 : 0;
    uint64_t n_body = n - head;
    p.recs = recs;
    p.n_recs = n;
    p.body = base + head * 16;
    p.n_pairs = n_body / 2;
    p.n_single = 0;
    if (head) p.single[p.n_single++] = base;
    if (n_body & 1) p.single[p.n_single++] = base + (n - 1) * 16;
    p.n_apps = h->cfg.n_apps;
    p.n_phases = h->cfg.n_phases;
    p.phase_lim = h->cfg.n_phases << 16;
    p.appw_in_smem = h->L.appw_in_smem ? 1u : 0u;
    p.app_w = h->d_appw;
    p.hot_keys = h->hot_keys;
    p.hot_slots = h->L.hot_slots;
    p.hot_buckets = h->L.hot_slots / 4;
    p.hot_img = h->hot_img;
    p.t = h->table_ref();
    p.spill = h->spill;
    p.spill_cnt = h->spill_cnt;
    p.n_groups = h->L.n_groups;
    p.cap = h->L.cap;
    const ull pairs_per_cta_iter = 2048;
    ull want = (p.n_pairs + pairs_per_cta_iter - 1) / pairs_per_cta_iter;
    int grid = (int)(want < 1 ? 1 : (want > (ull)h->n_sms ? (ull)h->n_sms : want));
    p.drain_above = h->L.cap / 4 * 3;
    p.seq = ++h->scatter_seq;
    CU(h, launch_scatter(p, h->hot_ready, grid, s));
    if (h->hot_ready) h->hot_dirty = true;
    h->spill_pending = true;
    h->launches++;
    return drain_spill(h, /*force=*/false, s);
}

int atrex_agg_ingest(atrex_agg_t* h, const atrex_record_t* d_records, uint64_t n, void* stream) {
    TraceRange range("atrex_agg_ingest");
    if (!h) return ATREX_ERR_INVALID;
    if (n == 0) return ATREX_OK;
    if (!d_records || ((uintptr_t)d_records & 15u) != 0) return ATREX_ERR_INVALID;
    if (h->n_records + n >= MAX_RECORDS_TOTAL) return ATREX_ERR_STATE;
    DeviceGuard guard(h->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    h->finalized = false;
    for (uint64_t off = 0; off < n; off += h->L.sub_launch) {
        uint64_t m = n - off < h->L.sub_launch ? n - off : h->L.sub_launch;
        int rc = ingest_launch(h, d_records + off, m, s);
        if (rc != ATREX_OK) return rc;
    }
    h->n_records += n;
    return ATREX_OK;
}

int atrex_agg_ingest_host(atrex_agg_t* h, const atrex_record_t* h_records, uint64_t n, void* stream) {
    TraceRange range("atrex_agg_ingest_host");
    if (!h) return ATREX_ERR_INVALID;
    if (n == 0) return ATREX_OK;
    if (!h_records) return ATREX_ERR_INVALID;
    if (h->n_records + n >= MAX_RECORDS_TOTAL) return ATREX_ERR_STATE;
    DeviceGuard guard(h->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    h->finalized = false;
    const uint64_t per_piece = STAGING_BYTES / sizeof(atrex_record_t);
    int b = 0;
    for (uint64_t off = 0; off < n; off += per_piece, b ^= 1) {
        uint64_t m = n - off < per_piece ? n - off : per_piece;
        CU(h, cudaStreamWaitEvent(h->copy_stream, h->ev_free[b], 0));
        CU(h, cudaMemcpyAsync(h->staging[b], h_records + off, m * sizeof(atrex_record_t), cudaMemcpyHostToDevice, h->copy_stream));
        CU(h, cudaEventRecord(h->ev_ready[b], h->copy_stream));
        CU(h, cudaStreamWaitEvent(s, h->ev_ready[b], 0));
        int rc = ingest_launch(h, (const atrex_record_t*)h->staging[b], m, s);
        if (rc != ATREX_OK) return rc;
        CU(h, cudaEventRecord(h->ev_free[b], s));
    }
    h->n_records += n;
    return ATREX_OK;
}

int atrex_agg_merge(atrex_agg_t* h, const atrex_entry_t* d_entries, uint64_t n, void* stream) {
    TraceRange range("atrex_agg_merge");
    if (!h) return ATREX_ERR_INVALID;
    if (n == 0) return ATREX_OK;
    if (!d_entries || ((uintptr_t)d_entries & 15u) != 0) return ATREX_ERR_INVALID;
    DeviceGuard guard(h->cfg.device);
    h->finalized = false;
    CU(h, launch_merge(d_entries, n, h->table_ref(), h->scan_grid(n, 256), (cudaStream_t)stream));
    h->launches++;
    return ATREX_OK;
}

static int run_totals(atrex_agg* h, cudaStream_t s) {
    size_t off = offsetof(Control, total_lo);
    CU(h, cudaMemsetAsync((unsigned char*)h->ctl + off, 0, offsetof(Control, hist) - off, s));
    CU(h, launch_totals(h->table_ref(), h->L.n_slots, h->scan_grid(h->L.n_slots, 128 * 8), s));
    h->launches++;
    return ATREX_OK;
}

static FinalizeParams finalize_params(const atrex_agg* h, atrex_entry_t* out, uint64_t cap) {
    FinalizeParams p;
    p.t = h->table_ref();
    p.n_slots = h->L.n_slots;
    p.ctl = h->ctl;
    p.work = h->work_ref();
    p.peaks = h->peaks;
    p.out = out;
    p.out_cap = cap;
    return p;
}

static int finalize_impl(atrex_agg_t* h, const atrex_hw_peaks_t* peaks, const uint64_t* total_lo,
                         const uint64_t* total_hi, atrex_entry_t* d_out, uint64_t out_cap, uint64_t* n_out,
                         void* stream);

int atrex_agg_finalize(atrex_agg_t* h, const atrex_hw_peaks_t* peaks, atrex_entry_t* d_out, uint64_t out_cap,
                       uint64_t* n_out, void* stream) {
    return finalize_impl(h, peaks, nullptr, nullptr, d_out, out_cap, n_out, stream);
}

int atrex_agg_finalize_with_totals(atrex_agg_t* h, const atrex_hw_peaks_t* peaks, const uint64_t* total_lo,
                                   const uint64_t* total_hi, atrex_entry_t* d_out, uint64_t out_cap,
                                   uint64_t* n_out, void* stream) {
    if (!total_lo || !total_hi) return ATREX_ERR_INVALID;
    return finalize_impl(h, peaks, total_lo, total_hi, d_out, out_cap, n_out, stream);
}

static int finalize_impl(atrex_agg_t* h, const atrex_hw_peaks_t* peaks, const uint64_t* total_lo,
                         const uint64_t* total_hi, atrex_entry_t* d_out, uint64_t out_cap, uint64_t* n_out,
                         void* stream) {
    TraceRange range("atrex_agg_finalize");
    if (!h || !peaks || !n_out) return ATREX_ERR_INVALID;
    if (d_out && ((uintptr_t)d_out & 15u) != 0) return ATREX_ERR_INVALID;
    if (!d_out) out_cap = 0;
    if (!(std::isfinite(peaks->peak_bw) && peaks->peak_bw > 0)) return ATREX_ERR_INVALID;
    for (int i = 0; i < ATREX_MAX_DTYPES; ++i)
        if (!(std::isfinite(peaks->peak_flops[i]) && peaks->peak_flops[i] > 0)) return ATREX_ERR_INVALID;
    DeviceGuard guard(h->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    h->peaks = *peaks;
    int rc = drain_spill(h, /*force=*/true, s);
    if (rc != ATREX_OK) return rc;
    rc = run_totals(h, s);
    if (rc != ATREX_OK) return rc;
    if (total_lo) {
        // normalise by the totals over all shards instead of this handle's own
        CU(h, cudaMemcpyAsync(h->ctl->total_lo, total_lo, sizeof(ull) * ATREX_MAX_PHASES, cudaMemcpyHostToDevice, s));
        CU(h, cudaMemcpyAsync(h->ctl->total_hi, total_hi, sizeof(ull) * ATREX_MAX_PHASES, cudaMemcpyHostToDevice, s));
    }
    CU(h, cudaMemsetAsync(&h->ctl->n_out, 0, sizeof(ull), s));
    CU(h, launch_emit(finalize_params(h, d_out, out_cap), h->scan_grid(h->L.n_slots, 256 * 4), s));
    h->launches++;
    CU(h, cudaMemcpyAsync(h->h_ctl, h->ctl, offsetof(Control, hist), cudaMemcpyDeviceToHost, s));
    CU(h, cudaStreamSynchronize(s));
    *n_out = h->h_ctl->n_out;
    rc = device_status_to_error(h->h_ctl);
    if (rc != ATREX_OK) return rc;
    h->finalized = true;
    h->fin_gen++;
    if (d_out && h->h_ctl->n_out > out_cap) return ATREX_ERR_OUT_TOO_SMALL;
    return ATREX_OK;
}

// Radix-select plan of one phase for the best k: fixes leading digits of the ranking composite until
// the class holding the k-th entry is small enough to sort.  The first digit comes from the cached
// all-phase histograms; deeper digits (only when more than TOPK_CAND_CAP keys share the leading
// digits) take one single-phase pass each.
static int plan_phase(atrex_agg_t* h, uint32_t q, uint32_t k, TopkAllParams* all, ull* total, cudaStream_t s) {
    const ull n_phase = h->h_ctl->keys_per_phase[q];
    all->n_prefix_digits[q] = 0;
    if (n_phase == 0) {
        *total = 0;
        return ATREX_OK;
    }
    all->active_mask |= 1u << q;
    if (n_phase <= k) {
        all->collect_all_mask |= 1u << q;
        *total = n_phase;
        return ATREX_OK;
    }
    const uint32_t n_digits = (144 - all->shift[q] + 11) / 12;
    ull need = k, cand = 0;
    const uint32_t* hist = h->h_hist_all + (size_t)q * TOPK_BINS;
    while (true) {
        ull above = 0;
        int bin = TOPK_BINS - 1;
        for (; bin > 0; --bin) {
            if (above + hist[bin] >= need) break;
            above += hist[bin];
        }
        need -= above;
        cand = hist[bin];
        all->prefix_digit[q][all->n_prefix_digits[q]++] = (uint16_t)bin;
        if (cand <= TOPK_CAND_CAP || all->n_prefix_digits[q] == n_digits) break;
        // next digit of this phase alone
        TopkParams p;
        memset(&p, 0, sizeof(p));
        p.t = h->table_ref();
        p.n_slots = h->L.n_slots;
        p.ctl = h->ctl;
        p.phase = q;
        p.shift = all->shift[q];
        p.n_prefix_digits = all->n_prefix_digits[q];
        memcpy(p.prefix_digit, all->prefix_digit[q], sizeof(p.prefix_digit));
        CU(h, cudaMemsetAsync(h->ctl->hist, 0, sizeof(h->ctl->hist), s));
        CU(h, launch_topk_hist(p, h->scan_grid(h->L.n_slots, 256 * 4), s));
        h->launches++;
        CU(h, cudaMemcpyAsync(h->h_ctl->hist, h->ctl->hist, sizeof(h->ctl->hist), cudaMemcpyDeviceToHost, s));
        CU(h, cudaStreamSynchronize(s));
        hist = h->h_ctl->hist;
    }
    *total = (k - need) + cand;
    return ATREX_OK;
}

int atrex_agg_topk(atrex_agg_t* h, uint32_t phase, uint32_t k, atrex_entry_t* h_out, uint32_t* n_out, void* stream) {
    TraceRange range("atrex_agg_topk");
    if (!h || !n_out || (k && !h_out) || k > ATREX_MAX_TOPK || phase >= h->cfg.n_phases) return ATREX_ERR_INVALID;
    *n_out = 0;
    if (!h->finalized) return ATREX_ERR_STATE;
    if (k == 0) return ATREX_OK;
    DeviceGuard guard(h->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    if (h->h_ctl->keys_per_phase[phase] == 0) return ATREX_OK;
    const uint32_t n_phases = h->cfg.n_phases;
    TopkCache& cache = h->topk;

    if (cache.sel_gen != h->fin_gen || cache.k != k) {
        TopkAllParams all;
        memset(&all, 0, sizeof(all));
        all.t = h->table_ref();
        all.n_slots = h->L.n_slots;
        all.hist = h->hist_all;
        all.sel = h->sel;
        all.sel_count = h->ctl->sel_count_all;
        all.sel_cap = SEL_CAP;
        // digits start at the highest bit a phase's total has (no key's weighted time exceeds it)
        for (uint32_t q = 0; q < n_phases; ++q) {
            ull hi = h->h_ctl->total_hi[q], lo = h->h_ctl->total_lo[q];
            int top_bit = hi ? 64 + (63 - __builtin_clzll(hi)) : (lo ? 63 - __builtin_clzll(lo) : 0);
            all.shift[q] = (uint32_t)(143 - (top_bit + 56));
        }
        if (cache.hist_gen != h->fin_gen) {
            // first digit of every non-empty phase: one pass over the table
            for (uint32_t q = 0; q < n_phases; ++q)
                if (h->h_ctl->keys_per_phase[q] != 0) all.active_mask |= 1u << q;
            CU(h, cudaMemsetAsync(h->hist_all, 0, (size_t)ATREX_MAX_PHASES * TOPK_BINS * 4, s));
            CU(h, launch_topk_hist_all(all, h->n_sms, s));
            h->launches++;
            CU(h, cudaMemcpyAsync(h->h_hist_all, h->hist_all, (size_t)ATREX_MAX_PHASES * TOPK_BINS * 4,
                                  cudaMemcpyDeviceToHost, s));
            CU(h, cudaStreamSynchronize(s));
            cache.hist_gen = h->fin_gen;
            all.active_mask = 0;
        }
        for (uint32_t q = 0; q < n_phases; ++q) {
            int rc = plan_phase(h, q, k, &all, &cache.total[q], s);
            if (rc != ATREX_OK) return rc;
            if (cache.total[q] > SEL_CAP) return ATREX_ERR_STATE;  // cannot happen: composites are unique
        }
        // every phase's candidates in one pass, each into its own zero-padded region
        CU(h, cudaMemsetAsync(h->ctl->sel_count_all, 0, sizeof(h->ctl->sel_count_all), s));
        for (uint32_t q = 0; q < n_phases; ++q) {
            if (cache.total[q] == 0) continue;
            const size_t n_pow2 = pow2_at_least(cache.total[q] < 2 ? 2 : cache.total[q]);
            CU(h, cudaMemsetAsync(h->sel + (size_t)q * SEL_CAP * 4, 0, n_pow2 * 32, s));
        }
        CU(h, launch_topk_collect_all(all, h->scan_grid(h->L.n_slots, 256 * 4), s));
        h->launches++;
        for (uint32_t q = 0; q < n_phases; ++q) {   // sorted once, read by this and later calls
            if (cache.total[q] == 0) continue;
            const uint32_t n_pow2 = (uint32_t)pow2_at_least(cache.total[q] < 2 ? 2 : cache.total[q]);
            CU(h, launch_topk_sort(h->sel + (size_t)q * SEL_CAP * 4, n_pow2, s));
            h->launches++;
        }
        cache.sel_gen = h->fin_gen;
        cache.k = k;
    }
    const ull total = cache.total[phase];
    const uint32_t m = (uint32_t)(total < k ? total : k);
    CU(h, launch_topk_emit(finalize_params(h, h->topk_out, m), h->sel + (size_t)phase * SEL_CAP * 4, m, s));
    h->launches++;
    CU(h, cudaMemcpyAsync(h_out, h->topk_out, (size_t)m * sizeof(atrex_entry_t), cudaMemcpyDeviceToHost, s));
    CU(h, cudaStreamSynchronize(s));
    *n_out = m;
    return ATREX_OK;
}

int atrex_agg_totals(const atrex_agg_t* h, uint64_t* h_lo, uint64_t* h_hi) {
    if (!h || !h_lo || !h_hi) return ATREX_ERR_INVALID;
    if (!h->finalized) return ATREX_ERR_STATE;
    for (int p = 0; p < ATREX_MAX_PHASES; ++p) {
        h_lo[p] = h->h_ctl->total_lo[p];
        h_hi[p] = h->h_ctl->total_hi[p];
    }
    return ATREX_OK;
}

int atrex_agg_stats(atrex_agg_t* h, atrex_stats_t* out, void* stream) {
    TraceRange range("atrex_agg_stats");
    if (!h || !out) return ATREX_ERR_INVALID;
    DeviceGuard guard(h->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    int rc = drain_spill(h, /*force=*/true, s);
    if (rc != ATREX_OK) return rc;
    rc = run_totals(h, s);
    if (rc != ATREX_OK) return rc;
    CU(h, cudaMemcpyAsync(h->h_ctl, h->ctl, offsetof(Control, hist), cudaMemcpyDeviceToHost, s));
    CU(h, cudaStreamSynchronize(s));
    memset(out, 0, sizeof(*out));
    const Control* c = h->h_ctl;
    out->n_rejected = c->n_rejected;
    out->n_dropped = c->n_dropped;
    for (int p = 0; p < ATREX_MAX_PHASES; ++p) {
        out->total_lo[p] = c->total_lo[p];
        out->total_hi[p] = c->total_hi[p];
        out->keys_per_phase[p] = c->keys_per_phase[p];
        out->n_keys += c->keys_per_phase[p];
        out->n_valid += c->count_per_phase[p];
    }
    out->table_slots = h->L.n_slots;
    out->hot_slots = c->hot_n;
    out->n_spilled = c->n_spilled;
    out->n_overflow = c->n_overflow;
    out->max_spill_fill = c->max_fill;
    out->spill_cap = h->L.cap;
    out->n_drains = c->n_drains;
    return device_status_to_error(c);
}

int atrex_agg_hot_directory(atrex_agg_t* h, uint64_t* h_keys, uint32_t cap, uint32_t* n_out, void* stream) {
    if (!h || !n_out || (cap && !h_keys)) return ATREX_ERR_INVALID;
    *n_out = 0;
    if (!h->hot_ready || h->L.hot_slots == 0) return ATREX_OK;
    DeviceGuard guard(h->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    ull* image = (ull*)malloc((size_t)h->L.hot_slots * 8);
    if (!image) return ATREX_ERR_NOMEM;
    cudaError_t e = cudaMemcpyAsync(image, h->hot_keys, (size_t)h->L.hot_slots * 8, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        free(image);
        h->last_cuda_error = (int)e;
        return ATREX_ERR_CUDA;
    }
    uint32_t n = 0;
    for (uint32_t i = 0; i < h->L.hot_slots; ++i) {
        if (image[i] == 0) continue;
        if (n < cap) h_keys[n] = ~image[i];
        ++n;
    }
    free(image);
    *n_out = n;
    return ATREX_OK;
}

const char* atrex_strerror(int status) {
    switch (status) {
        case ATREX_OK: return "ok";
        case ATREX_ERR_INVALID: return "invalid argument";
        case ATREX_ERR_CAPACITY: return "more distinct keys than provisioned";
        case ATREX_ERR_OUT_TOO_SMALL: return "output buffer too small";
        case ATREX_ERR_CUDA: return "CUDA runtime error";
        case ATREX_ERR_TIMEOUT: return "bounded device wait gave up";
        case ATREX_ERR_STATE: return "call not valid in this state";
        case ATREX_ERR_NOMEM: return "workspace too small or allocation failed";
        case ATREX_ERR_TOO_LARGE: return "input larger than the fixed internal buffer";
        case ATREX_ERR_BOUNDS: return "checked build: a kernel index was out of range";
        default: return "unknown status";
    }
}

int atrex_build_has_bounds_checks(void) {
#ifdef ATREX_DEBUG_BOUNDS
    return 1;
#else
    return 0;
#endif
}

int atrex_agg_last_cuda_error(const atrex_agg_t* h) { return h ? h->last_cuda_error : 0; }

uint64_t atrex_agg_launch_count(const atrex_agg_t* h) { return h ? h->launches : 0; }

}  // extern "C"
