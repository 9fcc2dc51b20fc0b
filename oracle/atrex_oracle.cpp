// TEST INFRASTRUCTURE -- not part of the product path.
//
// Plain, slow, obviously-correct CPU statement of what the trace-aggregation path
// computes, written from the paper's definitions.  Only the test-suite, the smoke
// check and the benchmark's CPU-baseline leg may call it.  It shares no source,
// header, table or helper with the CUDA library; the structs below restate the byte
// layouts of the buffers independently.
//
// What it computes, per distinct (operator, shape, phase) key k:
//   count[k]  = number of valid records carrying k           (Eq. 2: the sum over the
//                                                              m_{a,phi,r} invocations)
//   wt[k]     = sum over those records of                    (Eq. 2's cumulative device
//               app_weight[app] * duration_ns, exact u128     time D, each application's
//                                                              time scaled by its card-hour
//                                                              weight as in Eq. 3's p_a)
//   T[phi]    = sum of wt[k] over keys of phase phi           (Eq. 2's per-phase total)
//   phase_weight[k] = fl(fl(wt[k]) / fl(T[phi]))              (Eq. 3's normalisation so that
//                                                              weights sum to 1, done
//                                                              separately per serving phase)
//   roofline_s[k]   = max(F/P_dtype, M/beta)                  (Eq. 1)
//   topk(phi, k)    = first k keys of phase phi by (wt descending, key ascending)
//                                                             (Table 2's ranking)
// and, downstream of the weights, the roofline score aggregation of Eq. 4-6
// (oracle_score_candidate below), the literal Eq. 2-3 operator weights (oracle_eq3_weights)
// and the ranked list with running share and coverage cut behind Table 2
// (oracle_rank_phase, oracle_sort_by_key).
//
// Readings where the paper is silent: invalid records (application or phase out of
// range) are skipped and counted; the `pad` byte is ignored; a phase whose total is zero
// gives weight +0.0; a key without a work-table row gets the quiet-NaN pattern
// 0x7FF8000000000000; ties in the ranking go to the smaller packed key; the ranking
// compares the exact integer wt, not the rounded double.
//
// Floating point: u128 -> binary64 is one round-to-nearest-even conversion (the compiler
// runtime's integer-to-double conversion), then IEEE division.  Build with
// -O2 -ffp-contract=off and without -ffast-math.
//
// Every function here is pinned by tests/test_oracle_*.py against hand-computed traces,
// closed forms, brute force in Python integers, and invariants.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <map>
#include <thread>
#include <vector>

typedef unsigned __int128 u128;

namespace {

struct Rec {
    uint32_t app_id;
    uint16_t op_id;
    uint8_t phase;
    uint8_t pad;
    uint32_t shape_id;
    uint32_t duration_ns;
};
static_assert(sizeof(Rec) == 16, "record is 16 bytes");

struct WorkRow {
    uint32_t shape_id;
    uint16_t op_id;
    uint16_t dtype;
    uint64_t flops;
    uint64_t bytes;
};
static_assert(sizeof(WorkRow) == 24, "work row is 24 bytes");

struct Entry {
    uint64_t key;
    uint64_t count;
    uint64_t wt_lo;
    uint64_t wt_hi;
    double phase_weight;
    double roofline_s;
};
static_assert(sizeof(Entry) == 48, "entry is 48 bytes");

struct Peaks {
    double peak_bw;
    double peak_flops[8];
};

struct Acc {
    uint64_t count = 0;
    u128 wt = 0;
};

typedef std::map<uint64_t, Acc> Groups;

struct Oracle {
    uint32_t n_apps = 0, n_phases = 0;
    std::vector<uint32_t> app_weight;
    Groups groups;
    std::map<uint64_t, WorkRow> work;  // (op << 32 | shape) -> row
    uint64_t n_valid = 0, n_rejected = 0;
};

inline uint64_t pack_key(const Rec& r) {
    return ((uint64_t)r.phase << 48) | ((uint64_t)r.op_id << 32) | (uint64_t)r.shape_id;
}

// Eq. 2 restricted to a slice of the trace: group-by sum into `g`.
void aggregate_slice(const Oracle& o, const Rec* recs, uint64_t n, Groups& g,
                     uint64_t& n_valid, uint64_t& n_rejected) {
    for (uint64_t i = 0; i < n; ++i) {
        const Rec& r = recs[i];
        if (r.app_id >= o.n_apps || r.phase >= o.n_phases) {
            ++n_rejected;
            continue;
        }
        Acc& a = g[pack_key(r)];
        a.count += 1;
        a.wt += (u128)o.app_weight[r.app_id] * (u128)r.duration_ns;
        ++n_valid;
    }
}

void phase_totals(const Oracle& o, u128 totals[8]) {
    for (int p = 0; p < 8; ++p) totals[p] = 0;
    for (const auto& kv : o.groups) totals[kv.first >> 48] += kv.second.wt;
}

double quiet_nan() {
    uint64_t bits = 0x7FF8000000000000ull;
    double d;
    std::memcpy(&d, &bits, 8);
    return d;
}

// Eq. 1 for one (operator, shape) unit.
double roofline_time(const Oracle& o, const Peaks& pk, uint64_t key) {
    auto it = o.work.find(key & 0x0000FFFFFFFFFFFFull);
    if (it == o.work.end()) return quiet_nan();
    const WorkRow& w = it->second;
    double t_compute = (double)w.flops / pk.peak_flops[w.dtype];
    double t_memory = (double)w.bytes / pk.peak_bw;
    return std::fmax(t_compute, t_memory);
}

Entry make_entry(const Oracle& o, const Peaks& pk, const u128 totals[8], uint64_t key, const Acc& a) {
    Entry e;
    e.key = key;
    e.count = a.count;
    e.wt_lo = (uint64_t)a.wt;
    e.wt_hi = (uint64_t)(a.wt >> 64);
    u128 t = totals[key >> 48];
    e.phase_weight = (t == 0) ? 0.0 : (double)a.wt / (double)t;  // Eq. 3, per phase
    e.roofline_s = roofline_time(o, pk, key);
    return e;
}

}  // namespace

extern "C" {

void* oracle_create(const uint32_t* app_weights, uint32_t n_apps, uint32_t n_phases) {
    if (!app_weights || n_apps == 0 || n_phases == 0 || n_phases > 8) return nullptr;
    Oracle* o = new Oracle;
    o->n_apps = n_apps;
    o->n_phases = n_phases;
    o->app_weight.assign(app_weights, app_weights + n_apps);
    return o;
}

void oracle_destroy(void* h) { delete (Oracle*)h; }

void oracle_reset(void* h) {
    Oracle* o = (Oracle*)h;
    o->groups.clear();
    o->n_valid = o->n_rejected = 0;
}

// Single-threaded ingest of n records.
void oracle_ingest(void* h, const void* records, uint64_t n) {
    Oracle* o = (Oracle*)h;
    aggregate_slice(*o, (const Rec*)records, n, o->groups, o->n_valid, o->n_rejected);
}

// Threaded variant: thread t aggregates a contiguous slice into its own map; the maps
// are merged by key with integer adds (identical by associativity).  Returns the number
// of threads used.
uint32_t oracle_ingest_threads(void* h, const void* records, uint64_t n, uint32_t threads) {
    Oracle* o = (Oracle*)h;
    if (threads == 0) threads = std::thread::hardware_concurrency();
    if (threads == 0) threads = 1;
    if (n < threads) threads = 1;
    std::vector<Groups> parts(threads);
    std::vector<uint64_t> nv(threads, 0), nr(threads, 0);
    std::vector<std::thread> pool;
    const Rec* recs = (const Rec*)records;
    for (uint32_t t = 0; t < threads; ++t) {
        uint64_t lo = n * t / threads, hi = n * (t + 1) / threads;
        pool.emplace_back([&, t, lo, hi] { aggregate_slice(*o, recs + lo, hi - lo, parts[t], nv[t], nr[t]); });
    }
    for (auto& th : pool) th.join();
    for (uint32_t t = 0; t < threads; ++t) {
        for (const auto& kv : parts[t]) {
            Acc& a = o->groups[kv.first];
            a.count += kv.second.count;
            a.wt += kv.second.wt;
        }
        o->n_valid += nv[t];
        o->n_rejected += nr[t];
    }
    return threads;
}

// Full-size spot checks: aggregate only the records whose key is in `keys` (n_keys values,
// any order).  Same definition as oracle_ingest restricted to those keys, so that sampled
// outputs of a trace too large for the full map can be computed one by one.
void oracle_ingest_filtered(void* h, const void* records, uint64_t n, const uint64_t* keys, uint64_t n_keys) {
    Oracle* o = (Oracle*)h;
    std::vector<uint64_t> want(keys, keys + n_keys);
    std::sort(want.begin(), want.end());
    const Rec* recs = (const Rec*)records;
    for (uint64_t i = 0; i < n; ++i) {
        const Rec& r = recs[i];
        if (r.app_id >= o->n_apps || r.phase >= o->n_phases) continue;
        uint64_t k = pack_key(r);
        if (!std::binary_search(want.begin(), want.end(), k)) continue;
        Acc& a = o->groups[k];
        a.count += 1;
        a.wt += (u128)o->app_weight[r.app_id] * (u128)r.duration_ns;
    }
}

// Full-size slice checks.  The key space is cut into `modulus` classes by a fixed scramble of the
// packed key (a function of the key alone -- nothing here looks at anybody's output), and only the
// valid records whose key falls into class `residue` are aggregated: the same definition as
// oracle_ingest restricted to a slice of the key space, so that a trace too large for the full map
// can still be compared entry by entry on that slice, lost and invented keys included.
// Threads aggregate contiguous runs of the records into their own maps, merged by key with integer
// adds as in oracle_ingest_threads.  Returns the number of threads used.
inline uint64_t slice_class(uint64_t key, uint64_t modulus) {
    uint64_t z = key + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    return z % modulus;
}

uint32_t oracle_ingest_slice(void* h, const void* records, uint64_t n, uint64_t modulus, uint64_t residue,
                             uint32_t threads) {
    Oracle* o = (Oracle*)h;
    if (modulus == 0) return 0;
    if (threads == 0) threads = std::thread::hardware_concurrency();
    if (threads == 0) threads = 1;
    if (n < threads) threads = 1;
    std::vector<Groups> parts(threads);
    std::vector<std::thread> pool;
    const Rec* recs = (const Rec*)records;
    for (uint32_t t = 0; t < threads; ++t) {
        uint64_t lo = n * t / threads, hi = n * (t + 1) / threads;
        pool.emplace_back([&, t, lo, hi] {
            Groups& g = parts[t];
            for (uint64_t i = lo; i < hi; ++i) {
                const Rec& r = recs[i];
                if (r.app_id >= o->n_apps || r.phase >= o->n_phases) continue;
                uint64_t k = pack_key(r);
                if (slice_class(k, modulus) != residue) continue;
                Acc& a = g[k];
                a.count += 1;
                a.wt += (u128)o->app_weight[r.app_id] * (u128)r.duration_ns;
            }
        });
    }
    for (auto& th : pool) th.join();
    for (uint32_t t = 0; t < threads; ++t) {
        for (const auto& kv : parts[t]) {
            Acc& a = o->groups[kv.first];
            a.count += kv.second.count;
            a.wt += kv.second.wt;
        }
    }
    return threads;
}

// The class oracle_ingest_slice puts a key in (exported so that a test can cut another
// implementation's output along the same lines).
void oracle_slice_classes(const uint64_t* keys, uint64_t n, uint64_t modulus, uint64_t* out) {
    for (uint64_t i = 0; i < n; ++i) out[i] = modulus ? slice_class(keys[i], modulus) : 0;
}

// Per-phase totals straight from the records, without any grouping: Eq. 2's D^phi as a plain
// sum.  acc[2p], acc[2p+1] (low, high) are updated in place so the call can be repeated per
// chunk; valid[0] / valid[1] accumulate the valid and rejected record counts.
void oracle_direct_totals(void* h, const void* records, uint64_t n, uint64_t acc[16], uint64_t valid[2]) {
    Oracle* o = (Oracle*)h;
    const Rec* recs = (const Rec*)records;
    u128 t[8];
    for (int p = 0; p < 8; ++p) t[p] = ((u128)acc[2 * p + 1] << 64) | acc[2 * p];
    for (uint64_t i = 0; i < n; ++i) {
        const Rec& r = recs[i];
        if (r.app_id >= o->n_apps || r.phase >= o->n_phases) {
            ++valid[1];
            continue;
        }
        ++valid[0];
        t[r.phase] += (u128)o->app_weight[r.app_id] * (u128)r.duration_ns;
    }
    for (int p = 0; p < 8; ++p) {
        acc[2 * p] = (uint64_t)t[p];
        acc[2 * p + 1] = (uint64_t)(t[p] >> 64);
    }
}

// Install the per-(operator, shape) semantic work table.  Returns 0, or -1 on a
// duplicate pair or a dtype index >= 8 (table left empty).
int oracle_set_work(void* h, const void* rows, uint64_t n) {
    Oracle* o = (Oracle*)h;
    o->work.clear();
    const WorkRow* w = (const WorkRow*)rows;
    for (uint64_t i = 0; i < n; ++i) {
        uint64_t k = ((uint64_t)w[i].op_id << 32) | w[i].shape_id;
        if (w[i].dtype >= 8 || !o->work.emplace(k, w[i]).second) {
            o->work.clear();
            return -1;
        }
    }
    return 0;
}

uint64_t oracle_n_keys(void* h) { return ((Oracle*)h)->groups.size(); }

// out[0] = valid records, out[1] = rejected records, out[2] = distinct keys,
// out[3 + 2p], out[4 + 2p] = low and high 64 bits of T[p] for p in 0..7.
void oracle_stats(void* h, uint64_t out[19]) {
    Oracle* o = (Oracle*)h;
    u128 totals[8];
    phase_totals(*o, totals);
    out[0] = o->n_valid;
    out[1] = o->n_rejected;
    out[2] = o->groups.size();
    for (int p = 0; p < 8; ++p) {
        out[3 + 2 * p] = (uint64_t)totals[p];
        out[4 + 2 * p] = (uint64_t)(totals[p] >> 64);
    }
}

// All entries, key ascending.  Returns 0, or -1 if cap is too small (*n_out = needed).
int oracle_finalize(void* h, const void* peaks, void* out, uint64_t cap, uint64_t* n_out) {
    Oracle* o = (Oracle*)h;
    const Peaks& pk = *(const Peaks*)peaks;
    *n_out = o->groups.size();
    if (cap < o->groups.size()) return -1;
    u128 totals[8];
    phase_totals(*o, totals);
    Entry* e = (Entry*)out;
    uint64_t i = 0;
    for (const auto& kv : o->groups) e[i++] = make_entry(*o, pk, totals, kv.first, kv.second);
    return 0;
}

// As oracle_finalize, but Eq. 3's per-phase denominators are given (totals[2p], totals[2p+1] = low
// and high 64 bits of T[p]) instead of summed over this handle's own keys: used when the handle
// holds only a slice of the key space and the totals come from oracle_direct_totals.
int oracle_finalize_given_totals(void* h, const void* peaks, const uint64_t totals_in[16], void* out, uint64_t cap,
                                 uint64_t* n_out) {
    Oracle* o = (Oracle*)h;
    const Peaks& pk = *(const Peaks*)peaks;
    *n_out = o->groups.size();
    if (cap < o->groups.size()) return -1;
    u128 totals[8];
    for (int p = 0; p < 8; ++p) totals[p] = ((u128)totals_in[2 * p + 1] << 64) | totals_in[2 * p];
    Entry* e = (Entry*)out;
    uint64_t i = 0;
    for (const auto& kv : o->groups) e[i++] = make_entry(*o, pk, totals, kv.first, kv.second);
    return 0;
}

// The first min(k, n_phase) entries of `phase` ordered by (wt descending, key ascending).
int oracle_topk(void* h, const void* peaks, uint32_t phase, uint32_t k, void* out, uint32_t* n_out) {
    Oracle* o = (Oracle*)h;
    const Peaks& pk = *(const Peaks*)peaks;
    u128 totals[8];
    phase_totals(*o, totals);
    std::vector<std::pair<uint64_t, Acc>> v;
    for (const auto& kv : o->groups)
        if ((kv.first >> 48) == phase) v.push_back(kv);
    std::sort(v.begin(), v.end(), [](const std::pair<uint64_t, Acc>& a, const std::pair<uint64_t, Acc>& b) {
        if (a.second.wt != b.second.wt) return a.second.wt > b.second.wt;
        return a.first < b.first;
    });
    uint32_t m = (uint32_t)std::min<uint64_t>(k, v.size());
    Entry* e = (Entry*)out;
    for (uint32_t i = 0; i < m; ++i) e[i] = make_entry(*o, pk, totals, v[i].first, v[i].second);
    *n_out = m;
    return 0;
}

// Score aggregation (Eq. 4-6), one candidate at a time.
//   Eq. 4  S_j = T_roofline,j / T_cand,j for every unit j = (operator, shape) that passed the
//          correctness gate; a value above 1 is an evaluation error: it is counted, not clipped.
//   Eq. 5  S_i = median of the S_j of operator i's correct shapes, 0 if it has none
//          (even count: mean of the two middle values).
//   Eq. 6  S_agg = sum_i w_i * S_i, accumulated in operator order.
// Readings where the paper is silent: a correct unit whose candidate time is not a finite
// positive number is an evaluation error too and is left out of the median; units are
// identified by position, `unit_op[j]` names unit j's operator (any order).
// out_s_op (n_ops doubles, may be null) receives S_i; returns S_agg; *n_errors counts the errors.
double oracle_score_candidate(const double* roofline_s, const uint32_t* unit_op, uint64_t n_units,
                              const double* t_cand, const uint8_t* correct, const double* w, uint32_t n_ops,
                              double* out_s_op, uint64_t* n_errors) {
    std::vector<std::vector<double>> per_op(n_ops);
    uint64_t errors = 0;
    for (uint64_t j = 0; j < n_units; ++j) {
        if (!correct[j] || unit_op[j] >= n_ops) continue;
        double t = t_cand[j];
        if (!(t > 0.0) || std::isinf(t)) {
            ++errors;
            continue;
        }
        double s = roofline_s[j] / t;                 // Eq. 4
        if (s > 1.0) ++errors;
        per_op[unit_op[j]].push_back(s);
    }
    double agg = 0.0;
    for (uint32_t i = 0; i < n_ops; ++i) {
        std::vector<double>& v = per_op[i];
        double s_i = 0.0;                             // Eq. 5: no correct shape -> 0
        if (!v.empty()) {
            std::sort(v.begin(), v.end());
            size_t m = v.size();
            s_i = (m & 1) ? v[m / 2] : (v[m / 2 - 1] + v[m / 2]) / 2.0;
        }
        if (out_s_op) out_s_op[i] = s_i;
        agg = agg + w[i] * s_i;                       // Eq. 6, operator order
    }
    if (n_errors) *n_errors = errors;
    return agg;
}

// Operator importance weights exactly as Eq. 2-3 state them (per-application denominators).
//   Eq. 2  D[i][a][phi] = sum of the durations of operator i's invocations in application a during
//          phase phi;  D_a[phi] = sum over ALL operators j of D[j][a][phi].
//   Eq. 3  wtilde_i = sum_a p_a * (1/|Phi_i|) * sum_{phi in Phi_i} D[i][a][phi] / D_a[phi],
//          w_i = wtilde_i / sum_{j retained} wtilde_j.
//   p_a = c_a / sum_a c_a (card-hour fractions); Phi_i = the phases in which operator i has any
//   observed time.  A record is valid iff app < n_apps, op < n_ops and phase < n_phases.
// Readings where the paper is silent: a phase in which application a has no time at all
// contributes nothing for that application (0/0 := skipped); an operator with no observed time,
// or not retained, gets weight 0; sums run in ascending phase, application and operator order and
// every operation is rounded once (this fixes the bit pattern).
// retained: n_ops flags or null (= all).  Returns the number of rejected records.
uint64_t oracle_eq3_weights(const void* records, uint64_t n, const uint32_t* app_weights, uint32_t n_apps,
                            uint32_t n_ops, uint32_t n_phases, const uint8_t* retained, double* out_w,
                            double* out_wtilde) {
    const Rec* recs = (const Rec*)records;
    std::vector<u128> D((size_t)n_phases * n_ops * n_apps, 0), Da((size_t)n_phases * n_apps, 0);
    uint64_t rejected = 0;
    for (uint64_t r = 0; r < n; ++r) {
        const Rec& x = recs[r];
        if (x.app_id >= n_apps || x.op_id >= n_ops || x.phase >= n_phases) {
            ++rejected;
            continue;
        }
        D[((size_t)x.phase * n_ops + x.op_id) * n_apps + x.app_id] += x.duration_ns;   // Eq. 2
        Da[(size_t)x.phase * n_apps + x.app_id] += x.duration_ns;
    }
    u128 c_total = 0;
    for (uint32_t a = 0; a < n_apps; ++a) c_total += app_weights[a];
    std::vector<double> wt(n_ops, 0.0);
    for (uint32_t i = 0; i < n_ops; ++i) {
        std::vector<uint32_t> phi;                                   // Phi_i
        for (uint32_t p = 0; p < n_phases; ++p) {
            bool any = false;
            for (uint32_t a = 0; a < n_apps && !any; ++a) any = D[((size_t)p * n_ops + i) * n_apps + a] != 0;
            if (any) phi.push_back(p);
        }
        double acc = 0.0;
        if (!phi.empty() && c_total != 0) {
            for (uint32_t a = 0; a < n_apps; ++a) {
                double inner = 0.0;
                for (uint32_t p : phi) {
                    u128 d_a = Da[(size_t)p * n_apps + a];
                    if (d_a == 0) continue;
                    inner = inner + (double)D[((size_t)p * n_ops + i) * n_apps + a] / (double)d_a;
                }
                double avg = inner / (double)phi.size();
                double p_a = (double)app_weights[a] / (double)c_total;
                acc = acc + p_a * avg;                              // Eq. 3, first part
            }
        }
        wt[i] = acc;
    }
    double total = 0.0;
    for (uint32_t i = 0; i < n_ops; ++i)
        if (!retained || retained[i]) total = total + wt[i];
    for (uint32_t i = 0; i < n_ops; ++i) {
        if (out_wtilde) out_wtilde[i] = wt[i];
        out_w[i] = ((!retained || retained[i]) && total > 0.0) ? wt[i] / total : 0.0;    // Eq. 3, normalisation
    }
    return rejected;
}

// The integer -> binary64 conversion used above, exposed so tests can pin its rounding.
double oracle_u128_to_f64(uint64_t hi, uint64_t lo) { return (double)(((u128)hi << 64) | lo); }

// Release artefacts made from a list of aggregated units (any order, one entry per key).
//
// oracle_sort_by_key: the same entries ordered by packed key ascending (entries with equal keys
// keep their input order).
void oracle_sort_by_key(const void* in, uint64_t n, void* out) {
    const Entry* e = (const Entry*)in;
    std::vector<Entry> v(e, e + n);
    std::stable_sort(v.begin(), v.end(), [](const Entry& a, const Entry& b) { return a.key < b.key; });
    if (n) std::memcpy(out, v.data(), n * sizeof(Entry));
}

// oracle_rank_phase: the construction behind Table 2 (operators ordered by weight with a
// running "Cum." share), for the units of one phase:
//   order   (wt descending, key ascending), wt the exact 128-bit integer;
//   T       sum of wt over the phase's units;
//   cum[i]  fl(fl(wt_0 + ... + wt_i) / fl(T)): the running sum is kept as an exact integer and
//           rounded once, so the column does not drift with the length of the list; +0.0
//           when T = 0;
//   n_keep  the coverage cut: the smallest k whose first k units hold at least
//           coverage_ppm / 10^6 of T, i.e. 10^6 * (wt_0 + ... + wt_{k-1}) >= coverage_ppm * T
//           in integers (k = 0 when coverage_ppm = 0 or T = 0; units of weight zero are never
//           needed, so k <= number of units with wt > 0).
// The first min(n_phase, out_cap) ranked entries go to out_ranked and their cum to out_cum.
// result = {n_phase, n_keep, T low, T high, covered low, covered high}, covered = the sum of the
// first n_keep units.  Requires T * 10^6 < 2^128 (T < 2^108).
void oracle_rank_phase(const void* in, uint64_t n, uint32_t phase, uint32_t coverage_ppm, void* out_ranked,
                       double* out_cum, uint64_t out_cap, uint64_t result[6]) {
    const Entry* e = (const Entry*)in;
    std::vector<Entry> v;
    u128 total = 0;
    for (uint64_t i = 0; i < n; ++i)
        if ((e[i].key >> 48) == phase) {
            v.push_back(e[i]);
            total += ((u128)e[i].wt_hi << 64) | e[i].wt_lo;
        }
    std::sort(v.begin(), v.end(), [](const Entry& a, const Entry& b) {
        u128 wa = ((u128)a.wt_hi << 64) | a.wt_lo, wb = ((u128)b.wt_hi << 64) | b.wt_lo;
        if (wa != wb) return wa > wb;
        return a.key < b.key;
    });
    const u128 need = (u128)coverage_ppm * total;
    u128 running = 0, covered = 0;
    uint64_t n_keep = 0;
    bool cut_found = (u128)1000000 * running >= need;  // k = 0 already covers a target of nothing
    Entry* out = (Entry*)out_ranked;
    for (uint64_t i = 0; i < v.size(); ++i) {
        running += ((u128)v[i].wt_hi << 64) | v[i].wt_lo;
        if (!cut_found && (u128)1000000 * running >= need) {
            cut_found = true;
            n_keep = i + 1;
            covered = running;
        }
        if (i < out_cap) {
            out[i] = v[i];
            out_cum[i] = total == 0 ? 0.0 : (double)running / (double)total;
        }
    }
    result[0] = v.size();
    result[1] = n_keep;
    result[2] = (uint64_t)total;
    result[3] = (uint64_t)(total >> 64);
    result[4] = (uint64_t)covered;
    result[5] = (uint64_t)(covered >> 64);
}

}  // extern "C"
