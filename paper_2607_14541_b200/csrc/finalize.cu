// Finalize: per-phase totals (Eq. 2's D^phi), per-key weights (Eq. 3 normalised per phase),
// roofline times (Eq. 1), compaction, and the ranked top-k (Table 2).
//
// All floating-point results come from explicit round-to-nearest intrinsics on exact
// integers, so they have one correct bit pattern: fl(fl(wt) / fl(T)) and
// fmax(fl(F) / P, fl(M) / beta).
#include "atrex_dev.cuh"
#include "kernels.h"

namespace atrex {

constexpr int FIN_THREADS = 256;
constexpr int TOT_THREADS = 128;

struct SlotView {
    ull key, count, lo, hi;
    bool live;
};

__device__ __forceinline__ SlotView load_slot(const TableRef& t, ull i) {
    SlotView v;
    ull sk = t.keys[i];
    v.live = sk != 0;
    v.key = ~sk;
    v.lo = v.count = v.hi = 0;
    if (v.live) {
        ulonglong2 x = t.vals[i];
        v.lo = x.x;
        v.count = x.y & COUNT_MASK;
        v.hi = x.y >> HI_SHIFT;
    }
    return v;
}

// ---- per-phase totals -------------------------------------------------------------------
// Each thread keeps private per-phase 128-bit sums in its own shared-memory column; columns
// are added per CTA and folded into the control block with a carry-aware pair of atomics.
__global__ void __launch_bounds__(TOT_THREADS) totals_kernel(TableRef tab, ull n_slots) {
    Control* ctl = tab.ctl;
    __shared__ ull s_lo[ATREX_MAX_PHASES][TOT_THREADS];
    __shared__ ull s_hi[ATREX_MAX_PHASES][TOT_THREADS];
    __shared__ ull s_cnt[ATREX_MAX_PHASES][TOT_THREADS];
    __shared__ uint32_t s_nk[ATREX_MAX_PHASES][TOT_THREADS];
    const int t = threadIdx.x;
#pragma unroll
    for (int p = 0; p < ATREX_MAX_PHASES; ++p) {
        s_lo[p][t] = 0; s_hi[p][t] = 0; s_cnt[p][t] = 0; s_nk[p][t] = 0;
    }
    // four slots per thread in flight: all key loads first, then the values of the live ones
    constexpr int ILP = 4;
    const ull stride = (ull)gridDim.x * blockDim.x;
    for (ull i0 = (ull)blockIdx.x * blockDim.x + t; i0 < n_slots; i0 += stride * ILP) {
        ull sk[ILP];
        ulonglong2 x[ILP];
#pragma unroll
        for (int u = 0; u < ILP; ++u) sk[u] = i0 + u * stride < n_slots ? tab.keys[i0 + u * stride] : 0ull;
#pragma unroll
        for (int u = 0; u < ILP; ++u) x[u] = i0 + u * stride < n_slots ? tab.vals[i0 + u * stride] : make_ulonglong2(0, 0);  // unconditional: no wait for the keys
#pragma unroll
        for (int u = 0; u < ILP; ++u) {
            if (sk[u] == 0) continue;
            const int p = (int)(~sk[u] >> 48) & (ATREX_MAX_PHASES - 1);
            const ull o = s_lo[p][t], n = o + x[u].x;
            s_lo[p][t] = n;
            s_hi[p][t] += (x[u].y >> HI_SHIFT) + (n < o ? 1ull : 0ull);
            s_cnt[p][t] += x[u].y & COUNT_MASK;
            s_nk[p][t] += 1;
        }
    }
    __syncthreads();
    if (t < ATREX_MAX_PHASES) {
        ull lo = 0, hi = 0, cnt = 0, nk = 0;
        for (int j = 0; j < TOT_THREADS; ++j) {
            ull n = lo + s_lo[t][j];
            hi += s_hi[t][j] + (n < lo ? 1ull : 0ull);
            lo = n;
            cnt += s_cnt[t][j];
            nk += s_nk[t][j];
        }
        if (nk != 0) {
            ull old = atomicAdd(&ctl->total_lo[t], lo);
            atomicAdd(&ctl->total_hi[t], hi + (old + lo < old ? 1ull : 0ull));
            atomicAdd(&ctl->count_per_phase[t], cnt);
            atomicAdd(&ctl->keys_per_phase[t], nk);
        }
    }
}

// ---- per-key results ----------------------------------------------------------------------
// The work table is probed by double hashing (strides coprime to the partition's slot count): with
// linear probing the longest of a warp's 32 probe sequences -- which is what the warp waits for --
// was several times the average.
__device__ __forceinline__ uint32_t work_stride(const WorkRef& w, uint32_t h) {
    return (uint32_t)(w.strides >> (8 * stride_index(h))) & 0xFFu;
}
__device__ __forceinline__ double roofline_time(const WorkRef& w, const atrex_hw_peaks_t& pk, ull key) {
    const double qnan = __longlong_as_double(0x7FF8000000000000ll);
    if (w.table == nullptr) return qnan;
    ull pair = key & 0x0000FFFFFFFFFFFFull;
    ull skey = ~pair;
    const uint32_t h = hash32(pair);
    const WorkSlot* part = w.table + (ull)part_of(h, w.lp) * w.Cw;
    uint32_t s = local_of(h, 0u, w.Cw);
    const uint32_t advance = work_stride(w, h);
    for (uint32_t probe = 0; probe < w.Cw; ++probe) {
        const WorkSlot* e = part + s;
        ull k = e->skey;
        if (k == skey) {
            double t_compute = __ddiv_rn(__ull2double_rn(e->flops), pk.peak_flops[e->dtype & (ATREX_MAX_DTYPES - 1)]);
            double t_memory = __ddiv_rn(__ull2double_rn(e->bytes), pk.peak_bw);
            return fmax(t_compute, t_memory);
        }
        if (k == 0) break;
        s += advance;
        if (s >= w.Cw) s -= w.Cw;
    }
    return qnan;
}

__device__ __forceinline__ atrex_entry_t make_entry(const SlotView& v, const double* dT, const bool* zeroT,
                                                    const FinalizeParams& p) {
    atrex_entry_t e;
    e.key = v.key;
    e.count = v.count;
    e.wt_lo = v.lo;
    e.wt_hi = v.hi;
    int ph = (int)(v.key >> 48) & (ATREX_MAX_PHASES - 1);
    e.phase_weight = zeroT[ph] ? 0.0 : __ddiv_rn(u128_to_f64_rn(v.hi, v.lo), dT[ph]);
    e.roofline_s = roofline_time(p.work, p.peaks, v.key);
    return e;
}

__device__ __forceinline__ void store_entry(atrex_entry_t* dst, const atrex_entry_t& e) {
    ulonglong2* q = reinterpret_cast<ulonglong2*>(dst);
    q[0] = make_ulonglong2(e.key, e.count);
    q[1] = make_ulonglong2(e.wt_lo, e.wt_hi);
    q[2] = make_ulonglong2((ull)__double_as_longlong(e.phase_weight), (ull)__double_as_longlong(e.roofline_s));
}

__device__ __forceinline__ void load_phase_totals(const Control* ctl, double* dT, bool* zeroT) {
    if (threadIdx.x < ATREX_MAX_PHASES) {
        ull lo = ctl->total_lo[threadIdx.x], hi = ctl->total_hi[threadIdx.x];
        dT[threadIdx.x] = u128_to_f64_rn(hi, lo);
        zeroT[threadIdx.x] = (lo | hi) == 0;
    }
    __syncthreads();
}

// Each warp looks at 128 slots per round (four coalesced rows), queues the live ones in shared
// memory and then works through the queue with all lanes busy: at a table load of a third, the
// divisions and the work-table probe run on full warps instead of one lane in three.
constexpr int EMIT_ILP = 4;
constexpr int EMIT_WARPS = FIN_THREADS / 32;

__global__ void __launch_bounds__(FIN_THREADS) emit_kernel(FinalizeParams p) {
    __shared__ double dT[ATREX_MAX_PHASES];
    __shared__ bool zeroT[ATREX_MAX_PHASES];
    __shared__ ull q_key[EMIT_WARPS][32 * EMIT_ILP];
    __shared__ ulonglong2 q_val[EMIT_WARPS][32 * EMIT_ILP];
    load_phase_totals(p.ctl, dT, zeroT);
    const unsigned lane = threadIdx.x & 31u, w = threadIdx.x >> 5;
    const ull stride = (ull)gridDim.x * blockDim.x;
    const ull rounds = (p.n_slots + stride * EMIT_ILP - 1) / (stride * EMIT_ILP);  // uniform: warps stay converged
    for (ull r = 0; r < rounds; ++r) {
        ull sk[EMIT_ILP];
        ulonglong2 xv[EMIT_ILP];
#pragma unroll
        for (int u = 0; u < EMIT_ILP; ++u) {
            const ull i = (r * EMIT_ILP + u) * stride + (ull)blockIdx.x * blockDim.x + threadIdx.x;
            sk[u] = i < p.n_slots ? p.t.keys[i] : 0ull;
            xv[u] = i < p.n_slots ? p.t.vals[i] : make_ulonglong2(0, 0);  // with the key, not after it
        }
        uint32_t total = 0;
#pragma unroll
        for (int u = 0; u < EMIT_ILP; ++u) {
            const unsigned live = __ballot_sync(0xFFFFFFFFu, sk[u] != 0);
            if (sk[u] != 0) {
                const uint32_t at = total + __popc(live & ((1u << lane) - 1u));
                q_key[w][at] = ~sk[u];
                q_val[w][at] = xv[u];
            }
            total += __popc(live);
        }
        if (total == 0) continue;
        ull base = 0;
        if (lane == 0) base = atomicAdd(&p.ctl->n_out, (ull)total);
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        __syncwarp();
        for (uint32_t j = lane; j < total; j += 32) {
            SlotView v;
            const ulonglong2 x = q_val[w][j];
            v.key = q_key[w][j];
            v.live = true;
            v.lo = x.x;
            v.count = x.y & COUNT_MASK;
            v.hi = x.y >> HI_SHIFT;
            const ull pos = base + j;
            if (pos < p.out_cap) store_entry(p.out + pos, make_entry(v, dT, zeroT, p));
        }
        __syncwarp();  // the queue is refilled in the next round
    }
}

// ---- work table ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) work_insert_kernel(const atrex_work_t* rows, ull n, WorkRef w, Control* ctl) {
    for (ull i = (ull)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (ull)gridDim.x * blockDim.x) {
        atrex_work_t r = rows[i];
        if (r.dtype >= ATREX_MAX_DTYPES) {
            atomicOr(&ctl->work_status, ST_WORK_DTYPE);
            continue;
        }
        ull pair = ((ull)r.op_id << 32) | (ull)r.shape_id;
        ull skey = ~pair;
        const uint32_t h = hash32(pair);
        WorkSlot* part = w.table + (ull)part_of(h, w.lp) * w.Cw;
        uint32_t s = local_of(h, 0u, w.Cw);
        const uint32_t advance = work_stride(w, h);
        bool done = false;
        for (uint32_t probe = 0; probe < w.Cw && !done; ++probe) {
            WorkSlot* e = part + s;
            ull old = atomicCAS(&e->skey, 0ull, skey);
            if (old == 0) {
                e->flops = r.flops;
                e->bytes = r.bytes;
                e->dtype = r.dtype;
                done = true;
            } else if (old == skey) {
                atomicOr(&ctl->work_status, ST_WORK_DUP);
                done = true;
            } else {
                s += advance;
                if (s >= w.Cw) s -= w.Cw;
            }
        }
        if (!done) atomicOr(&ctl->work_status, ST_WORK_FULL);
    }
}

// ---- top-k --------------------------------------------------------------------------------
// Ranking composite, larger = better: bits 56..143 hold the 88-bit weighted time, bits 0..55
// the complemented key (so the smaller key wins a tie).  Unique per key.  A most-significant-
// digit radix select (12-bit digits) narrows the table down to the definite winners plus a
// bounded set of candidates, which one CTA then sorts.
struct Composite {
    ull c[3];  // c[2] = bits 128..143
};

__device__ __forceinline__ Composite composite_of(const SlotView& v) {
    Composite x;
    x.c[0] = ((~v.key) & 0x00FFFFFFFFFFFFFFull) | (v.lo << 56);
    x.c[1] = (v.lo >> 8) | (v.hi << 56);
    x.c[2] = v.hi >> 8;
    return x;
}

// Digit d (most significant first) of the composite shifted left by `shift` bits.  The shift
// drops the leading zero bits that every key of the phase shares (no weighted time exceeds the
// phase total), so that the first digit already separates the top of the ranking.
__device__ __forceinline__ uint32_t digit_of(const Composite& x, int d, int shift) {
    int off = 144 - 12 * (d + 1) - shift;
    if (off < 0) return (uint32_t)(x.c[0] << (-off)) & 0xFFFu;  // last, partial digit
    int wi = off >> 6, sh = off & 63;
    ull v = x.c[wi] >> sh;
    if (sh > 52 && wi < 2) v |= x.c[wi + 1] << (64 - sh);
    return (uint32_t)v & 0xFFFu;
}

// -1: below the prefix, 0: equal on all fixed digits, +1: above
__device__ __forceinline__ int compare_prefix(const Composite& x, const TopkParams& p) {
    for (uint32_t d = 0; d < p.n_prefix_digits; ++d) {
        uint32_t a = digit_of(x, (int)d, (int)p.shift), b = p.prefix_digit[d];
        if (a != b) return a > b ? 1 : -1;
    }
    return 0;
}

__global__ void __launch_bounds__(FIN_THREADS) topk_hist_kernel(TopkParams p) {
    __shared__ uint32_t h[TOPK_BINS];
    for (int i = threadIdx.x; i < TOPK_BINS; i += blockDim.x) h[i] = 0;
    __syncthreads();
    for (ull i = (ull)blockIdx.x * blockDim.x + threadIdx.x; i < p.n_slots; i += (ull)gridDim.x * blockDim.x) {
        SlotView v = load_slot(p.t, i);
        if (!v.live || (uint32_t)(v.key >> 48) != p.phase) continue;
        Composite x = composite_of(v);
        if (compare_prefix(x, p) != 0) continue;
        atomicAdd(&h[digit_of(x, (int)p.n_prefix_digits, (int)p.shift)], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < TOPK_BINS; i += blockDim.x)
        if (h[i] != 0) atomicAdd(&p.ctl->hist[i], h[i]);
}

// -1: below the prefix, 0: equal on all fixed digits, +1: above (one phase of a multi-phase pass)
__device__ __forceinline__ int compare_prefix_of(const Composite& x, const TopkAllParams& p, uint32_t q) {
    for (uint32_t d = 0; d < p.n_prefix_digits[q]; ++d) {
        uint32_t a = digit_of(x, (int)d, (int)p.shift[q]), b = p.prefix_digit[q][d];
        if (a != b) return a > b ? 1 : -1;
    }
    return 0;
}

// Next-digit histograms of all active phases in one pass (shared memory: one row per phase).
__global__ void __launch_bounds__(1024) topk_hist_all_kernel(const __grid_constant__ TopkAllParams p) {
    extern __shared__ uint32_t h_all[];  // [ATREX_MAX_PHASES][TOPK_BINS], rows of inactive phases unused
    for (uint32_t i = threadIdx.x; i < ATREX_MAX_PHASES * TOPK_BINS; i += blockDim.x)
        if ((p.active_mask >> (i / TOPK_BINS)) & 1u) h_all[i] = 0;
    __syncthreads();
    constexpr int ILP = 4;
    const ull stride = (ull)gridDim.x * blockDim.x;
    for (ull i0 = (ull)blockIdx.x * blockDim.x + threadIdx.x; i0 < p.n_slots; i0 += stride * ILP) {
        ull sk[ILP];
        ulonglong2 x[ILP];
#pragma unroll
        for (int u = 0; u < ILP; ++u) sk[u] = i0 + u * stride < p.n_slots ? p.t.keys[i0 + u * stride] : 0ull;
#pragma unroll
        for (int u = 0; u < ILP; ++u) {
            x[u] = i0 + u * stride < p.n_slots ? p.t.vals[i0 + u * stride] : make_ulonglong2(0, 0);  // no wait for the keys
        }
#pragma unroll
        for (int u = 0; u < ILP; ++u) {
            const uint32_t q = (uint32_t)(~sk[u] >> 48) & (ATREX_MAX_PHASES - 1);
            if (!(sk[u] != 0 && ((p.active_mask >> q) & 1u))) sk[u] = 0;
        }
#pragma unroll
        for (int u = 0; u < ILP; ++u) {
            if (sk[u] == 0) continue;
            SlotView v;
            v.key = ~sk[u];
            v.lo = x[u].x;
            v.hi = x[u].y >> HI_SHIFT;
            const uint32_t q = (uint32_t)(v.key >> 48) & (ATREX_MAX_PHASES - 1);
            const Composite c = composite_of(v);
            if (compare_prefix_of(c, p, q) != 0) continue;
            atomicAdd(&h_all[q * TOPK_BINS + digit_of(c, (int)p.n_prefix_digits[q], (int)p.shift[q])], 1u);
        }
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < ATREX_MAX_PHASES * TOPK_BINS; i += blockDim.x)
        if (((p.active_mask >> (i / TOPK_BINS)) & 1u) && h_all[i] != 0) atomicAdd(&p.hist[i], h_all[i]);
}

// Candidates of all active phases in one pass, each phase into its own selection region.
__global__ void __launch_bounds__(FIN_THREADS) topk_collect_all_kernel(const __grid_constant__ TopkAllParams p) {
    constexpr int ILP = 4;
    const ull stride = (ull)gridDim.x * blockDim.x;
    for (ull i0 = (ull)blockIdx.x * blockDim.x + threadIdx.x; i0 < p.n_slots; i0 += stride * ILP) {
        ull sk[ILP];
        ulonglong2 x[ILP];
#pragma unroll
        for (int u = 0; u < ILP; ++u) sk[u] = i0 + u * stride < p.n_slots ? p.t.keys[i0 + u * stride] : 0ull;
#pragma unroll
        for (int u = 0; u < ILP; ++u) {
            x[u] = i0 + u * stride < p.n_slots ? p.t.vals[i0 + u * stride] : make_ulonglong2(0, 0);  // no wait for the keys
        }
#pragma unroll
        for (int u = 0; u < ILP; ++u) {
            const uint32_t q = (uint32_t)(~sk[u] >> 48) & (ATREX_MAX_PHASES - 1);
            if (!(sk[u] != 0 && ((p.active_mask >> q) & 1u))) sk[u] = 0;
        }
#pragma unroll
        for (int u = 0; u < ILP; ++u) {
            if (sk[u] == 0) continue;
            SlotView v;
            v.key = ~sk[u];
            v.lo = x[u].x;
            v.hi = x[u].y >> HI_SHIFT;
            const uint32_t q = (uint32_t)(v.key >> 48) & (ATREX_MAX_PHASES - 1);
            const Composite c = composite_of(v);
            if (!((p.collect_all_mask >> q) & 1u) && compare_prefix_of(c, p, q) < 0) continue;
            const ull pos = atomicAdd(&p.sel_count[q], 1ull);
            if (pos < p.sel_cap) {
                ull* dst = p.sel + ((ull)q * p.sel_cap + pos) * 4;
                dst[0] = c.c[2]; dst[1] = c.c[1]; dst[2] = c.c[0]; dst[3] = i0 + u * stride;
            }
        }
    }
}

__device__ __forceinline__ bool sel_less(const ull* a, const ull* b) {
    if (a[0] != b[0]) return a[0] < b[0];
    if (a[1] != b[1]) return a[1] < b[1];
    return a[2] < b[2];
}

// Bitonic sort, descending by composite, of n (power of two) 32-byte items in global memory,
// by a single CTA.  Padding items are all-zero and sink to the end.
__global__ void __launch_bounds__(1024) topk_sort_kernel(ull* sel, uint32_t n) {
    for (uint32_t k = 2; k <= n; k <<= 1) {
        for (uint32_t j = k >> 1; j > 0; j >>= 1) {
            for (uint32_t i = threadIdx.x; i < n; i += blockDim.x) {
                uint32_t l = i ^ j;
                if (l > i) {
                    ull* a = sel + (ull)i * 4;
                    ull* b = sel + (ull)l * 4;
                    bool descending = (i & k) == 0;
                    bool swap = descending ? sel_less(a, b) : sel_less(b, a);
                    if (swap) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            ull t = a[q]; a[q] = b[q]; b[q] = t;
                        }
                    }
                }
            }
            __syncthreads();
        }
    }
}

__global__ void __launch_bounds__(FIN_THREADS) topk_emit_kernel(FinalizeParams p, const ull* sel, uint32_t n) {
    __shared__ double dT[ATREX_MAX_PHASES];
    __shared__ bool zeroT[ATREX_MAX_PHASES];
    load_phase_totals(p.ctl, dT, zeroT);
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        SlotView v = load_slot(p.t, sel[(ull)i * 4 + 3]);
        store_entry(p.out + i, make_entry(v, dT, zeroT, p));
    }
}

// ---- launchers ----------------------------------------------------------------------------
cudaError_t finalize_prepare() {
    return cudaFuncSetAttribute(topk_hist_all_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)(ATREX_MAX_PHASES * TOPK_BINS * sizeof(uint32_t)));
}

cudaError_t launch_totals(const TableRef& t, ull n_slots, int grid, cudaStream_t stream) {
    totals_kernel<<<grid, TOT_THREADS, 0, stream>>>(t, n_slots);
    return cudaGetLastError();
}

cudaError_t launch_emit(const FinalizeParams& p, int grid, cudaStream_t stream) {
    emit_kernel<<<grid, FIN_THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_work_insert(const atrex_work_t* rows, ull n, const WorkRef& w, Control* ctl, int grid,
                               cudaStream_t stream) {
    work_insert_kernel<<<grid, 256, 0, stream>>>(rows, n, w, ctl);
    return cudaGetLastError();
}

cudaError_t launch_topk_hist_all(const TopkAllParams& p, int n_sms, cudaStream_t stream) {
    const size_t smem = (size_t)ATREX_MAX_PHASES * TOPK_BINS * sizeof(uint32_t);
    topk_hist_all_kernel<<<n_sms, 1024, smem, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_topk_collect_all(const TopkAllParams& p, int grid, cudaStream_t stream) {
    topk_collect_all_kernel<<<grid, FIN_THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_topk_hist(const TopkParams& p, int grid, cudaStream_t stream) {
    topk_hist_kernel<<<grid, FIN_THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_topk_sort(ull* sel, uint32_t n_pow2, cudaStream_t stream) {
    topk_sort_kernel<<<1, 1024, 0, stream>>>(sel, n_pow2);
    return cudaGetLastError();
}

cudaError_t launch_topk_emit(const FinalizeParams& p, const ull* sel, uint32_t n, cudaStream_t stream) {
    int grid = (int)((n + FIN_THREADS - 1) / FIN_THREADS);
    if (grid < 1) grid = 1;
    topk_emit_kernel<<<grid, FIN_THREADS, 0, stream>>>(p, sel, n);
    return cudaGetLastError();
}

}  // namespace atrex
