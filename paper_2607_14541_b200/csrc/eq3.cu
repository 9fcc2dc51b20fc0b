// Operator importance weights exactly as Eq. 2-3 state them.
//
//   Eq. 2  D[i][a][phi] = summed duration of operator i's invocations in application a, phase phi;
//          D_a[phi] = sum over all operators of D[.][a][phi]
//   Eq. 3  wtilde_i = sum_a p_a (1/|Phi_i|) sum_{phi in Phi_i} D[i][a][phi] / D_a[phi];
//          w_i = wtilde_i / sum over retained j of wtilde_j
//
// The group-by runs over (operator, application, phase) cells, a space of at most a few million
// cells that stays resident in L2.  With uniformly spread applications no subset of the cells is hot
// and equal cells hardly ever meet inside a warp, so there is nothing to pre-aggregate: ingest is one
// 64-bit reduction per record into L2, and what matters is that it does not return a value.  While
// fewer than 2^32 records have been ingested no cell can overflow 64 bits (durations are below 2^32),
// so the reduction is fire-and-forget; from then on every add returns the old value and wraps are
// counted in a second limb.  The floating-point part sums in ascending phase, application and
// operator order with every operation rounded once, which gives one bit pattern.
#include <cmath>
#include <new>

#include "kernels.h"

using namespace atrex;

struct atrex_eq3 {
    uint32_t n_apps = 0, n_ops = 0, n_phases = 0;
    int device = 0, n_sms = 0;
    uint32_t* d_appw = nullptr;   // [n_apps]
    ull* d_lo = nullptr;          // [n_phases][n_ops][n_apps] low 64 bits of D
    ull* d_hi = nullptr;          //                           wraps of the low limb
    ull* d_tot = nullptr;         // [n_phases][n_apps][2] D_a (lo, hi)
    double* d_wt = nullptr;       // [n_ops] wtilde
    double* d_w = nullptr;        // [n_ops] w
    uint8_t* d_ret = nullptr;     // [n_ops] retained flags
    ull* d_rejected = nullptr;
    size_t cells = 0;
    ull n_ingested = 0;           // records handed to ingest since create/reset (decides the carry handling)
};

namespace {

struct Guard {
    int prev = -1;
    explicit Guard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) cudaSetDevice(dev);
    }
    ~Guard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

__device__ __forceinline__ void red_add_u64(ull* p, ull v) {
    asm volatile("red.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// One record's duration into its cell.  CARRY: the low limb may wrap, so the add returns the old value.
template <bool CARRY>
__device__ __forceinline__ uint32_t eq3_add(uint32_t app, uint32_t w1, uint32_t dur, uint32_t n_apps, uint32_t n_ops,
                                            uint32_t n_phases, ull* lo, ull* hi) {
    const uint32_t op = w1 & 0xFFFFu, phase = (w1 >> 16) & 0xFFu;
    if (app >= n_apps || op >= n_ops || phase >= n_phases) return 1u;
    const size_t cell = ((size_t)phase * n_ops + op) * n_apps + app;
    if (CARRY) {
        const ull d = dur, old = atomicAdd(&lo[cell], d);
        if (old + d < old) atomicAdd(&hi[cell], 1ull);
    } else {
        red_add_u64(&lo[cell], (ull)dur);
    }
    return 0u;
}

// Two records per 32-byte load, two loads in flight per thread.
template <bool CARRY>
__global__ void __launch_bounds__(512) eq3_ingest_kernel(const unsigned char* __restrict__ body, ull n_pairs, const uint4* head,
                                                         const uint4* tail, uint32_t n_apps, uint32_t n_ops, uint32_t n_phases,
                                                         ull* lo, ull* hi, ull* rejected) {
    uint32_t bad = 0;
    const ull stride = (ull)gridDim.x * blockDim.x;
    for (ull i = (ull)blockIdx.x * blockDim.x + threadIdx.x; i < n_pairs; i += 2 * stride) {
        uint32_t a[8], b[8];
        const bool second = i + stride < n_pairs;
        asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]), "=r"(a[4]), "=r"(a[5]), "=r"(a[6]), "=r"(a[7])
                     : "l"(body + i * 32));
        if (second)
            asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3]), "=r"(b[4]), "=r"(b[5]), "=r"(b[6]), "=r"(b[7])
                         : "l"(body + (i + stride) * 32));
        bad += eq3_add<CARRY>(a[0], a[1], a[3], n_apps, n_ops, n_phases, lo, hi);
        bad += eq3_add<CARRY>(a[4], a[5], a[7], n_apps, n_ops, n_phases, lo, hi);
        if (second) {
            bad += eq3_add<CARRY>(b[0], b[1], b[3], n_apps, n_ops, n_phases, lo, hi);
            bad += eq3_add<CARRY>(b[4], b[5], b[7], n_apps, n_ops, n_phases, lo, hi);
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < 2) {   // records outside the 32-byte aligned body
        const uint4* one = threadIdx.x == 0 ? head : tail;
        if (one) {
            const uint4 r = *one;
            bad += eq3_add<CARRY>(r.x, r.y, r.w, n_apps, n_ops, n_phases, lo, hi);
        }
    }
    bad = __reduce_add_sync(0xFFFFFFFFu, bad);
    if ((threadIdx.x & 31u) == 0 && bad) atomicAdd(rejected, (ull)bad);
}

// D_a[phi]: one thread per (phase, application), summing over operators
__global__ void eq3_app_totals_kernel(const ull* lo, const ull* hi, uint32_t n_apps, uint32_t n_ops, uint32_t n_phases, ull* tot) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)n_phases * n_apps) return;
    const uint32_t phase = (uint32_t)(idx / n_apps), app = (uint32_t)(idx % n_apps);
    ull s_lo = 0, s_hi = 0;
    for (uint32_t i = 0; i < n_ops; ++i) {
        const size_t cell = ((size_t)phase * n_ops + i) * n_apps + app;
        const ull x = lo[cell];
        const ull nl = s_lo + x;
        s_hi += hi[cell] + (nl < s_lo ? 1ull : 0ull);
        s_lo = nl;
    }
    tot[2 * idx] = s_lo;
    tot[2 * idx + 1] = s_hi;
}

// wtilde_i: one CTA per operator.  The CTA finds Phi_i, then every thread works out the terms
// p_a * (1/|Phi_i|) * sum_phi D[i][a][phi] / D_a[phi] of its applications (each a fixed sequence of
// rounded operations, independent of the others) into shared memory in chunks; only the running sum
// over the applications, whose order is part of the result, is left to one thread.
constexpr int WT_THREADS = 256;
constexpr uint32_t WT_CHUNK = 2048;   // terms held in shared memory at a time

__global__ void __launch_bounds__(WT_THREADS) eq3_wtilde_kernel(const ull* lo, const ull* hi, const ull* tot, const uint32_t* appw,
                                                                uint32_t n_apps, uint32_t n_ops, uint32_t n_phases, double* wt) {
    __shared__ double s_term[WT_CHUNK];
    __shared__ uint32_t s_present;
    __shared__ ull s_weights;
    const uint32_t i = blockIdx.x;
    if (threadIdx.x == 0) {
        s_present = 0;
        s_weights = 0;
    }
    __syncthreads();
    uint32_t present = 0;  // bit phi: operator i has time in phase phi
    ull c_part = 0;
    for (uint32_t a = threadIdx.x; a < n_apps; a += WT_THREADS) {
        c_part += appw[a];  // < 2^64 in total: fewer than 2^32 weights below 2^32
        for (uint32_t p = 0; p < n_phases; ++p) {
            const size_t cell = ((size_t)p * n_ops + i) * n_apps + a;
            if ((lo[cell] | hi[cell]) != 0) present |= 1u << p;
        }
    }
    if (present) atomicOr(&s_present, present);
    atomicAdd(&s_weights, c_part);
    __syncthreads();
    present = s_present;
    const ull c_lo = s_weights;
    const int n_phi = __popc(present);
    if (n_phi == 0 || c_lo == 0) {
        if (threadIdx.x == 0) wt[i] = 0.0;
        return;
    }
    const double c_total = __ull2double_rn(c_lo), d_phi = (double)n_phi;
    double acc = 0.0;   // thread 0's
    for (uint32_t a0 = 0; a0 < n_apps; a0 += WT_CHUNK) {
        for (uint32_t a = a0 + threadIdx.x; a < min(a0 + WT_CHUNK, n_apps); a += WT_THREADS) {
            double inner = 0.0;
            for (uint32_t p = 0; p < n_phases; ++p) {
                if (!(present & (1u << p))) continue;
                const size_t ta = (size_t)p * n_apps + a;
                const ull t_lo = tot[2 * ta], t_hi = tot[2 * ta + 1];
                if ((t_lo | t_hi) == 0) continue;
                const size_t cell = ((size_t)p * n_ops + i) * n_apps + a;
                inner = __dadd_rn(inner, __ddiv_rn(u128_to_f64_rn(hi[cell], lo[cell]), u128_to_f64_rn(t_hi, t_lo)));
            }
            const double avg = __ddiv_rn(inner, d_phi);
            const double p_a = __ddiv_rn(__ull2double_rn((ull)appw[a]), c_total);
            s_term[a - a0] = __dmul_rn(p_a, avg);
        }
        __syncthreads();
        if (threadIdx.x == 0)
            for (uint32_t a = a0; a < min(a0 + WT_CHUNK, n_apps); ++a) acc = __dadd_rn(acc, s_term[a - a0]);
        __syncthreads();
    }
    if (threadIdx.x == 0) wt[i] = acc;
}

__global__ void eq3_normalise_kernel(const double* wt, const uint8_t* retained, uint32_t n_ops, double* w) {
    __shared__ double s_total;
    if (threadIdx.x == 0) {
        double total = 0.0;
        for (uint32_t i = 0; i < n_ops; ++i)
            if (retained[i]) total = __dadd_rn(total, wt[i]);
        s_total = total;
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < n_ops; i += blockDim.x)
        w[i] = (retained[i] && s_total > 0.0) ? __ddiv_rn(wt[i], s_total) : 0.0;
}

}  // namespace

extern "C" {

int atrex_eq3_create(uint32_t n_apps, uint32_t n_ops, uint32_t n_phases, const uint32_t* app_weights, int32_t device,
                     atrex_eq3_t** out) {
    if (!out) return ATREX_ERR_INVALID;
    *out = nullptr;
    if (!app_weights || n_apps == 0 || n_ops == 0 || n_ops > 65536 || n_phases == 0 || n_phases > ATREX_MAX_PHASES)
        return ATREX_ERR_INVALID;
    const size_t cells = (size_t)n_apps * n_ops * n_phases;
    if (cells > ((size_t)1 << 28)) return ATREX_ERR_TOO_LARGE;
    atrex_eq3* h = new (std::nothrow) atrex_eq3;
    if (!h) return ATREX_ERR_NOMEM;
    h->n_apps = n_apps; h->n_ops = n_ops; h->n_phases = n_phases; h->device = device; h->cells = cells;
    Guard g(device);
    cudaError_t e = cudaDeviceGetAttribute(&h->n_sms, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_appw, (size_t)n_apps * 4);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_lo, cells * 8);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_hi, cells * 8);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_tot, (size_t)n_phases * n_apps * 16);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_wt, (size_t)n_ops * 8);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_w, (size_t)n_ops * 8);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_ret, n_ops);
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->d_rejected, 8);
    if (e == cudaSuccess) e = cudaMemcpy(h->d_appw, app_weights, (size_t)n_apps * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(h->d_lo, 0, cells * 8);
    if (e == cudaSuccess) e = cudaMemset(h->d_hi, 0, cells * 8);
    if (e == cudaSuccess) e = cudaMemset(h->d_rejected, 0, 8);
    if (e != cudaSuccess) {
        cudaGetLastError();
        atrex_eq3_destroy(h);
        return e == cudaErrorMemoryAllocation ? ATREX_ERR_NOMEM : ATREX_ERR_CUDA;
    }
    *out = h;
    return ATREX_OK;
}

void atrex_eq3_destroy(atrex_eq3_t* h) {
    if (!h) return;
    Guard g(h->device);
    cudaDeviceSynchronize();
    cudaFree(h->d_appw); cudaFree(h->d_lo); cudaFree(h->d_hi); cudaFree(h->d_tot);
    cudaFree(h->d_wt); cudaFree(h->d_w); cudaFree(h->d_ret); cudaFree(h->d_rejected);
    delete h;
}

int atrex_eq3_reset(atrex_eq3_t* h, void* stream) {
    if (!h) return ATREX_ERR_INVALID;
    Guard g(h->device);
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(h->d_lo, 0, h->cells * 8, s) != cudaSuccess || cudaMemsetAsync(h->d_hi, 0, h->cells * 8, s) != cudaSuccess ||
        cudaMemsetAsync(h->d_rejected, 0, 8, s) != cudaSuccess)
        return ATREX_ERR_CUDA;
    h->n_ingested = 0;
    return ATREX_OK;
}

int atrex_eq3_ingest(atrex_eq3_t* h, const atrex_record_t* d_records, uint64_t n, void* stream) {
    if (!h) return ATREX_ERR_INVALID;
    if (n == 0) return ATREX_OK;
    if (!d_records || ((uintptr_t)d_records & 15u)) return ATREX_ERR_INVALID;
    Guard g(h->device);
    // the 32-byte aligned body as record pairs; at most one record before and one after it
    const unsigned char* base = (const unsigned char*)d_records;
    const uint64_t head = ((uintptr_t)base & 31u) ? 1 : 0;
    const uint64_t n_body = n - head, n_pairs = n_body / 2;
    const uint4* head_rec = head ? (const uint4*)base : nullptr;
    const uint4* tail_rec = (n_body & 1) ? (const uint4*)(base + (n - 1) * 16) : nullptr;
    ull blocks = (n_pairs + 1023) / 1024;
    if (blocks > (ull)h->n_sms * 4) blocks = (ull)h->n_sms * 4;
    if (blocks == 0) blocks = 1;
    // below 2^32 records in total no cell's 64-bit sum can wrap: fire-and-forget reductions
    const bool carry = h->n_ingested + n >= (1ull << 32);
    h->n_ingested += n;
    if (carry)
        eq3_ingest_kernel<true><<<(unsigned)blocks, 512, 0, (cudaStream_t)stream>>>(base + head * 16, n_pairs, head_rec, tail_rec, h->n_apps,
                                                                                    h->n_ops, h->n_phases, h->d_lo, h->d_hi, h->d_rejected);
    else
        eq3_ingest_kernel<false><<<(unsigned)blocks, 512, 0, (cudaStream_t)stream>>>(base + head * 16, n_pairs, head_rec, tail_rec, h->n_apps,
                                                                                     h->n_ops, h->n_phases, h->d_lo, h->d_hi, h->d_rejected);
    return cudaGetLastError() == cudaSuccess ? ATREX_OK : ATREX_ERR_CUDA;
}

int atrex_eq3_finalize(atrex_eq3_t* h, const uint8_t* h_retained, double* h_w, double* h_wtilde, uint64_t* h_rejected,
                       void* stream) {
    if (!h || !h_w) return ATREX_ERR_INVALID;
    Guard g(h->device);
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* all = nullptr;
    if (!h_retained) {
        all = (uint8_t*)malloc(h->n_ops);
        if (!all) return ATREX_ERR_NOMEM;
        memset(all, 1, h->n_ops);
    }
    cudaError_t e = cudaMemcpyAsync(h->d_ret, h_retained ? h_retained : all, h->n_ops, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && all) e = cudaStreamSynchronize(s);  // `all` is freed below
    free(all);
    if (e != cudaSuccess) return ATREX_ERR_CUDA;
    const size_t pa = (size_t)h->n_phases * h->n_apps;
    eq3_app_totals_kernel<<<(unsigned)((pa + 255) / 256), 256, 0, s>>>(h->d_lo, h->d_hi, h->n_apps, h->n_ops, h->n_phases, h->d_tot);
    eq3_wtilde_kernel<<<h->n_ops, WT_THREADS, 0, s>>>(h->d_lo, h->d_hi, h->d_tot, h->d_appw, h->n_apps, h->n_ops, h->n_phases, h->d_wt);
    eq3_normalise_kernel<<<1, 256, 0, s>>>(h->d_wt, h->d_ret, h->n_ops, h->d_w);
    if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
    e = cudaMemcpyAsync(h_w, h->d_w, (size_t)h->n_ops * 8, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && h_wtilde) e = cudaMemcpyAsync(h_wtilde, h->d_wt, (size_t)h->n_ops * 8, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && h_rejected) e = cudaMemcpyAsync(h_rejected, h->d_rejected, 8, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    return e == cudaSuccess ? ATREX_OK : ATREX_ERR_CUDA;
}

}  // extern "C"
