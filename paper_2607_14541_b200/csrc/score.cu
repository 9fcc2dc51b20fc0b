// Roofline score aggregation (Eq. 4-6), batched over candidates: one CTA per candidate.
//
//   Eq. 4  S_j = T_roofline,j / T_cand,j for units that passed correctness (a value above 1, or a
//          candidate time that is not a finite positive number, is counted as an evaluation
//          error; values above 1 are not clipped, unusable times are left out)
//   Eq. 5  S_i = median over operator i's correct shapes (even count: mean of the middle two),
//          0 when there is none
//   Eq. 6  S_agg = sum_i w_i S_i, accumulated in operator order
//
// Every floating-point step is one explicit round-to-nearest operation in a fixed order, so
// the result has one bit pattern.  The median of a small group is found by ranking (each value's
// rank is the number of values that sort before it, ties broken by position), that of a large one
// by a bitwise search for the wanted order statistics; neither needs a sorting network or scratch
// memory beyond the CTA's shared memory.
#include <mutex>

#include "kernels.h"

using namespace atrex;

namespace {

constexpr int SCORE_THREADS = 256;

// Order statistics of a large group.  A double's bit pattern, with the sign bit flipped for positive
// values and all bits flipped for negative ones, orders like the value; the k-th smallest key (k from
// 0) is the largest v with #{key < v} <= k, found one bit at a time.  Called by a whole warp; every
// lane returns the value.
constexpr uint32_t SELECT_ABOVE = 128;   // below this, ranking every value against every other is cheaper
__device__ __forceinline__ unsigned long long order_key(double x) {
    const unsigned long long b = (unsigned long long)__double_as_longlong(x);
    return b ^ ((b >> 63) ? ~0ull : (1ull << 63));
}
__device__ __forceinline__ double select_kth(const double* v, uint32_t m, uint32_t k, uint32_t lane) {
    unsigned long long ans = 0;
    for (int bit = 63; bit >= 0; --bit) {
        const unsigned long long trial = ans | (1ull << bit);
        uint32_t below = 0;
        for (uint32_t a = lane; a < m; a += 32) below += order_key(v[a]) < trial ? 1u : 0u;
        below = __reduce_add_sync(0xFFFFFFFFu, below);
        if (below <= k) ans = trial;
    }
    const unsigned long long b = ans ^ ((ans >> 63) ? (1ull << 63) : ~0ull);
    return __longlong_as_double((long long)b);
}

__global__ void __launch_bounds__(SCORE_THREADS) score_kernel(const double* __restrict__ roofline_s,
                                                              const uint32_t* __restrict__ unit_op, uint32_t n_units,
                                                              const double* __restrict__ t_cand,
                                                              const uint8_t* __restrict__ correct,
                                                              const double* __restrict__ w, uint32_t n_ops,
                                                              double* s_agg, double* s_op_out, ull* errors_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double* s_val = reinterpret_cast<double*>(smem_raw);                   // [n_units] S_j grouped by operator
    double* s_med = s_val + n_units;                                       // [n_ops]   S_i
    uint32_t* s_start = reinterpret_cast<uint32_t*>(s_med + n_ops);        // [n_ops + 1]
    uint32_t* s_fill = s_start + n_ops + 1;                                // [n_ops]
    __shared__ unsigned int s_errors;
    const ull cand = blockIdx.x;
    const double* t = t_cand + cand * n_units;
    const uint8_t* ok = correct + cand * n_units;

    for (uint32_t i = threadIdx.x; i < n_ops; i += blockDim.x) s_fill[i] = 0;
    if (threadIdx.x == 0) s_errors = 0;
    __syncthreads();
    // count the usable units of each operator
    for (uint32_t j = threadIdx.x; j < n_units; j += blockDim.x) {
        const uint32_t op = unit_op[j];
        if (!ok[j] || op >= n_ops) continue;
        const double tj = t[j];
        if (!(tj > 0.0) || isinf(tj)) {
            atomicAdd(&s_errors, 1u);
            continue;
        }
        atomicAdd(&s_fill[op], 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t run = 0;
        for (uint32_t i = 0; i < n_ops; ++i) {
            s_start[i] = run;
            run += s_fill[i];
            s_fill[i] = 0;
        }
        s_start[n_ops] = run;
    }
    __syncthreads();
    // Eq. 4, placed into the operator's segment
    for (uint32_t j = threadIdx.x; j < n_units; j += blockDim.x) {
        const uint32_t op = unit_op[j];
        if (!ok[j] || op >= n_ops) continue;
        const double tj = t[j];
        if (!(tj > 0.0) || isinf(tj)) continue;
        const double s = __ddiv_rn(roofline_s[j], tj);
        if (s > 1.0) atomicAdd(&s_errors, 1u);
        s_val[s_start[op] + atomicAdd(&s_fill[op], 1u)] = s;
    }
    __syncthreads();
    // Eq. 5: one warp per operator, median by ranking
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u, n_warps = blockDim.x >> 5;
    for (uint32_t op = warp; op < n_ops; op += n_warps) {
        const uint32_t lo = s_start[op], m = s_start[op + 1] - lo;
        if (m == 0) {
            if (lane == 0) s_med[op] = 0.0;
            continue;
        }
        const uint32_t want_hi = m / 2, want_lo = (m & 1u) ? m / 2 : m / 2 - 1;
        double v_hi = 0.0, v_lo = 0.0;
        if (m > SELECT_ABOVE) {
            // a large group: the wanted order statistics by a bitwise search over order-preserving keys
            // (64 counting passes over the group instead of m)
            const double hi = select_kth(s_val + lo, m, want_hi, lane);
            const double lw = (m & 1u) ? hi : select_kth(s_val + lo, m, want_lo, lane);
            if (lane == 0) s_med[op] = (m & 1u) ? hi : __dmul_rn(__dadd_rn(lw, hi), 0.5);
            continue;
        }
        for (uint32_t a = lane; a < m; a += 32) {
            const double x = s_val[lo + a];
            uint32_t rank = 0;
            for (uint32_t b = 0; b < m; ++b) {
                const double y = s_val[lo + b];
                rank += (y < x || (y == x && b < a)) ? 1u : 0u;
            }
            if (rank == want_hi) v_hi = x;
            if (rank == want_lo) v_lo = x;
        }
        // exactly one lane holds each of the two wanted values; the others contribute +0.0
        for (int off = 16; off > 0; off >>= 1) {
            v_hi += __shfl_xor_sync(0xFFFFFFFFu, v_hi, off);
            v_lo += __shfl_xor_sync(0xFFFFFFFFu, v_lo, off);
        }
        if (lane == 0) s_med[op] = (m & 1u) ? v_hi : __dmul_rn(__dadd_rn(v_lo, v_hi), 0.5);
    }
    __syncthreads();
    if (s_op_out)
        for (uint32_t i = threadIdx.x; i < n_ops; i += blockDim.x) s_op_out[cand * n_ops + i] = s_med[i];
    if (threadIdx.x == 0) {
        double agg = 0.0;  // Eq. 6 in operator order
        for (uint32_t i = 0; i < n_ops; ++i) agg = __dadd_rn(agg, __dmul_rn(w[i], s_med[i]));
        s_agg[cand] = agg;
        if (errors_out) errors_out[cand] = s_errors;
    }
}

constexpr int SCORE_MAX_DEVICES = 64;
std::mutex g_score_lock;
bool g_score_prepared[SCORE_MAX_DEVICES];   // per device: the kernel's shared-memory limit has been raised

struct ScoreDeviceGuard {
    int prev = -1;
    bool switched = false, ok = true;
    explicit ScoreDeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) {
            switched = cudaSetDevice(dev) == cudaSuccess;
            ok = switched;
        }
    }
    ~ScoreDeviceGuard() {
        if (switched && prev >= 0) cudaSetDevice(prev);
    }
};

}  // namespace

extern "C" int atrex_score_aggregate(const double* d_roofline_s, const uint32_t* d_unit_op, uint64_t n_units,
                                     const double* d_t_cand, const uint8_t* d_correct, uint64_t n_candidates,
                                     const double* d_w, uint32_t n_ops, double* d_s_agg, double* d_s_op,
                                     uint64_t* d_errors, void* stream) {
    if (n_candidates == 0) return ATREX_OK;
    if (!d_roofline_s || !d_unit_op || !d_t_cand || !d_correct || !d_w || !d_s_agg) return ATREX_ERR_INVALID;
    if (n_units == 0 || n_ops == 0) return ATREX_ERR_INVALID;
    if (n_units > ATREX_SCORE_MAX_UNITS || n_ops > ATREX_SCORE_MAX_OPS || n_candidates > 0x7FFFFFFFull)
        return ATREX_ERR_TOO_LARGE;
    const size_t smem = (size_t)n_units * 8 + (size_t)n_ops * 8 + ((size_t)2 * n_ops + 1) * 4;
    // the inputs live on some device: run there, and raise that device's shared-memory limit once
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, d_t_cand) != cudaSuccess || attr.type != cudaMemoryTypeDevice || attr.device < 0 ||
        attr.device >= SCORE_MAX_DEVICES) {
        cudaGetLastError();
        return ATREX_ERR_INVALID;
    }
    ScoreDeviceGuard guard(attr.device);
    if (!guard.ok) {
        cudaGetLastError();
        return ATREX_ERR_CUDA;
    }
    {
        std::lock_guard<std::mutex> hold(g_score_lock);
        if (!g_score_prepared[attr.device]) {
            if (cudaFuncSetAttribute(score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) {
                cudaGetLastError();
                return ATREX_ERR_CUDA;
            }
            g_score_prepared[attr.device] = true;
        }
    }
    score_kernel<<<(unsigned)n_candidates, SCORE_THREADS, smem, (cudaStream_t)stream>>>(
        d_roofline_s, d_unit_op, (uint32_t)n_units, d_t_cand, d_correct, d_w, n_ops, d_s_agg, d_s_op,
        reinterpret_cast<ull*>(d_errors));
    return cudaGetLastError() == cudaSuccess ? ATREX_OK : ATREX_ERR_CUDA;
}
