// CUDA restatement of the seeded record law in tracegen/cpu.py: record i is a pure integer
// function of (base, i) over host-built tables.  Input generation only -- no aggregation,
// weighting or roofline arithmetic lives here.
#include <cstdint>
#include <cuda_runtime.h>

typedef unsigned long long ull;

struct TracegenParams {
    ull base;
    uint32_t kind;        // 0 uniform, 1 zipf-per-op, 2 key list, 3 hot key
    uint32_t n_apps, n_ops, n_shapes, n_phases;
    uint32_t phase_cum[8];
    ull n_ranks;
    const ull* cum;       // device, n_ranks
    const uint32_t* perm_a;
    const uint32_t* perm_b;
    ull kl_a, kl_b;
    uint32_t hot_thresh, hot_phase, hot_op, hot_shape;
    uint32_t dur_kind, dur_lo, dur_range;
    const uint32_t* qtable;  // device, 65536
};

__device__ __forceinline__ ull mix64(ull x) {
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

__device__ __forceinline__ ull rank_of(const TracegenParams& p, ull u) {
    // first index whose cumulative value exceeds u (numpy searchsorted side='right'), clamped
    ull lo = 0, hi = p.n_ranks;
    while (lo < hi) {
        ull mid = (lo + hi) >> 1;
        if (p.cum[mid] <= u) lo = mid + 1; else hi = mid;
    }
    return lo < p.n_ranks - 1 ? lo : p.n_ranks - 1;
}

__global__ void tracegen_kernel(TracegenParams p, ull start, ull count, uint4* out) {
    const ull GOLD = 0x9E3779B97F4A7C15ull;
    for (ull j = (ull)blockIdx.x * blockDim.x + threadIdx.x; j < count; j += (ull)gridDim.x * blockDim.x) {
        ull i = start + j;
        ull h0 = mix64(p.base + 0x0000000000000000ull + i * GOLD);
        ull h1 = mix64(p.base + 0x6A09E667F3BCC909ull + i * GOLD);
        ull h2 = mix64(p.base + 0xBB67AE8584CAA73Bull + i * GOLD);
        uint32_t app = (uint32_t)(((h0 & 0xFFFFFFFFull) * p.n_apps) >> 32);
        ull per_phase = (ull)p.n_ops * p.n_shapes;
        uint32_t op, phase, shape;
        if (p.kind <= 1) {
            op = (uint32_t)((((h0 >> 32) & 0xFFFFull) * p.n_ops) >> 16);
            uint32_t u16 = (uint32_t)(h0 >> 48);
            phase = 0;
            for (uint32_t q = 0; q + 1 < p.n_phases; ++q) phase += (u16 >= p.phase_cum[q]) ? 1u : 0u;
            if (p.kind == 0) {
                shape = (uint32_t)(((h1 & 0xFFFFFFFFull) * p.n_shapes) >> 32);
            } else {
                ull rank = rank_of(p, h1);
                shape = (uint32_t)((rank * p.perm_a[op] + p.perm_b[op]) & (ull)(p.n_shapes - 1));
            }
        } else if (p.kind == 2) {
            ull rank = rank_of(p, h1);
            ull t = (rank * p.kl_a + p.kl_b) % (3ull * per_phase);
            phase = (uint32_t)(t / per_phase);
            ull rem = t % per_phase;
            op = (uint32_t)(rem / p.n_shapes);
            shape = (uint32_t)(rem % p.n_shapes);
        } else {
            bool hot = (uint32_t)(h1 & 0xFFFFFFFFull) < p.hot_thresh;
            ull cold = ((h1 >> 32) * ((ull)p.n_phases * per_phase)) >> 32;
            ull rem = cold % per_phase;
            phase = hot ? p.hot_phase : (uint32_t)(cold / per_phase);
            op = hot ? p.hot_op : (uint32_t)(rem / p.n_shapes);
            shape = hot ? p.hot_shape : (uint32_t)(rem % p.n_shapes);
        }
        uint32_t d;
        if (p.dur_kind == 0) d = p.dur_lo + (uint32_t)(((h2 & 0xFFFFFFFFull) * p.dur_range) >> 32);
        else if (p.dur_kind == 1) d = p.qtable[h2 >> 48];
        else d = p.dur_lo;
        out[j] = make_uint4(app, (op & 0xFFFFu) | ((phase & 0xFFu) << 16), shape, d);
    }
}

extern "C" int tracegen_generate(const TracegenParams* params, ull start, ull count, void* d_out, void* stream) {
    if (!params || (count && !d_out)) return -1;
    if (count == 0) return 0;
    ull blocks = (count + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    tracegen_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(*params, start, count, (uint4*)d_out);
    return cudaGetLastError() == cudaSuccess ? 0 : -2;
}
