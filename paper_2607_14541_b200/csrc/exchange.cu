// The exchange step of the multi-GPU path.  Eq. 2's sums run over independent records and every
// accumulator is an exact integer, so each GPU aggregates its own slice of the trace; afterwards every
// aggregated entry travels to the GPU that owns its key and is folded in there (atrex_agg_merge).
// This file holds the arithmetic of that step, so that none of it runs in the host language:
// the owner function, the grouping of an entry array by owner (count, reserve, scatter), and the exact
// 128-bit combination of the shards' per-phase totals (an element-wise reduction of 64-bit halves
// would lose carries).  The bytes themselves are moved by the caller's collective.
#include "kernels.h"

using namespace atrex;

namespace {

constexpr int BUCKET_THREADS = 256;
constexpr int BUCKET_PER_THREAD = 8;   // entries per thread: 2048 per CTA

__host__ __device__ __forceinline__ uint32_t owner_of(ull key, uint32_t world) {
    return (uint32_t)(((key * 0x9E3779B97F4A7C15ull) >> 33) % world);
}

// One CTA groups a tile of entries: every entry takes a ticket from its owner's shared-memory counter
// (its rank among the tile's entries of that owner), the CTA reserves one range per owner in the
// output with a single global atomic each, and the entries are written to range start + ticket.
// Tickets are drawn per warp and owner, not per entry: the lanes of a warp that share an owner are
// found with a match, one of them adds their number to the counter and the others take consecutive
// places (with a handful of owners, one atomic per entry on the same few counters took 4 ms for
// 16 M entries).  With `count_only` the tile's counts are just added to `counts` (first pass).
__global__ void __launch_bounds__(BUCKET_THREADS) bucket_kernel(const atrex_entry_t* in, ull n, uint32_t world, atrex_entry_t* out,
                                                                ull* counts, ull* cursors, int count_only) {
    extern __shared__ ull s_mem[];   // [world] range starts, then [world] 32-bit ticket counters
    ull* s_base = s_mem;
    uint32_t* s_count = reinterpret_cast<uint32_t*>(s_mem + world);
    const uint32_t lane = threadIdx.x & 31u;
    const ull tile = (ull)BUCKET_THREADS * BUCKET_PER_THREAD;
    for (ull t0 = (ull)blockIdx.x * tile; t0 < n; t0 += (ull)gridDim.x * tile) {
        for (uint32_t i = threadIdx.x; i < world; i += blockDim.x) s_count[i] = 0;
        __syncthreads();
        uint32_t owner[BUCKET_PER_THREAD], ticket[BUCKET_PER_THREAD];
#pragma unroll
        for (int u = 0; u < BUCKET_PER_THREAD; ++u) {
            const ull i = t0 + (ull)u * BUCKET_THREADS + threadIdx.x;
            owner[u] = i < n ? owner_of(in[i].key, world) : 0xFFFFFFFFu;
            const unsigned same = __match_any_sync(0xFFFFFFFFu, owner[u]);   // (all lanes take part)
            const int leader = __ffs(same) - 1;
            uint32_t first = 0;
            if ((int)lane == leader && owner[u] != 0xFFFFFFFFu) first = atomicAdd(&s_count[owner[u]], (uint32_t)__popc(same));
            ticket[u] = __shfl_sync(0xFFFFFFFFu, first, leader) + (uint32_t)__popc(same & ((1u << lane) - 1u));
        }
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < world; i += blockDim.x) {
            const ull c = s_count[i];
            if (c != 0) {
                if (count_only)
                    atomicAdd(&counts[i], c);
                else
                    s_base[i] = atomicAdd(&cursors[i], c);
            }
        }
        __syncthreads();
        if (!count_only) {
#pragma unroll
            for (int u = 0; u < BUCKET_PER_THREAD; ++u) {
                const ull i = t0 + (ull)u * BUCKET_THREADS + threadIdx.x;
                if (owner[u] != 0xFFFFFFFFu) out[s_base[owner[u]] + ticket[u]] = in[i];
            }
        }
        __syncthreads();
    }
}

}  // namespace

extern "C" {

uint32_t atrex_key_owner(uint64_t key, uint32_t world) { return world ? owner_of(key, world) : 0u; }

void atrex_keys_owner(const uint64_t* h_keys, uint64_t n, uint32_t world, uint32_t* h_out) {
    for (uint64_t i = 0; i < n; ++i) h_out[i] = world ? owner_of(h_keys[i], world) : 0u;
}

int atrex_entries_bucket_by_owner(const atrex_entry_t* d_entries, uint64_t n, uint32_t world, atrex_entry_t* d_out,
                                  uint64_t* d_scratch, uint64_t* h_counts, void* stream) {
    if (world == 0 || world > ATREX_MAX_WORLD || !h_counts || !d_scratch) return ATREX_ERR_INVALID;
    for (uint32_t i = 0; i < world; ++i) h_counts[i] = 0;
    if (n == 0) return ATREX_OK;
    if (!d_entries || !d_out || ((uintptr_t)d_entries & 15u) || ((uintptr_t)d_out & 15u) || ((uintptr_t)d_scratch & 7u))
        return ATREX_ERR_INVALID;
    if (n > (1ull << 32)) return ATREX_ERR_TOO_LARGE;
    // the entries live on some device: run there
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, d_entries) != cudaSuccess || attr.type != cudaMemoryTypeDevice) {
        cudaGetLastError();
        return ATREX_ERR_INVALID;
    }
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    if (prev != attr.device && cudaSetDevice(attr.device) != cudaSuccess) {
        cudaGetLastError();
        return ATREX_ERR_CUDA;
    }
    struct Restore {
        int dev;
        ~Restore() {
            if (dev >= 0) cudaSetDevice(dev);
        }
    } restore{prev != attr.device ? prev : -1};
    int n_sms = 148;
    if (cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, attr.device) != cudaSuccess || n_sms <= 0) n_sms = 148;
    cudaStream_t s = (cudaStream_t)stream;
    ull* counts = (ull*)d_scratch;
    ull* cursors = counts + world;
    const ull tile = (ull)BUCKET_THREADS * BUCKET_PER_THREAD;
    int grid = (int)((n + tile - 1) / tile);
    if (grid > n_sms * 8) grid = n_sms * 8;
    const size_t smem = (size_t)world * 16;
    if (cudaMemsetAsync(counts, 0, (size_t)world * 8, s) != cudaSuccess) return ATREX_ERR_CUDA;
    bucket_kernel<<<grid, BUCKET_THREADS, smem, s>>>(d_entries, n, world, d_out, counts, cursors, 1);
    if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
    if (cudaMemcpyAsync(h_counts, counts, (size_t)world * 8, cudaMemcpyDeviceToHost, s) != cudaSuccess) return ATREX_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return ATREX_ERR_CUDA;
    // range starts: exclusive prefix of the counts
    uint64_t starts[ATREX_MAX_WORLD];
    uint64_t acc = 0;
    for (uint32_t i = 0; i < world; ++i) {
        starts[i] = acc;
        acc += h_counts[i];
    }
    if (acc != n) return ATREX_ERR_CUDA;
    if (cudaMemcpyAsync(cursors, starts, (size_t)world * 8, cudaMemcpyHostToDevice, s) != cudaSuccess) return ATREX_ERR_CUDA;
    bucket_kernel<<<grid, BUCKET_THREADS, smem, s>>>(d_entries, n, world, d_out, counts, cursors, 0);
    if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return ATREX_ERR_CUDA;   // `starts` lives on this stack frame
    return ATREX_OK;
}

int atrex_totals_combine(const uint64_t* h_lo, const uint64_t* h_hi, uint32_t n_ranks, uint64_t* h_out_lo,
                         uint64_t* h_out_hi) {
    if (!h_lo || !h_hi || !h_out_lo || !h_out_hi) return ATREX_ERR_INVALID;
    for (int p = 0; p < ATREX_MAX_PHASES; ++p) {
        unsigned __int128 t = 0;
        for (uint32_t r = 0; r < n_ranks; ++r)
            t += ((unsigned __int128)h_hi[(size_t)r * ATREX_MAX_PHASES + p] << 64) | h_lo[(size_t)r * ATREX_MAX_PHASES + p];
        h_out_lo[p] = (uint64_t)t;
        h_out_hi[p] = (uint64_t)(t >> 64);
    }
    return ATREX_OK;
}

}  // extern "C"
