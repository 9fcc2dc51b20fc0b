// Release artefacts made from a list of aggregated entries: the list in key order, and the
// per-phase ranking with its running share and coverage cut (the construction behind Table 2:
// operators ordered by weight, a "Cum." column beside them).
//
// Both are built on one primitive, a stable least-significant-digit radix sort of
// (64-bit word, 32-bit entry index) pairs with 8-bit digits (tiles reordered in shared memory, so
// that every pass writes contiguous runs).  The ranking order
// (weighted time descending, key ascending) is a 3-word composite; since the sort is stable it
// is produced word by word, least significant first: key, then ~wt_lo, then ~wt_hi, each word
// gathered through the current permutation.  A digit on which all words agree (the bitwise OR
// and AND of the words match there) is skipped, so a pass is only paid for digits that carry
// information: 6 of 8 for the key of one phase, 3 or fewer for wt_hi.
//
// The running sum is an exact 128-bit prefix sum in rank order (block sums, a scan of the block
// sums, a block-local scan), rounded once per row when the share is formed.
#include <mutex>

#include "kernels.h"

using namespace atrex;

namespace {

constexpr int SORT_WARPS = 16;                                // 512 threads
constexpr int SORT_ROUNDS = 16;                               // 32 items per warp and round
constexpr uint32_t SORT_TILE = SORT_WARPS * SORT_ROUNDS * 32;  // 8192 items per CTA
constexpr uint32_t SCAN_BLOCK = 1024;
constexpr uint32_t FULL = 0xFFFFFFFFu;

struct ReleaseCtl {       // 256 bytes at the start of the scratch, cleared by every call
    ull counter;          // entries of the phase
    ull word_or, word_and;
    ull total_lo, total_hi;
    ull n_keep, covered_lo, covered_hi;
    ull pad[24];
};
static_assert(sizeof(ReleaseCtl) == 256, "control block is 256 bytes");

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (switched && prev >= 0) cudaSetDevice(prev);
    }
};

__device__ __forceinline__ void add128(ull& lo, ull& hi, ull alo, ull ahi) {
    const ull s = lo + alo;
    hi += ahi + (s < lo ? 1ull : 0ull);
    lo = s;
}

// Exact 128-bit sum of two 64-bit halves kept in global memory: the low half's returning add
// tells each adder whether it produced the carry, and carries commute.
__device__ __forceinline__ void atomic_add128(ull* lo, ull* hi, ull alo, ull ahi) {
    const ull old = atomicAdd(lo, alo);
    const ull carry = (old + alo < old) ? 1ull : 0ull;
    if (ahi + carry) atomicAdd(hi, ahi + carry);
}

__device__ __forceinline__ void warp_or_and(ull v_or, ull v_and, ReleaseCtl* ctl) {
#pragma unroll
    for (int d = 16; d; d >>= 1) {
        v_or |= __shfl_xor_sync(FULL, v_or, d);
        v_and &= __shfl_xor_sync(FULL, v_and, d);
    }
    if ((threadIdx.x & 31) == 0) {
        atomicOr(&ctl->word_or, v_or);
        atomicAnd(&ctl->word_and, v_and);
    }
}

// Sort words for the key order: all entries, word = packed key.
__global__ void __launch_bounds__(256) init_key_words_kernel(const atrex_entry_t* entries, uint32_t n, ull* words,
                                                             uint32_t* idx, ReleaseCtl* ctl) {
    ull v_or = 0, v_and = ~0ull;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const ull key = entries[i].key;
        words[i] = key;
        idx[i] = i;
        v_or |= key;
        v_and &= key;
    }
    warp_or_and(v_or, v_and, ctl);
}

// Entries of `phase` are compacted to (key, index) pairs; their weighted times are summed exactly.
__global__ void __launch_bounds__(256) filter_phase_kernel(const atrex_entry_t* entries, uint32_t n, uint32_t phase,
                                                           ull* words, uint32_t* idx, ReleaseCtl* ctl) {
    ull v_or = 0, v_and = ~0ull, sum_lo = 0, sum_hi = 0;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t n_round = (n + 31u) & ~31u;  // whole warps stay in the loop for the ballots
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n_round; i += gridDim.x * blockDim.x) {
        ull key = 0;
        bool mine = false;
        if (i < n) {
            key = entries[i].key;
            mine = (uint32_t)(key >> 48) == phase;
        }
        const uint32_t mask = __ballot_sync(FULL, mine);
        if (mask == 0) continue;
        ull base = 0;
        if (lane == (uint32_t)(__ffs(mask) - 1)) base = atomicAdd(&ctl->counter, (ull)__popc(mask));
        base = __shfl_sync(FULL, base, __ffs(mask) - 1);
        if (mine) {
            const ull pos = base + __popc(mask & ((1u << lane) - 1u));
            words[pos] = key;
            idx[pos] = i;
            v_or |= key;
            v_and &= key;
            add128(sum_lo, sum_hi, entries[i].wt_lo, entries[i].wt_hi);
        }
    }
    warp_or_and(v_or, v_and, ctl);
#pragma unroll
    for (int d = 16; d; d >>= 1) {
        const ull olo = __shfl_xor_sync(FULL, sum_lo, d), ohi = __shfl_xor_sync(FULL, sum_hi, d);
        add128(sum_lo, sum_hi, olo, ohi);
    }
    if (lane == 0 && (sum_lo | sum_hi)) atomic_add128(&ctl->total_lo, &ctl->total_hi, sum_lo, sum_hi);
}

// word[r] = ~(wt_lo or wt_hi) of the entry at the current position r: ascending order of the
// complement is descending order of the weighted time.
__global__ void __launch_bounds__(256) gather_wt_words_kernel(const atrex_entry_t* entries, const uint32_t* idx,
                                                              uint32_t m, int high, ull* words, ReleaseCtl* ctl) {
    ull v_or = 0, v_and = ~0ull;
    for (uint32_t r = blockIdx.x * blockDim.x + threadIdx.x; r < m; r += gridDim.x * blockDim.x) {
        const atrex_entry_t* e = entries + idx[r];
        const ull w = ~(high ? e->wt_hi : e->wt_lo);
        words[r] = w;
        v_or |= w;
        v_and &= w;
    }
    warp_or_and(v_or, v_and, ctl);
}

// ---- one radix pass: per-tile digit counts, per-digit exclusive scan over the tiles plus digit
// totals, stable scatter (which adds the scan of the 256 digit totals itself)

__global__ void __launch_bounds__(SORT_WARPS * 32) radix_hist_kernel(const ull* words, uint32_t m, int shift,
                                                                     uint32_t* hist, uint32_t n_tiles) {
    __shared__ uint32_t h[256];
    if (threadIdx.x < 256) h[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t tile = blockIdx.x * SORT_TILE;
    for (uint32_t j = threadIdx.x; j < SORT_TILE; j += SORT_WARPS * 32) {
        const uint32_t i = tile + j;
        if (i < m) atomicAdd(&h[(uint32_t)(words[i] >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (threadIdx.x < 256) hist[(size_t)threadIdx.x * n_tiles + blockIdx.x] = h[threadIdx.x];
}

// One CTA per digit value: exclusive scan of that digit's counts over the tiles (a contiguous row,
// 1024 at a time with a running carry), and the digit's total to bin_total[digit].
__global__ void __launch_bounds__(SCAN_BLOCK) radix_scan_kernel(uint32_t* hist, uint32_t n_tiles, uint32_t* bin_total) {
    __shared__ uint32_t warp_sum[32];
    uint32_t* row = hist + (size_t)blockIdx.x * n_tiles;
    const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t carry = 0;
    for (uint32_t base = 0; base < n_tiles; base += SCAN_BLOCK) {
        const uint32_t i = base + threadIdx.x;
        const uint32_t c = i < n_tiles ? row[i] : 0u;
        uint32_t incl = c;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t o = __shfl_up_sync(FULL, incl, d);
            if (lane >= (uint32_t)d) incl += o;
        }
        if (lane == 31) warp_sum[w] = incl;
        __syncthreads();
        if (w == 0) {
            uint32_t iv = warp_sum[lane];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_up_sync(FULL, iv, d);
                if (lane >= (uint32_t)d) iv += o;
            }
            warp_sum[lane] = iv;  // inclusive over warps
        }
        __syncthreads();
        if (i < n_tiles) row[i] = carry + (w ? warp_sum[w - 1] : 0u) + incl - c;
        carry += warp_sum[31];
        __syncthreads();  // warp_sum is reused by the next round
    }
    if (threadIdx.x == 0) bin_total[blockIdx.x] = carry;
}

// Stable: item order inside a tile is (warp, round, lane) = input order; a lane's rank among
// equal digits is (items of earlier warps) + (earlier rounds of its warp) + (lower lanes of its
// round), and tiles are ordered by the scanned (digit, tile) counters.  The tile is first put in
// digit order in shared memory and then written out run by run, so that the global stores are
// contiguous per digit (about 32 items per digit and tile) instead of one scattered 12-byte piece
// per item.
constexpr size_t SCATTER_SMEM = (size_t)SORT_TILE * 12;   // words (8 B) and indices (4 B) of one tile

__global__ void __launch_bounds__(SORT_WARPS * 32) radix_scatter_kernel(const ull* words_in, const uint32_t* idx_in,
                                                                        ull* words_out, uint32_t* idx_out, uint32_t m,
                                                                        int shift, const uint32_t* hist,
                                                                        uint32_t n_tiles, const uint32_t* bin_total) {
    extern __shared__ __align__(16) unsigned char sort_smem[];
    ull* s_words = reinterpret_cast<ull*>(sort_smem);                          // [SORT_TILE] the tile in digit order
    uint32_t* s_idx = reinterpret_cast<uint32_t*>(sort_smem + (size_t)SORT_TILE * 8);
    __shared__ uint32_t wh[SORT_WARPS][256];
    __shared__ uint32_t bin_base[256];   // exclusive scan of the digit totals (global)
    __shared__ uint32_t bin_warp[8];
    __shared__ uint32_t tile_base[256];  // first position of digit d inside this tile's digit order
    __shared__ uint32_t tile_warp[8];
    __shared__ uint32_t out_base[256];   // global position of this tile's first item of digit d
    for (uint32_t j = threadIdx.x; j < SORT_WARPS * 256; j += SORT_WARPS * 32) (&wh[0][0])[j] = 0;
    __syncthreads();
    const uint32_t w = threadIdx.x >> 5, lane = threadIdx.x & 31, lt = (1u << lane) - 1u;
    const uint32_t tile_start = blockIdx.x * SORT_TILE;
    const uint32_t first = tile_start + w * (SORT_ROUNDS * 32) + lane;
    uint32_t packed[SORT_ROUNDS];  // digit | rank inside the warp << 9
#pragma unroll
    for (int r = 0; r < SORT_ROUNDS; ++r) {
        const uint32_t i = first + r * 32;
        const bool valid = i < m;
        const uint32_t d = valid ? (uint32_t)(words_in[i] >> shift) & 255u : 256u + lane;  // padding never groups
        const uint32_t same = __match_any_sync(FULL, d);
        const uint32_t base = valid ? wh[w][d] : 0u;
        __syncwarp();
        if (valid && (same & lt) == 0) wh[w][d] = base + __popc(same);
        __syncwarp();
        packed[r] = d | ((base + __popc(same & lt)) << 9);
    }
    __syncthreads();
    uint32_t tile_count = 0;
    if (threadIdx.x < 256) {
        // this digit's items in the tile, per warp -> running offsets; the digit totals -> global bases
#pragma unroll
        for (int k = 0; k < SORT_WARPS; ++k) {
            const uint32_t c = wh[k][threadIdx.x];
            wh[k][threadIdx.x] = tile_count;     // items of this digit in earlier warps
            tile_count += c;
        }
        const uint32_t c = bin_total[threadIdx.x];
        uint32_t incl = c, tincl = tile_count;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t o = __shfl_up_sync(FULL, incl, d), to = __shfl_up_sync(FULL, tincl, d);
            if (lane >= (uint32_t)d) {
                incl += o;
                tincl += to;
            }
        }
        if (lane == 31) {
            bin_warp[w] = incl;
            tile_warp[w] = tincl;
        }
        bin_base[threadIdx.x] = incl - c;
        tile_base[threadIdx.x] = tincl - tile_count;
    }
    __syncthreads();
    if (threadIdx.x < 256) {
        uint32_t g = bin_base[threadIdx.x] + hist[(size_t)threadIdx.x * n_tiles + blockIdx.x], t = tile_base[threadIdx.x];
        for (uint32_t k = 0; k < w; ++k) {
            g += bin_warp[k];
            t += tile_warp[k];
        }
        out_base[threadIdx.x] = g;
        tile_base[threadIdx.x] = t;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < SORT_ROUNDS; ++r) {
        const uint32_t i = first + r * 32;
        if (i < m) {
            const uint32_t d = packed[r] & 511u;
            const uint32_t at = tile_base[d] + wh[w][d] + (packed[r] >> 9);
            s_words[at] = words_in[i];
            s_idx[at] = idx_in[i];
        }
    }
    __syncthreads();
    const uint32_t tile_n = min(SORT_TILE, m - tile_start);
    for (uint32_t j = threadIdx.x; j < tile_n; j += SORT_WARPS * 32) {
        const ull word = s_words[j];
        const uint32_t d = (uint32_t)(word >> shift) & 255u;
        const uint32_t pos = out_base[d] + (j - tile_base[d]);
        words_out[pos] = word;
        idx_out[pos] = s_idx[j];
    }
}

__global__ void __launch_bounds__(256) gather_entries_kernel(const atrex_entry_t* entries, const uint32_t* idx,
                                                             uint32_t m, atrex_entry_t* out) {
    for (uint32_t r = blockIdx.x * blockDim.x + threadIdx.x; r < m; r += gridDim.x * blockDim.x)
        out[r] = entries[idx[r]];
}

// ---- exact running sum in rank order

__device__ __forceinline__ void block_scan128(ull& lo, ull& hi, ull (*warp_tot)[2], ull& block_lo, ull& block_hi) {
    const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const ull olo = __shfl_up_sync(FULL, lo, d), ohi = __shfl_up_sync(FULL, hi, d);
        if (lane >= (uint32_t)d) add128(lo, hi, olo, ohi);
    }
    if (lane == 31) {
        warp_tot[w][0] = lo;
        warp_tot[w][1] = hi;
    }
    __syncthreads();
    if (w == 0) {
        ull tlo = warp_tot[lane][0], thi = warp_tot[lane][1];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const ull olo = __shfl_up_sync(FULL, tlo, d), ohi = __shfl_up_sync(FULL, thi, d);
            if (lane >= (uint32_t)d) add128(tlo, thi, olo, ohi);
        }
        warp_tot[lane][0] = tlo;  // inclusive over warps
        warp_tot[lane][1] = thi;
    }
    __syncthreads();
    if (w > 0) add128(lo, hi, warp_tot[w - 1][0], warp_tot[w - 1][1]);
    block_lo = warp_tot[31][0];
    block_hi = warp_tot[31][1];
}

__global__ void __launch_bounds__(SCAN_BLOCK) rank_block_sums_kernel(const atrex_entry_t* entries, const uint32_t* idx,
                                                                     uint32_t m, ull* bsums) {
    __shared__ ull warp_tot[32][2];
    const uint32_t r = blockIdx.x * SCAN_BLOCK + threadIdx.x;
    ull lo = 0, hi = 0;
    if (r < m) {
        const atrex_entry_t* e = entries + idx[r];
        lo = e->wt_lo;
        hi = e->wt_hi;
    }
    ull blo, bhi;
    block_scan128(lo, hi, warp_tot, blo, bhi);
    if (threadIdx.x == 0) {
        bsums[2 * blockIdx.x] = blo;
        bsums[2 * blockIdx.x + 1] = bhi;
    }
}

// Exclusive scan of the block sums by one CTA, 1024 at a time with a running carry-in.
__global__ void __launch_bounds__(SCAN_BLOCK) rank_scan_sums_kernel(ull* bsums, uint32_t nb) {
    __shared__ ull warp_tot[32][2];
    ull run_lo = 0, run_hi = 0;
    for (uint32_t base = 0; base < nb; base += SCAN_BLOCK) {
        const uint32_t b = base + threadIdx.x;
        ull lo = 0, hi = 0;
        if (b < nb) {
            lo = bsums[2 * b];
            hi = bsums[2 * b + 1];
        }
        const ull own_lo = lo, own_hi = hi;
        ull blo, bhi;
        block_scan128(lo, hi, warp_tot, blo, bhi);
        if (b < nb) {
            // exclusive = carry-in + inclusive - own
            ull elo = lo - own_lo, ehi = hi - own_hi - (lo < own_lo ? 1ull : 0ull);
            add128(elo, ehi, run_lo, run_hi);
            bsums[2 * b] = elo;
            bsums[2 * b + 1] = ehi;
        }
        add128(run_lo, run_hi, blo, bhi);
        __syncthreads();  // warp_tot is reused by the next round
    }
}

__device__ __forceinline__ bool less128(ull alo, ull ahi, ull blo, ull bhi) {
    return ahi < bhi || (ahi == bhi && alo < blo);
}

// Row r of the ranking: the entry, its running share fl(fl(prefix) / fl(T)), and the coverage cut
// (the one row whose exclusive prefix is below the needed sum and whose inclusive prefix reaches it).
__global__ void __launch_bounds__(SCAN_BLOCK) rank_emit_kernel(const atrex_entry_t* entries, const uint32_t* idx,
                                                               uint32_t m, const ull* bsums, ull total_lo, ull total_hi,
                                                               ull need_lo, ull need_hi, atrex_entry_t* out,
                                                               double* cum, uint32_t out_cap, ReleaseCtl* ctl) {
    __shared__ ull warp_tot[32][2];
    const uint32_t r = blockIdx.x * SCAN_BLOCK + threadIdx.x;
    ull lo = 0, hi = 0;
    const atrex_entry_t* e = nullptr;
    if (r < m) {
        e = entries + idx[r];
        lo = e->wt_lo;
        hi = e->wt_hi;
    }
    const ull own_lo = lo, own_hi = hi;
    ull blo, bhi;
    block_scan128(lo, hi, warp_tot, blo, bhi);
    if (r >= m) return;
    add128(lo, hi, bsums[2 * blockIdx.x], bsums[2 * blockIdx.x + 1]);  // inclusive prefix of the whole list
    const ull ex_lo = lo - own_lo, ex_hi = hi - own_hi - (lo < own_lo ? 1ull : 0ull);
    if ((need_lo | need_hi) && less128(ex_lo, ex_hi, need_lo, need_hi) && !less128(lo, hi, need_lo, need_hi)) {
        ctl->n_keep = (ull)r + 1;
        ctl->covered_lo = lo;
        ctl->covered_hi = hi;
    }
    if (r < out_cap) {
        out[r] = *e;
        cum[r] = (total_lo | total_hi) ? __ddiv_rn(u128_to_f64_rn(hi, lo), u128_to_f64_rn(total_hi, total_lo)) : 0.0;
    }
}

// ---- host side

struct Scratch {
    ReleaseCtl* ctl;
    ull* words[2];
    uint32_t* idx[2];
    uint32_t* hist;
    uint32_t* bin_total;
    ull* bsums;
};

inline uint64_t align256(uint64_t x) { return (x + 255u) & ~(uint64_t)255u; }

uint64_t scratch_bytes_for(uint64_t n) {
    const uint64_t tiles = (n + SORT_TILE - 1) / SORT_TILE, blocks = (n + SCAN_BLOCK - 1) / SCAN_BLOCK;
    return sizeof(ReleaseCtl) + 2 * align256(n * 8) + 2 * align256(n * 4) + align256(tiles * 256 * 4) +
           1024 + align256(blocks * 16) + 256;
}

Scratch carve(void* base, uint64_t n) {
    const uint64_t tiles = (n + SORT_TILE - 1) / SORT_TILE;
    unsigned char* p = (unsigned char*)base;
    Scratch s;
    s.ctl = (ReleaseCtl*)p;
    p += sizeof(ReleaseCtl);
    for (int b = 0; b < 2; ++b) {
        s.words[b] = (ull*)p;
        p += align256(n * 8);
    }
    for (int b = 0; b < 2; ++b) {
        s.idx[b] = (uint32_t*)p;
        p += align256(n * 4);
    }
    s.hist = (uint32_t*)p;
    p += align256(tiles * 256 * 4);
    s.bin_total = (uint32_t*)p;
    p += 1024;
    s.bsums = (ull*)p;
    return s;
}

int grid_for(uint64_t n, int block) {
    uint64_t g = (n + block - 1) / block;
    return (int)(g < 1 ? 1 : (g > 148 * 8 ? 148 * 8 : g));
}

// Reads back the control block (synchronises the stream).
int read_ctl(const Scratch& sc, ReleaseCtl* host, cudaStream_t s) {
    if (cudaMemcpyAsync(host, sc.ctl, sizeof(ReleaseCtl), cudaMemcpyDeviceToHost, s) != cudaSuccess) return ATREX_ERR_CUDA;
    return cudaStreamSynchronize(s) == cudaSuccess ? ATREX_OK : ATREX_ERR_CUDA;
}

int reset_or_and(const Scratch& sc, cudaStream_t s) {
    const ull init[2] = {0ull, ~0ull};
    return cudaMemcpyAsync(&sc.ctl->word_or, init, sizeof(init), cudaMemcpyHostToDevice, s) == cudaSuccess ? ATREX_OK
                                                                                                             : ATREX_ERR_CUDA;
}

// Sorts the m pairs in buffer `cur` by the digits of the word on which the words differ.
// Returns the buffer that holds the result, or a negative status.
// The scatter kernel keeps a whole tile in shared memory: raise its dynamic shared-memory limit once per
// device (the caller has made the entries' device current).
int prepare_sort_kernels() {
    static std::mutex lock;
    static bool prepared[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ATREX_ERR_CUDA;
    std::lock_guard<std::mutex> hold(lock);
    if (!prepared[dev]) {
        if (cudaFuncSetAttribute(radix_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SCATTER_SMEM) != cudaSuccess) {
            cudaGetLastError();
            return ATREX_ERR_CUDA;
        }
        prepared[dev] = true;
    }
    return ATREX_OK;
}

int sort_by_word(const Scratch& sc, int cur, uint32_t m, ull differing_bits, cudaStream_t s) {
    const uint32_t tiles = (m + SORT_TILE - 1) / SORT_TILE;
    if (prepare_sort_kernels() != ATREX_OK) return ATREX_ERR_CUDA;
    for (int shift = 0; shift < 64; shift += 8) {
        if (((differing_bits >> shift) & 255u) == 0) continue;
        radix_hist_kernel<<<tiles, SORT_WARPS * 32, 0, s>>>(sc.words[cur], m, shift, sc.hist, tiles);
        radix_scan_kernel<<<256, SCAN_BLOCK, 0, s>>>(sc.hist, tiles, sc.bin_total);
        radix_scatter_kernel<<<tiles, SORT_WARPS * 32, SCATTER_SMEM, s>>>(sc.words[cur], sc.idx[cur], sc.words[cur ^ 1],
                                                                sc.idx[cur ^ 1], m, shift, sc.hist, tiles,
                                                                sc.bin_total);
        if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
        cur ^= 1;
    }
    return cur;
}

int check_device_pointer(const void* p, int* dev) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, p) != cudaSuccess || attr.type != cudaMemoryTypeDevice) {
        cudaGetLastError();
        return ATREX_ERR_INVALID;
    }
    *dev = attr.device;
    return ATREX_OK;
}

}  // namespace

extern "C" uint64_t atrex_release_scratch_bytes(uint64_t n) {
    if (n > ATREX_RELEASE_MAX_ENTRIES) return 0;
    return scratch_bytes_for(n < 1 ? 1 : n);
}

extern "C" int atrex_entries_sort_by_key(const atrex_entry_t* d_entries, uint64_t n, atrex_entry_t* d_out,
                                         void* d_scratch, uint64_t scratch_bytes, void* stream) {
    if (n > ATREX_RELEASE_MAX_ENTRIES) return ATREX_ERR_TOO_LARGE;
    if (n == 0) return ATREX_OK;
    if (!d_entries || !d_out || !d_scratch || d_entries == d_out) return ATREX_ERR_INVALID;
    if (((uintptr_t)d_entries & 7u) || ((uintptr_t)d_out & 7u) || ((uintptr_t)d_scratch & 255u)) return ATREX_ERR_INVALID;
    if (scratch_bytes < scratch_bytes_for(n)) return ATREX_ERR_NOMEM;
    int dev = 0;
    if (check_device_pointer(d_entries, &dev) != ATREX_OK) return ATREX_ERR_INVALID;
    DeviceGuard guard(dev);
    cudaStream_t s = (cudaStream_t)stream;
    const Scratch sc = carve(d_scratch, n);
    const uint32_t m = (uint32_t)n;

    if (cudaMemsetAsync(sc.ctl, 0, sizeof(ReleaseCtl), s) != cudaSuccess) return ATREX_ERR_CUDA;
    if (reset_or_and(sc, s) != ATREX_OK) return ATREX_ERR_CUDA;
    init_key_words_kernel<<<grid_for(n, 256), 256, 0, s>>>(d_entries, m, sc.words[0], sc.idx[0], sc.ctl);
    if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
    ReleaseCtl host;
    if (read_ctl(sc, &host, s) != ATREX_OK) return ATREX_ERR_CUDA;
    const int cur = sort_by_word(sc, 0, m, host.word_or ^ host.word_and, s);
    if (cur < 0) return cur;
    gather_entries_kernel<<<grid_for(n, 256), 256, 0, s>>>(d_entries, sc.idx[cur], m, d_out);
    if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
    return cudaStreamSynchronize(s) == cudaSuccess ? ATREX_OK : ATREX_ERR_CUDA;
}

extern "C" int atrex_entries_rank(const atrex_entry_t* d_entries, uint64_t n, uint32_t phase, uint32_t coverage_ppm,
                                  atrex_entry_t* d_ranked, double* d_cum_share, uint64_t out_cap,
                                  atrex_rank_result_t* h_result, void* d_scratch, uint64_t scratch_bytes,
                                  void* stream) {
    if (!h_result) return ATREX_ERR_INVALID;
    *h_result = atrex_rank_result_t{};
    if (n > ATREX_RELEASE_MAX_ENTRIES) return ATREX_ERR_TOO_LARGE;
    if (phase >= ATREX_MAX_PHASES || coverage_ppm > 1000000u) return ATREX_ERR_INVALID;
    if (n == 0) return ATREX_OK;
    if (!d_entries || !d_scratch || (out_cap && (!d_ranked || !d_cum_share))) return ATREX_ERR_INVALID;
    if (((uintptr_t)d_entries & 7u) || ((uintptr_t)d_ranked & 7u) || ((uintptr_t)d_cum_share & 7u) ||
        ((uintptr_t)d_scratch & 255u) || (const void*)d_entries == (const void*)d_ranked)
        return ATREX_ERR_INVALID;
    if (scratch_bytes < scratch_bytes_for(n)) return ATREX_ERR_NOMEM;
    int dev = 0;
    if (check_device_pointer(d_entries, &dev) != ATREX_OK) return ATREX_ERR_INVALID;
    DeviceGuard guard(dev);
    cudaStream_t s = (cudaStream_t)stream;
    const Scratch sc = carve(d_scratch, n);

    // 1. the phase's entries as (key, index) pairs, their count and exact total
    if (cudaMemsetAsync(sc.ctl, 0, sizeof(ReleaseCtl), s) != cudaSuccess) return ATREX_ERR_CUDA;
    if (reset_or_and(sc, s) != ATREX_OK) return ATREX_ERR_CUDA;
    filter_phase_kernel<<<grid_for(n, 256), 256, 0, s>>>(d_entries, (uint32_t)n, phase, sc.words[0], sc.idx[0], sc.ctl);
    if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
    ReleaseCtl host;
    if (read_ctl(sc, &host, s) != ATREX_OK) return ATREX_ERR_CUDA;
    const uint32_t m = (uint32_t)host.counter;
    const ull total_lo = host.total_lo, total_hi = host.total_hi;
    h_result->n_phase = m;
    h_result->total_lo = total_lo;
    h_result->total_hi = total_hi;
    if (m == 0) return ATREX_OK;
    if ((total_hi >> 44) != 0) return ATREX_ERR_TOO_LARGE;  // T * 10^6 must fit 128 bits

    // 2. least significant word first: key ascending, then ~wt_lo, then ~wt_hi
    int cur = sort_by_word(sc, 0, m, host.word_or ^ host.word_and, s);
    if (cur < 0) return cur;
    for (int high = 0; high < 2; ++high) {
        if (reset_or_and(sc, s) != ATREX_OK) return ATREX_ERR_CUDA;
        gather_wt_words_kernel<<<grid_for(m, 256), 256, 0, s>>>(d_entries, sc.idx[cur], m, high, sc.words[cur], sc.ctl);
        if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
        if (read_ctl(sc, &host, s) != ATREX_OK) return ATREX_ERR_CUDA;
        cur = sort_by_word(sc, cur, m, host.word_or ^ host.word_and, s);
        if (cur < 0) return cur;
    }

    // 3. exact running sum, shares, coverage cut: the smallest k with 10^6 * prefix_k >= ppm * T,
    //    i.e. prefix_k >= ceil(ppm * T / 10^6)
    typedef unsigned __int128 u128;
    const u128 total = ((u128)total_hi << 64) | total_lo;
    const u128 need = ((u128)coverage_ppm * total + 999999u) / 1000000u;
    const uint32_t blocks = (m + SCAN_BLOCK - 1) / SCAN_BLOCK;
    rank_block_sums_kernel<<<blocks, SCAN_BLOCK, 0, s>>>(d_entries, sc.idx[cur], m, sc.bsums);
    rank_scan_sums_kernel<<<1, SCAN_BLOCK, 0, s>>>(sc.bsums, blocks);
    rank_emit_kernel<<<blocks, SCAN_BLOCK, 0, s>>>(d_entries, sc.idx[cur], m, sc.bsums, total_lo, total_hi, (ull)need,
                                                   (ull)(need >> 64), d_ranked, d_cum_share,
                                                   (uint32_t)(out_cap < m ? out_cap : m), sc.ctl);
    if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
    if (read_ctl(sc, &host, s) != ATREX_OK) return ATREX_ERR_CUDA;
    h_result->n_keep = host.n_keep;
    h_result->covered_lo = host.covered_lo;
    h_result->covered_hi = host.covered_hi;
    return ATREX_OK;
}
