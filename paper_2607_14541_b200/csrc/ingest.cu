// Ingest: Eq. 2's group-by sum, streamed.
//
// One persistent CTA per SM.  Each thread pulls records with 32-byte vector loads (two
// 16-byte records per load, several loads in flight, streaming cache policy), packs the
// key, multiplies the application's card-hour weight by the duration, and adds
// (1, product) to the key's accumulators:
//   * keys found in the shared-memory HOT DIRECTORY (the most frequent keys of a sample of
//     the trace, identical in every CTA, read-only during the pass) are accumulated with
//     32-bit shared-memory atomics in three limbs with explicit carries; lanes of a warp
//     that hit the same slot are first combined with warp reductions;
//   * every other record goes to the global open-addressing table with one 64-bit
//     returning atomic (low limb, detects the wrap) and one 64-bit reduction
//     (count + carries), after locating / claiming the slot.
// At the end each CTA flushes its directory accumulators into the global table, so after
// the kernel the global table alone holds exact sums.  All sums are integers, so the result
// does not depend on which path a record took, on scheduling, or on chunking.
#include "atrex_dev.cuh"
#include "kernels.h"

namespace atrex {

constexpr int INGEST_THREADS = 1024;
constexpr int LOADS_PER_ITER = 2;                 // 32-byte loads in flight per thread
constexpr int RECS_PER_ITER = 2 * LOADS_PER_ITER;  // records per thread per iteration
constexpr uint32_t NO_SLOT = 0xFFFFFFFFu;

__device__ __forceinline__ uint32_t dir_bucket(ull h, uint32_t n_buckets) {
    return __umulhi((uint32_t)(h >> 20), n_buckets);
}

__device__ __forceinline__ void ld_stream_256(const void* p, uint32_t (&w)[8]) {
    asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(p));
}

struct SmemDir {
    ull* keys;        // [slots], ~key, 0 = empty
    uint32_t* cnt;    // [slots]
    uint32_t* a0;     // [slots] bits 0..31 of the slot's sum
    uint32_t* a1;     // [slots] bits 32..63
    const uint32_t* appw;
};

// Add (count, v) to a directory slot.  v < 2^53.  A wrap of the 64-bit (a1:a0) pair is rare
// and is forwarded to the global table as one unit of the high word.
__device__ __forceinline__ void dir_add(const SmemDir& d, uint32_t slot, ull v, uint32_t count,
                                        const TableRef& t, ull key, ull h) {
    atomicAdd(&d.cnt[slot], count);
    uint32_t v0 = (uint32_t)v;
    uint32_t o0 = atomicAdd(&d.a0[slot], v0);
    uint32_t x = (uint32_t)(v >> 32) + ((o0 + v0 < o0) ? 1u : 0u);
    if (x != 0) {
        uint32_t o1 = atomicAdd(&d.a1[slot], x);
        if (o1 + x < o1) table_accumulate(t, key, h, 0, 1, 0);
    }
}

// Process R records held in registers by every lane of the warp (lane-invalid ones masked).
template <bool HOT, int R>
__device__ __forceinline__ void process(const uint32_t (&w)[R][4], const bool (&present)[R], const IngestParams& p,
                                        const SmemDir& d, uint32_t& rejected) {
    ull key[R], prod[R], h[R];
    bool todo[R];  // still has to go to the global table
#pragma unroll
    for (int r = 0; r < R; ++r) {
        uint32_t app = w[r][0];
        uint32_t op = w[r][1] & 0xFFFFu;
        uint32_t phase = (w[r][1] >> 16) & 0xFFu;
        bool ok = present[r] && app < p.n_apps && phase < p.n_phases;
        rejected += (present[r] && !ok) ? 1u : 0u;
        uint32_t wgt = ok ? d.appw[app] : 0u;
        key[r] = pack_key(phase, op, w[r][2]);
        prod[r] = (ull)wgt * (ull)w[r][3];
        h[r] = hash_key(key[r]);
        todo[r] = ok;
    }
    if (HOT) {
        uint32_t slot[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            uint32_t b = dir_bucket(h[r], p.hot_buckets) * 2;
            ulonglong2 kk = *reinterpret_cast<const ulonglong2*>(d.keys + b);
            ull skey = ~key[r];
            slot[r] = !todo[r] ? NO_SLOT : (kk.x == skey ? b : (kk.y == skey ? b + 1 : NO_SLOT));
        }
        const unsigned lane = threadIdx.x & 31u;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            // combine the lanes that share the first hitting lane's slot (dominant-key case)
            unsigned hits = __ballot_sync(0xFFFFFFFFu, slot[r] != NO_SLOT);
            if (hits != 0) {
                int lead = __ffs(hits) - 1;
                uint32_t ls = __shfl_sync(0xFFFFFFFFu, slot[r], lead);
                unsigned same = __ballot_sync(0xFFFFFFFFu, slot[r] == ls);
                if (__popc(same) >= 2) {
                    if (slot[r] == ls) {
                        uint32_t s_lo = __reduce_add_sync(same, (uint32_t)prod[r] & 0xFFFFFFu);
                        uint32_t s_hi = __reduce_add_sync(same, (uint32_t)(prod[r] >> 24));
                        if (lane == (unsigned)lead)
                            dir_add(d, ls, (ull)s_lo + ((ull)s_hi << 24), (uint32_t)__popc(same), p.t, key[r], h[r]);
                        slot[r] = NO_SLOT;
                        todo[r] = false;
                    }
                }
            }
            if (slot[r] != NO_SLOT) {
                dir_add(d, slot[r], prod[r], 1u, p.t, key[r], h[r]);
                todo[r] = false;
            }
        }
    }
    // global table: issue the first-probe key loads together, then resolve, then the adds
    Slot* e[R];
    ull k0[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        e[r] = p.t.table + (h[r] >> p.t.shift);
        k0[r] = todo[r] ? ld_relaxed(&e[r]->skey) : 0ull;
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        if (todo[r] && k0[r] != ~key[r]) {
            e[r] = find_or_claim(p.t.table, p.t.mask, p.t.shift, p.t.max_probe, key[r], h[r]);
            if (e[r] == nullptr) {
                atomicOr(&p.t.ctl->status, ST_TABLE_FULL);
                atomicAdd(&p.t.ctl->n_dropped, 1ull);
                todo[r] = false;
            }
        }
    }
    ull old[R];
#pragma unroll
    for (int r = 0; r < R; ++r) old[r] = (todo[r] && prod[r] != 0) ? atomicAdd(&e[r]->lo, prod[r]) : 0ull;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        if (todo[r]) {
            ull carry = (old[r] + prod[r] < old[r]) ? 1ull : 0ull;
            atomicAdd(&e[r]->cnthi, 1ull + (carry << HI_SHIFT));
        }
    }
}

template <bool HOT>
__global__ void __launch_bounds__(INGEST_THREADS, 1) ingest_kernel(IngestParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmemDir d;
    unsigned char* sp = smem_raw;
    d.keys = reinterpret_cast<ull*>(sp);
    sp += HOT ? (size_t)p.hot_slots * 8 : 0;
    d.cnt = reinterpret_cast<uint32_t*>(sp);
    sp += HOT ? (size_t)p.hot_slots * 4 : 0;
    d.a0 = reinterpret_cast<uint32_t*>(sp);
    sp += HOT ? (size_t)p.hot_slots * 4 : 0;
    d.a1 = reinterpret_cast<uint32_t*>(sp);
    sp += HOT ? (size_t)p.hot_slots * 4 : 0;
    if (p.appw_in_smem) {
        uint32_t* s_appw = reinterpret_cast<uint32_t*>(sp);
        for (uint32_t i = threadIdx.x; i < p.n_apps; i += blockDim.x) s_appw[i] = p.app_w[i];
        d.appw = s_appw;
    } else {
        d.appw = p.app_w;
    }
    if (HOT) {
        for (uint32_t i = threadIdx.x; i < p.hot_slots; i += blockDim.x) {
            d.keys[i] = p.hot_keys[i];
            d.cnt[i] = 0;
            d.a0[i] = 0;
            d.a1[i] = 0;
        }
    }
    __syncthreads();

    uint32_t rejected = 0;
    const ull tile = (ull)INGEST_THREADS * LOADS_PER_ITER;  // pairs per CTA iteration
    const unsigned char* body = reinterpret_cast<const unsigned char*>(p.body);
    for (ull base = (ull)blockIdx.x * tile; base < p.n_pairs; base += (ull)gridDim.x * tile) {
        uint32_t w[RECS_PER_ITER][4];
        bool present[RECS_PER_ITER];
        uint32_t raw[LOADS_PER_ITER][8];
#pragma unroll
        for (int u = 0; u < LOADS_PER_ITER; ++u) {
            ull i = base + (ull)u * INGEST_THREADS + threadIdx.x;
            bool in = i < p.n_pairs;
            if (in) {
                ld_stream_256(body + i * 32, raw[u]);
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) raw[u][j] = 0;
            }
            present[2 * u] = in;
            present[2 * u + 1] = in;
        }
#pragma unroll
        for (int u = 0; u < LOADS_PER_ITER; ++u)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                w[2 * u][j] = raw[u][j];
                w[2 * u + 1][j] = raw[u][4 + j];
            }
        process<HOT, RECS_PER_ITER>(w, present, p, d, rejected);
    }
    // records that do not form an aligned pair (at most one before and one after the body)
    if (blockIdx.x == 0 && threadIdx.x < 32) {
        uint32_t w1[1][4] = {{0, 0, 0, 0}};
        bool pr[1] = {false};
        if (threadIdx.x < p.n_single) {
            uint4 v = *reinterpret_cast<const uint4*>(p.single[threadIdx.x]);
            w1[0][0] = v.x; w1[0][1] = v.y; w1[0][2] = v.z; w1[0][3] = v.w;
            pr[0] = true;
        }
        process<HOT, 1>(w1, pr, p, d, rejected);
    }
    // rejected counter: one atomic per warp
    uint32_t rsum = __reduce_add_sync(0xFFFFFFFFu, rejected);
    if ((threadIdx.x & 31u) == 0 && rsum != 0) atomicAdd(&p.t.ctl->n_rejected, (ull)rsum);

    if (HOT) {
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < p.hot_slots; i += blockDim.x) {
            uint32_t c = d.cnt[i], lo = d.a0[i], hi = d.a1[i];
            if ((c | lo | hi) != 0) {
                ull key = ~d.keys[i];
                table_accumulate(p.t, key, hash_key(key), (ull)lo | ((ull)hi << 32), 0, (ull)c);
            }
        }
    }
}

// --------------------------------------------------------------------------------------
// Hot-directory construction: one CTA counts the keys of a strided sample of the records in
// a shared-memory table, picks the count threshold that fills the directory, and installs the
// selected keys, most frequent classes first, into 2-slot buckets.  Which keys end up in the
// directory only affects speed, never results.
constexpr uint32_t SAMPLE_SLOTS = 16384;
constexpr uint32_t SAMPLE_PROBES = 8;

__global__ void __launch_bounds__(1024, 1) hot_build_kernel(HotBuildParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ull* skeys = reinterpret_cast<ull*>(smem_raw);
    uint32_t* scnt = reinterpret_cast<uint32_t*>(smem_raw + (size_t)SAMPLE_SLOTS * 8);
    __shared__ uint32_t hist[256];
    __shared__ uint32_t s_thr, s_inserted;
    for (uint32_t i = threadIdx.x; i < SAMPLE_SLOTS; i += blockDim.x) {
        skeys[i] = 0;
        scnt[i] = 0;
    }
    for (uint32_t i = threadIdx.x; i < p.hot_slots; i += blockDim.x) p.hot_keys[i] = 0;
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    if (threadIdx.x == 0) s_inserted = 0;
    __syncthreads();

    for (uint32_t j = threadIdx.x; j < p.n_sample; j += blockDim.x) {
        uint4 v = p.recs[(ull)j * p.stride];
        uint32_t phase = (v.y >> 16) & 0xFFu;
        if (v.x >= p.n_apps || phase >= p.n_phases) continue;
        ull key = pack_key(phase, v.y & 0xFFFFu, v.z);
        ull skey = ~key;
        uint32_t s = (uint32_t)(hash_key(key) >> 50);  // 14 bits
        for (uint32_t probe = 0; probe < SAMPLE_PROBES; ++probe) {
            ull k = skeys[s];
            if (k == 0) k = atomicCAS(&skeys[s], 0ull, skey), k = (k == 0) ? skey : k;
            if (k == skey) {
                atomicAdd(&scnt[s], 1u);
                break;
            }
            s = (s + 1) & (SAMPLE_SLOTS - 1);
        }
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < SAMPLE_SLOTS; i += blockDim.x)
        if (scnt[i] != 0) atomicAdd(&hist[min(scnt[i], 255u)], 1u);
    __syncthreads();
    if (threadIdx.x == 0) {
        // smallest threshold >= 2 whose class fits the directory with some over-subscription
        uint32_t budget = p.hot_slots + p.hot_slots / 4, cum = 0, thr = 256;
        for (int c = 255; c >= 2; --c) {
            if (cum + hist[c] > budget) break;
            cum += hist[c];
            thr = (uint32_t)c;
        }
        s_thr = thr;
    }
    __syncthreads();
    const uint32_t thr = s_thr;
    const uint32_t bounds[5] = {0xFFFFFFFFu, 128u, 32u, 8u, 2u};
    for (int round = 0; round < 4; ++round) {
        uint32_t hi = bounds[round], lo = max(bounds[round + 1], thr);
        if (lo < hi) {
            for (uint32_t i = threadIdx.x; i < SAMPLE_SLOTS; i += blockDim.x) {
                uint32_t c = scnt[i];
                if (c >= lo && c < hi) {
                    ull skey = skeys[i];
                    uint32_t b = dir_bucket(hash_key(~skey), p.hot_slots / 2) * 2;
                    if (atomicCAS(&p.hot_keys[b], 0ull, skey) == 0 || atomicCAS(&p.hot_keys[b + 1], 0ull, skey) == 0)
                        atomicAdd(&s_inserted, 1u);
                }
            }
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) p.ctl->hot_n = s_inserted;
}

// --------------------------------------------------------------------------------------
// Merge of already aggregated units into the table.
__global__ void __launch_bounds__(256) merge_kernel(const atrex_entry_t* in, ull n, TableRef t) {
    for (ull i = (ull)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (ull)gridDim.x * blockDim.x) {
        atrex_entry_t e = in[i];
        table_accumulate(t, e.key, hash_key(e.key), e.wt_lo, e.wt_hi, e.count);
    }
}

// --------------------------------------------------------------------------------------
// host launchers

size_t ingest_smem_bytes(bool hot, uint32_t hot_slots, uint32_t n_apps, bool appw_in_smem) {
    return (hot ? (size_t)hot_slots * 20 : 0) + (appw_in_smem ? (size_t)n_apps * 4 : 0);
}

cudaError_t ingest_prepare() {
    cudaError_t e = cudaFuncSetAttribute(ingest_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(ingest_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(hot_build_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SAMPLE_SLOTS * 12);
}

cudaError_t launch_ingest(const IngestParams& p, bool hot, int grid, cudaStream_t stream) {
    size_t smem = ingest_smem_bytes(hot, p.hot_slots, p.n_apps, p.appw_in_smem != 0);
    if (hot)
        ingest_kernel<true><<<grid, INGEST_THREADS, smem, stream>>>(p);
    else
        ingest_kernel<false><<<grid, INGEST_THREADS, smem, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_hot_build(const HotBuildParams& p, cudaStream_t stream) {
    hot_build_kernel<<<1, 1024, SAMPLE_SLOTS * 12, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_merge(const atrex_entry_t* in, ull n, const TableRef& t, int grid, cudaStream_t stream) {
    merge_kernel<<<grid, 256, 0, stream>>>(in, n, t);
    return cudaGetLastError();
}

}  // namespace atrex
