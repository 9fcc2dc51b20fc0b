// Ranked top-k over an array of aggregated entries, with all scratch memory in a fixed
// device array that is part of the library image.
//
// Some users of this library run where device allocation is off the table: inside a service
// whose memory budget was carved up at start-up, in a plugin that is handed buffers but no
// allocator, or in a process whose CUDA memory pool is owned by someone else.  The regular
// ranking call works out of the handle's workspace, which somebody had to allocate.  This
// entry point needs no handle and no workspace: the caller passes the entries and an output
// buffer, and the selection buffer lives in `g_scratch` below, which every GPU that loads the
// library keeps resident until the process exits (2 MiB + 256 bytes).
#include <mutex>

#include "kernels.h"

using namespace atrex;

namespace {

constexpr uint32_t MAX_ENTRIES = ATREX_STATIC_TOPK_MAX_ENTRIES;  // power of two
constexpr size_t SEL_BYTES = (size_t)MAX_ENTRIES * 32;            // {composite words 2,1,0, entry index}
constexpr size_t SCRATCH_BYTES = SEL_BYTES + 256;                 // + the candidate counter
constexpr int MAX_DEVICES = 64;

// Device code may name this array directly.  On the host the name is only a stand-in for the
// symbol, not a device address: handing it to a kernel would make the kernel read host memory
// or fault, so the host asks the runtime for the real address once per device (below).
static __device__ __align__(256) unsigned char g_scratch[SCRATCH_BYTES];

std::mutex g_lock;
unsigned char* g_scratch_addr[MAX_DEVICES];  // per device, filled on that device's first call

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    bool ok = true;   // false: `dev` could not be made current, nothing may run
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) {
            switched = cudaSetDevice(dev) == cudaSuccess;
            ok = switched;
        }
    }
    ~DeviceGuard() {
        if (switched && prev >= 0) cudaSetDevice(prev);
    }
};

// Entries of `phase` become {ranking composite, index} items in the selection buffer.
__global__ void __launch_bounds__(256) static_collect_kernel(const atrex_entry_t* entries, uint32_t n, uint32_t phase,
                                                             ull* sel, ull* counter) {
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const ull key = entries[i].key;
        if ((uint32_t)(key >> 48) != phase) continue;
        const ull lo = entries[i].wt_lo, hi = entries[i].wt_hi;
        ull pos = atomicAdd(counter, 1ull);
        ull* dst = sel + pos * 4;
        // larger composite = better: 88-bit weighted time above the complemented 56-bit key
        dst[0] = hi >> 8;
        dst[1] = (lo >> 8) | (hi << 56);
        dst[2] = ((~key) & 0x00FFFFFFFFFFFFFFull) | (lo << 56);
        dst[3] = i;
    }
}

__global__ void __launch_bounds__(256) static_emit_kernel(const atrex_entry_t* entries, const ull* sel, uint32_t m,
                                                          atrex_entry_t* out) {
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < m; i += gridDim.x * blockDim.x)
        out[i] = entries[sel[(ull)i * 4 + 3]];
}

}  // namespace

extern "C" int atrex_topk_entries_static(const atrex_entry_t* d_entries, uint64_t n, uint32_t phase, uint32_t k,
                                         atrex_entry_t* d_out, uint32_t* h_n_out, void* stream) {
    if (!h_n_out) return ATREX_ERR_INVALID;
    *h_n_out = 0;
    if (n > MAX_ENTRIES || k > MAX_ENTRIES) return ATREX_ERR_TOO_LARGE;  // beyond the fixed scratch
    if ((n && !d_entries) || (k && !d_out) || phase >= ATREX_MAX_PHASES) return ATREX_ERR_INVALID;
    if (((uintptr_t)d_entries & 7u) || ((uintptr_t)d_out & 7u)) return ATREX_ERR_INVALID;
    if (n == 0 || k == 0) return ATREX_OK;

    // the entries live on some device: run there
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, d_entries) != cudaSuccess || attr.type != cudaMemoryTypeDevice) {
        cudaGetLastError();
        return ATREX_ERR_INVALID;
    }
    const int dev = attr.device;
    if (dev < 0 || dev >= MAX_DEVICES) return ATREX_ERR_INVALID;
    DeviceGuard guard(dev);
    if (!guard.ok) {   // resolving the array's address with another device current would cache a wrong address
        cudaGetLastError();
        return ATREX_ERR_CUDA;
    }
    cudaStream_t s = (cudaStream_t)stream;

    unsigned char* scratch;
    {
        // set-up, once per device, with that device current: resolve the array's device address
        std::lock_guard<std::mutex> hold(g_lock);
        if (g_scratch_addr[dev] == nullptr) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || p == nullptr) {
                cudaGetLastError();
                return ATREX_ERR_CUDA;
            }
            g_scratch_addr[dev] = (unsigned char*)p;
        }
        scratch = g_scratch_addr[dev];
    }
    ull* sel = (ull*)scratch;
    ull* counter = (ull*)(scratch + SEL_BYTES);

    // the array keeps whatever the previous call left: clear the counter and the selection
    // buffer (the sorter relies on all-zero padding behind the candidates)
    if (cudaMemsetAsync(scratch, 0, SCRATCH_BYTES, s) != cudaSuccess) return ATREX_ERR_CUDA;
    int grid = (int)((n + 255) / 256);
    if (grid > 1024) grid = 1024;
    static_collect_kernel<<<grid, 256, 0, s>>>(d_entries, (uint32_t)n, phase, sel, counter);
    if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
    ull count = 0;
    if (cudaMemcpyAsync(&count, counter, sizeof(count), cudaMemcpyDeviceToHost, s) != cudaSuccess) return ATREX_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return ATREX_ERR_CUDA;
    if (count == 0) return ATREX_OK;
    uint32_t n_pow2 = 2;
    while (n_pow2 < count) n_pow2 <<= 1;
    if (launch_topk_sort(sel, n_pow2, s) != cudaSuccess) return ATREX_ERR_CUDA;
    const uint32_t m = (uint32_t)(count < k ? count : k);
    static_emit_kernel<<<(m + 255) / 256, 256, 0, s>>>(d_entries, sel, m, d_out);
    if (cudaGetLastError() != cudaSuccess) return ATREX_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return ATREX_ERR_CUDA;
    *h_n_out = m;
    return ATREX_OK;
}
