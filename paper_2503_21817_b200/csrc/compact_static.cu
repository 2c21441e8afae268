// skipffn_compact_static: the kept-row index list for callers that cannot allocate device memory.
//
// The regular route (skipffn_plan on a handle) keeps the compaction kernel's scratch -- the
// token -> rank map and the status block holding the kept count -- in a workspace the caller
// allocates.  Some callers cannot do that: a serving process whose framework has already handed
// the whole HBM to its own pool (a further cudaMalloc fails), a latency-critical loop that cannot
// afford cudaMalloc's implicit device-wide synchronisation, or a plug-in host that forbids
// allocation calls from extension code.  For them the same kernel runs with its scratch in a
// fixed array that is part of the library image: every device that loads the library holds
// SCRATCH_WORDS * 4 bytes (about 256 KiB) until the process exits, and problems larger than
// SKIPFFN_STATIC_MAX_TOKENS tokens are refused.
//
// The array is shared by every call on a device and keeps the previous call's contents.  The
// kernel overwrites every word it later reads (the kept count, and the rank of each token below
// N), so nothing has to be cleared between calls; two calls that overlap on the GPU (different
// streams, or different host threads) race on it and must be serialised by the caller.
#include <mutex>

#include "common.cuh"

namespace skipffn {

constexpr int SCRATCH_WORDS = ST_WORDS + SKIPFFN_STATIC_MAX_TOKENS;   // status block, then pos[]
static __device__ __align__(256) int32_t g_compact_scratch[SCRATCH_WORDS];

constexpr int MAX_DEVICES = 64;
static int32_t *g_scratch_addr[MAX_DEVICES];   // device address of the array, per device
static std::mutex g_scratch_mutex;

// In host code `g_compact_scratch` names a host-side shadow of the symbol, not device memory, so
// the device address has to be asked for, with the target device current.  Done once per device.
static cudaError_t scratch_address(int32_t **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_compact_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = (int32_t *)p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace skipffn

using namespace skipffn;

extern "C" skipffn_status skipffn_compact_static(const uint8_t *skip_mask, int64_t N, int32_t *idx,
                                                 int32_t *nk, void *stream)
{
    if (N < 0 || !nk || (N > 0 && (!skip_mask || !idx))) return SKIPFFN_EINVAL;
    if (N > SKIPFFN_STATIC_MAX_TOKENS) return SKIPFFN_EUNSUPPORTED;   // beyond the fixed scratch
    cudaStream_t st = (cudaStream_t)stream;
    if (N == 0) return cudaMemsetAsync(nk, 0, sizeof(int32_t), st) == cudaSuccess ? SKIPFFN_OK : SKIPFFN_ECUDA;
    int32_t *scratch = nullptr;
    if (scratch_address(&scratch) != cudaSuccess) return SKIPFFN_ECUDA;
    int32_t *status = scratch, *pos = scratch + ST_WORDS;
    // cap = N: the kernel's padding entries past the kept count stay inside idx[0 .. N-1]
    if (launch_compact(skip_mask, N, 0, idx, pos, status, N, N, st) != cudaSuccess) return SKIPFFN_ECUDA;
    if (cudaMemcpyAsync(nk, status + ST_NK, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return SKIPFFN_ECUDA;
    return SKIPFFN_OK;
}
