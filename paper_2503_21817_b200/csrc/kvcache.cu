// Skip KV-cache (Eq. 7): after prefill the keys / values of the skipped tokens are dropped from
// the cache, K' = K \ K_skip, V' = V \ V_skip.  With the ascending kept-row list this is a row
// gather, byte for byte; HBM-bound.
#include "common.cuh"

namespace skipffn {

// src: [planes, N, row_vecs] uint4;  dst: [planes, dst_rows, row_vecs].  Row r < Nk of every plane
// receives row idx[r].  blockIdx.x = r, blockIdx.y = a group of KV_PLANES planes: one CTA moves
// KV_PLANES rows (16 KiB at the 8B cache shape), four 16-byte loads in flight per thread.
constexpr int KV_THREADS = 256;
constexpr int KV_PLANES = 8;

__global__ void __launch_bounds__(KV_THREADS)
k_kv_compact(const uint4 *__restrict__ src, uint4 *__restrict__ dst, const int32_t *__restrict__ idx,
             const int32_t *__restrict__ status, int64_t planes, int64_t N, int64_t dst_rows,
             int row_vecs)
{
    const int nk = status[ST_NK];
    const int64_t r = blockIdx.x;
    if (r >= nk || r >= dst_rows) return;
    const int64_t t = idx[r];
    for (int64_t p0 = (int64_t)blockIdx.y * KV_PLANES; p0 < planes; p0 += (int64_t)gridDim.y * KV_PLANES) {
        const int np = (int)(planes - p0 < KV_PLANES ? planes - p0 : KV_PLANES);
        const int total = np * row_vecs;
        for (int i0 = threadIdx.x; i0 < total; i0 += 4 * KV_THREADS) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * KV_THREADS;
                if (i < total) {
                    const int p = i / row_vecs, c = i - p * row_vecs;
                    v[u] = __ldcs(src + ((p0 + p) * N + t) * row_vecs + c);     // read once: streaming
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * KV_THREADS;
                if (i < total) {
                    const int p = i / row_vecs, c = i - p * row_vecs;
                    dst[((p0 + p) * dst_rows + r) * row_vecs + c] = v[u];
                }
            }
        }
    }
}

// new_cu[s] = number of kept tokens before token cu[s] (lower bound of cu[s] in the ascending list)
__global__ void k_kept_cu_seqlens(const int32_t *__restrict__ cu, int32_t *__restrict__ new_cu, int n,
                                  const int32_t *__restrict__ idx, const int32_t *__restrict__ status)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n) return;
    const int nk = status[ST_NK], target = cu[s];
    int lo = 0, hi = nk;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (idx[mid] < target) lo = mid + 1; else hi = mid;
    }
    new_cu[s] = lo;
}

cudaError_t launch_kv_compact(const void *src, void *dst, const int32_t *idx, const int32_t *status,
                              int64_t planes, int64_t N, int64_t dst_rows, int64_t row_bytes,
                              cudaStream_t s)
{
    if (planes <= 0 || N <= 0 || dst_rows <= 0) return cudaSuccess;
    const int64_t rows = N < dst_rows ? N : dst_rows;
    const int64_t groups = (planes + KV_PLANES - 1) / KV_PLANES;
    dim3 grid((unsigned)rows, (unsigned)(groups < 65535 ? groups : 65535));
    k_kv_compact<<<grid, KV_THREADS, 0, s>>>((const uint4 *)src, (uint4 *)dst, idx, status, planes, N,
                                             dst_rows, (int)(row_bytes / 16));
    return cudaGetLastError();
}

cudaError_t launch_kept_cu_seqlens(const int32_t *cu, int32_t *new_cu, int n, const int32_t *idx,
                                   const int32_t *status, cudaStream_t s)
{
    if (n <= 0) return cudaSuccess;
    k_kept_cu_seqlens<<<(n + 127) / 128, 128, 0, s>>>(cu, new_cu, n, idx, status);
    return cudaGetLastError();
}

}  // namespace skipffn
