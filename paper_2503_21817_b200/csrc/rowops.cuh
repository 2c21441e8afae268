// Row-wise building blocks shared by the small token layers (summary token, token merge):
// one-warp-per-row dot products and fixed-order weighted row sums.  fp32 arithmetic throughout.
#pragma once
#include "common.cuh"

namespace skipffn {

constexpr int SM_THREADS = 256;

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

// out[i] = sum_c X[i, c] * v[seg(i)?, c]: one warp per row.  per_segment = 0: v is one vector (w);
// 1: v is [n_seg, C] and the row's segment is found by binary search in the offsets.
template <typename T, typename TV = T>
__global__ void __launch_bounds__(SM_THREADS)
k_row_dots(const T *__restrict__ X, const TV *__restrict__ v, const int32_t *__restrict__ off, int n_seg,
           int per_segment, float *__restrict__ out, int64_t n, int C)
{
    pdl_enter();
    const int64_t i = (int64_t)blockIdx.x * (SM_THREADS / 32) + (threadIdx.x >> 5);
    if (i >= n) return;
    const int lane = threadIdx.x & 31;
    const TV *vec = v;
    if (per_segment) {
        int lo = 0, hi = n_seg;            // largest s with off[s] <= i
        while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (off[mid] <= i) lo = mid; else hi = mid; }
        vec = v + (int64_t)lo * C;
    }
    const T *x = X + i * C;
    float acc = 0.0f;
    for (int c = 4 * lane; c < C; c += 128) {    // C is a multiple of 8
        float a[4], b[4];
        load4(x + c, a);
        load4(vec + c, b);
#pragma unroll
        for (int q = 0; q < 4; ++q) acc = fmaf(a[q], b[q], acc);
    }
    acc = warp_sum(acc);
    if (lane == 0) out[i] = acc;
}

// y[c] = sum over rows lo..hi-1 of coef[i] * X[i, c]; grid (column blocks of 64, parts); 4 row lanes
// per column, combined in lane order.  parts == n_seg with seg_mode (rows of segment blockIdx.y,
// output xs[seg]), else DG_CHUNKS equal chunks of all rows (output part[chunk]).
constexpr int SP_COLS = 64, SP_LANES = 8;

template <typename T, typename TO>
__global__ void __launch_bounds__(SP_COLS * SP_LANES)
k_weighted_rows(const T *__restrict__ X, const float *__restrict__ coef, const int32_t *__restrict__ off,
                int seg_mode, int64_t n, TO *__restrict__ out, int C)
{
    pdl_enter();
    __shared__ float red[SP_LANES][SP_COLS];
    int64_t lo, hi;
    if (seg_mode) { lo = off[blockIdx.y]; hi = off[blockIdx.y + 1]; }
    else { const int64_t per = (n + gridDim.y - 1) / gridDim.y; lo = blockIdx.y * per; hi = lo + per < n ? lo + per : n; }
    const int cl = threadIdx.x % SP_COLS, lane = threadIdx.x / SP_COLS;
    const int col = blockIdx.x * SP_COLS + cl;
    float acc = 0.0f;
    if (col < C) {
#pragma unroll 8
        for (int64_t i = lo + lane; i < hi; i += SP_LANES) acc = fmaf(coef[i], to_f32(X[i * C + col]), acc);
    }
    red[lane][cl] = acc;
    __syncthreads();
    if (lane == 0 && col < C) {
        float s = 0.0f;
#pragma unroll
        for (int l = 0; l < SP_LANES; ++l) s += red[l][cl];
        out[(int64_t)blockIdx.y * C + col] = from_f32<TO>(s);
    }
}

template <typename TO>
__global__ void k_sum_parts(const float *__restrict__ part, int parts, TO *__restrict__ out, int C)
{
    pdl_enter();
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    if (col >= C) return;
    float s = 0.0f;
    for (int k = 0; k < parts; ++k) s += part[(int64_t)k * C + col];
    out[col] = from_f32<TO>(s);
}

}  // namespace skipffn
