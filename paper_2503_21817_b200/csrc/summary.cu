// Adaptive summary token (paper section 4.2, Eq. 6):  x_s = softmax(X w^T)^T X  per segment of a
// packed X [n, C] (the retained or the skipped visual tokens of one sample), w [C].  A tiny layer
// run once per sample before the decoder; HBM / latency bound.  All sums are fp32 in a fixed order.
//   forward : scores (one warp per row) -> softmax per segment -> weighted row sum per column block
//   backward: a_i = dxs . X_i (warp per row) -> ds_i = p_i (a_i - sum_j p_j a_j) per segment
//             -> dX_i = p_i dxs + ds_i w (rows) and dw = sum_i ds_i X_i (two-stage column reduction)
#include "common.cuh"
#include "rowops.cuh"

namespace skipffn {

__device__ __forceinline__ float block_reduce(float v, float *red, bool is_max)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        const float o = __shfl_xor_sync(0xffffffffu, v, d);
        v = is_max ? fmaxf(v, o) : v + o;
    }
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < SM_THREADS / 32; ++w) r = is_max ? fmaxf(r, red[w]) : r + red[w];
    return r;
}

// probs[i] <- softmax of the scores in probs, per segment (one CTA per segment, in place)
__global__ void __launch_bounds__(SM_THREADS)
k_segment_softmax(float *__restrict__ probs, const int32_t *__restrict__ off)
{
    pdl_enter();
    __shared__ float red[SM_THREADS / 32];
    const int lo = off[blockIdx.x], hi = off[blockIdx.x + 1];
    float mx = -INFINITY;
    for (int i = lo + threadIdx.x; i < hi; i += SM_THREADS) mx = fmaxf(mx, probs[i]);
    mx = block_reduce(mx, red, true);
    float den = 0.0f;
    for (int i = lo + threadIdx.x; i < hi; i += SM_THREADS) den += expf(probs[i] - mx);
    den = block_reduce(den, red, false);
    for (int i = lo + threadIdx.x; i < hi; i += SM_THREADS) probs[i] = expf(probs[i] - mx) / den;
}

// a[i] <- ds_i = p_i (a_i - sum_j p_j a_j), per segment, in place
__global__ void __launch_bounds__(SM_THREADS)
k_segment_dscore(float *__restrict__ a, const float *__restrict__ probs, const int32_t *__restrict__ off)
{
    pdl_enter();
    __shared__ float red[SM_THREADS / 32];
    const int lo = off[blockIdx.x], hi = off[blockIdx.x + 1];
    float t = 0.0f;
    for (int i = lo + threadIdx.x; i < hi; i += SM_THREADS) t = fmaf(probs[i], a[i], t);
    t = block_reduce(t, red, false);
    for (int i = lo + threadIdx.x; i < hi; i += SM_THREADS) a[i] = probs[i] * (a[i] - t);
}

// dX[i, c] = p_i * dxs[seg(i), c] + ds_i * w[c]: one CTA per row
template <typename T>
__global__ void __launch_bounds__(SM_THREADS)
k_summary_dx(const T *__restrict__ dxs, const T *__restrict__ w, const float *__restrict__ probs,
             const float *__restrict__ ds, const int32_t *__restrict__ off, int n_seg, T *__restrict__ dX, int C)
{
    pdl_enter();
    const int64_t i = blockIdx.x;
    int lo = 0, hi = n_seg;
    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (off[mid] <= i) lo = mid; else hi = mid; }
    const T *g = dxs + (int64_t)lo * C;
    const float p = probs[i], d = ds[i];
    for (int c = threadIdx.x; c < C; c += SM_THREADS)
        dX[i * C + c] = from_f32<T>(fmaf(p, to_f32(g[c]), d * to_f32(w[c])));
}

template <typename T>
static cudaError_t fwd_t(const T *X, const int32_t *off, int n_seg, int64_t n, int C, const T *w, T *xs,
                         float *probs, cudaStream_t s)
{
    if (n > 0) {
        launch_pdl(k_row_dots<T>, dim3((unsigned)((n + 7) / 8)), dim3(SM_THREADS), s, X, w, off, n_seg, 0, probs, n, C);
        launch_pdl(k_segment_softmax, dim3(n_seg), dim3(SM_THREADS), s, probs, off);
    }
    dim3 grid((C + SP_COLS - 1) / SP_COLS, n_seg);     // empty segments write zeros
    launch_pdl(k_weighted_rows<T, T>, dim3(grid), dim3(SP_COLS * SP_LANES), s, X, probs, off, 1, n, xs, C);
    return cudaGetLastError();
}

template <typename T>
static cudaError_t bwd_t(const T *X, const int32_t *off, int n_seg, int64_t n, int C, const T *w,
                         const float *probs, const T *dxs, T *dX, void *dw, int dw_fp32, float *scratch,
                         cudaStream_t s)
{
    float *ds = scratch, *part = scratch + ((n + 63) / 64) * 64;
    if (n > 0) {
        launch_pdl(k_row_dots<T>, dim3((unsigned)((n + 7) / 8)), dim3(SM_THREADS), s, X, dxs, off, n_seg, 1, ds, n, C);
        launch_pdl(k_segment_dscore, dim3(n_seg), dim3(SM_THREADS), s, ds, probs, off);
        if (dX) launch_pdl(k_summary_dx<T>, dim3((unsigned)n), dim3(SM_THREADS), s, dxs, w, probs, ds, off, n_seg, dX, C);
    }
    if (dw) {
        dim3 grid((C + SP_COLS - 1) / SP_COLS, DG_CHUNKS);
        launch_pdl(k_weighted_rows<T, float>, dim3(grid), dim3(SP_COLS * SP_LANES), s, X, ds, off, 0, n, part, C);
        if (dw_fp32) launch_pdl(k_sum_parts<float>, dim3((C + 255) / 256), dim3(256), s, part, DG_CHUNKS, (float *)dw, C);
        else launch_pdl(k_sum_parts<T>, dim3((C + 255) / 256), dim3(256), s, part, DG_CHUNKS, (T *)dw, C);
    }
    return cudaGetLastError();
}

cudaError_t launch_summary_forward(const void *X, const int32_t *off, int n_seg, int64_t n, int C, int dtype,
                                   const void *w, void *xs, float *probs, cudaStream_t s)
{
    if (n_seg <= 0) return cudaSuccess;
    return dtype == SKIPFFN_BF16
               ? fwd_t<bf16>((const bf16 *)X, off, n_seg, n, C, (const bf16 *)w, (bf16 *)xs, probs, s)
               : fwd_t<float>((const float *)X, off, n_seg, n, C, (const float *)w, (float *)xs, probs, s);
}

cudaError_t launch_summary_backward(const void *X, const int32_t *off, int n_seg, int64_t n, int C, int dtype,
                                    const void *w, const float *probs, const void *dxs, void *dX, void *dw,
                                    int dw_fp32, float *scratch, cudaStream_t s)
{
    if (n_seg <= 0) return cudaSuccess;
    return dtype == SKIPFFN_BF16
               ? bwd_t<bf16>((const bf16 *)X, off, n_seg, n, C, (const bf16 *)w, probs, (const bf16 *)dxs,
                             (bf16 *)dX, dw, dw_fp32, scratch, s)
               : bwd_t<float>((const float *)X, off, n_seg, n, C, (const float *)w, probs, (const float *)dxs,
                              (float *)dX, dw, 1, scratch, s);
}

}  // namespace skipffn
