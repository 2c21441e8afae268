// Adaptive summary token (paper section 4.2, Eq. 6):  x_s = softmax(X w^T)^T X  per segment of a
// packed X [n, C] (the retained or the skipped visual tokens of one sample), w [C].  A tiny layer
// run once per sample before the decoder; HBM / latency bound.  All sums are fp32 in a fixed order.
// One thread-block cluster of 16 (or 8) CTAs works on one segment, each CTA on its share of the rows; what
// the softmax and the weighted sum need from the whole segment (maximum, denominator, partial
// column sums) is exchanged through the cluster's distributed shared memory, so that
//   forward  is ONE launch: scores (one warp per row) -> softmax -> weighted row sum (second read
//            of the rows, from L2), and
//   backward is one launch for a_i = dxs . X_i, ds_i = p_i (a_i - sum_j p_j a_j) and
//            dX_i = p_i dxs + ds_i w, followed by the two-stage column reduction dw = sum_i ds_i X_i.
#include <cooperative_groups.h>

#include "common.cuh"
#include "rowops.cuh"

namespace skipffn {

namespace cg = cooperative_groups;

constexpr int SC_THREADS = 512;
constexpr int SC_MAX_DEVICES = 64;
constexpr int SC_CLUSTER_MAX = 16;     // CTAs per cluster: 16 where the device schedules such clusters, else 8
constexpr int SC_PASS_COLS = 8192;     // columns whose partial sums one CTA holds at a time (32 KiB)

// sum or maximum over the CTA in a fixed order (valid in every thread)
__device__ __forceinline__ float cta_reduce(float v, float *red, bool is_max)
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
    for (int w = 1; w < SC_THREADS / 32; ++w) r = is_max ? fmaxf(r, red[w]) : r + red[w];
    return r;
}

// this CTA's share of segment [lo, hi): rows in order, an equal count per CTA of the cluster
__device__ __forceinline__ void cluster_rows(int lo, int hi, int rank, int nb, int &r0, int &r1)
{
    const int per = (hi - lo + nb - 1) / nb;
    r0 = min(lo + rank * per, hi);
    r1 = min(r0 + per, hi);
}

template <typename T> struct Vec16 { static constexpr int N = 16 / sizeof(T); };
__device__ __forceinline__ void load_vec(const float *p, float (&v)[4]) { load4(p, v); }
__device__ __forceinline__ void load_vec(const bf16 *p, float (&v)[8])
{
    const uint4 q = *reinterpret_cast<const uint4 *>(p);
    const uint32_t u[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        v[2 * k] = __uint_as_float(u[k] << 16);
        v[2 * k + 1] = __uint_as_float(u[k] & 0xffff0000u);
    }
}
__device__ __forceinline__ void store_vec(float *p, const float (&v)[4])
{
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store_vec(bf16 *p, const float (&v)[8])
{
    uint32_t u[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
        u[k] = *reinterpret_cast<const uint32_t *>(&h);
    }
    *reinterpret_cast<uint4 *>(p) = make_uint4(u[0], u[1], u[2], u[3]);
}

// dot product of two rows of C elements by one warp (the result in every lane)
template <typename T, int VN = Vec16<T>::N>
__device__ __forceinline__ float warp_row_dot(const T *x, const T *v, int C, int lane)
{
    float acc = 0.0f;
#pragma unroll 8
    for (int c = VN * lane; c < C; c += 32 * VN) {
        float a[VN], b[VN];
        load_vec(x + c, a);
        load_vec(v + c, b);
#pragma unroll
        for (int q = 0; q < VN; ++q) acc = fmaf(a[q], b[q], acc);
    }
    return warp_sum(acc);
}

// Forward of one segment per cluster: probs (saved for the backward) and xs[seg].
template <typename T>
__global__ void __launch_bounds__(SC_THREADS)
k_summary_fwd(const T *__restrict__ X, const T *__restrict__ w, const int32_t *__restrict__ off,
              float *__restrict__ probs, T *__restrict__ xs, int C)
{
    constexpr int VN = Vec16<T>::N;
    __shared__ __align__(16) float part[SC_PASS_COLS];
    __shared__ float red[SC_THREADS / 32];
    __shared__ float slot[2];
    cg::cluster_group cl = cg::this_cluster();
    const int rank = (int)cl.block_rank(), nb = (int)cl.num_blocks(), seg = blockIdx.x / nb;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_enter();
    int r0, r1;
    cluster_rows(off[seg], off[seg + 1], rank, nb, r0, r1);
    // ---- scores of this CTA's rows, their maximum over the segment
    float mx = -INFINITY;
    for (int i = r0 + warp; i < r1; i += SC_THREADS / 32) {
        const float sc = warp_row_dot(X + (int64_t)i * C, w, C, lane);
        if (lane == 0) probs[i] = sc;
        mx = fmaxf(mx, sc);
    }
    mx = cta_reduce(mx, red, true);
    if (tid == 0) slot[0] = mx;
    cl.sync();
    float gmx = -INFINITY;
    for (int k = 0; k < nb; ++k) gmx = fmaxf(gmx, *cl.map_shared_rank(&slot[0], k));
    // ---- denominator: ranks in order
    float den = 0.0f;
    for (int i = r0 + tid; i < r1; i += SC_THREADS) den += expf(probs[i] - gmx);
    den = cta_reduce(den, red, false);
    if (tid == 0) slot[1] = den;
    cl.sync();
    den = 0.0f;
    for (int k = 0; k < nb; ++k) den += *cl.map_shared_rank(&slot[1], k);
    for (int i = r0 + tid; i < r1; i += SC_THREADS) probs[i] = expf(probs[i] - gmx) / den;
    __syncthreads();
    // ---- weighted sum: this CTA's rows into `part`, then rank r adds the eight parts of its columns
    for (int cb = 0; cb < C; cb += SC_PASS_COLS) {
        const int cw = min(SC_PASS_COLS, C - cb);
        for (int c = VN * tid; c < cw; c += VN * SC_THREADS) {
            float acc[VN];
#pragma unroll
            for (int q = 0; q < VN; ++q) acc[q] = 0.0f;
#pragma unroll 8
            for (int i = r0; i < r1; ++i) {
                float x[VN];
                load_vec(X + (int64_t)i * C + cb + c, x);
                const float p = probs[i];
#pragma unroll
                for (int q = 0; q < VN; ++q) acc[q] = fmaf(p, x[q], acc[q]);
            }
#pragma unroll
            for (int q = 0; q < VN; ++q) part[c + q] = acc[q];
        }
        cl.sync();
        const int per = (cw + nb - 1) / nb;
        for (int c = rank * per + tid; c < min(cw, (rank + 1) * per); c += SC_THREADS) {
            float sum = 0.0f;
            for (int k = 0; k < nb; ++k) sum += cl.map_shared_rank(part, k)[c];
            xs[(int64_t)seg * C + cb + c] = from_f32<T>(sum);
        }
        cl.sync();     // nobody overwrites (or leaves with) a part that is still being read
    }
}

// Backward of one segment per cluster: ds (kept for the dw reduction) and dX.
template <typename T>
__global__ void __launch_bounds__(SC_THREADS)
k_summary_bwd(const T *__restrict__ X, const T *__restrict__ w, const int32_t *__restrict__ off,
              const float *__restrict__ probs, const T *__restrict__ dxs, float *__restrict__ ds,
              T *__restrict__ dX, int C)
{
    constexpr int VN = Vec16<T>::N;
    __shared__ float red[SC_THREADS / 32];
    __shared__ float slot;
    cg::cluster_group cl = cg::this_cluster();
    const int rank = (int)cl.block_rank(), nb = (int)cl.num_blocks(), seg = blockIdx.x / nb;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_enter();
    int r0, r1;
    cluster_rows(off[seg], off[seg + 1], rank, nb, r0, r1);
    const T *g = dxs + (int64_t)seg * C;
    // ---- a_i = dxs . X_i, t = sum_j p_j a_j over the segment (rows in order inside a warp, warps and
    // ranks in order)
    float t = 0.0f;
    for (int i = r0 + warp; i < r1; i += SC_THREADS / 32) {
        const float a = warp_row_dot(X + (int64_t)i * C, g, C, lane);
        if (lane == 0) { ds[i] = a; t = fmaf(probs[i], a, t); }
    }
    t = cta_reduce(t, red, false);
    if (tid == 0) slot = t;
    cl.sync();
    t = 0.0f;
    for (int k = 0; k < nb; ++k) t += *cl.map_shared_rank(&slot, k);
    for (int i = r0 + tid; i < r1; i += SC_THREADS) ds[i] = probs[i] * (ds[i] - t);
    __syncthreads();
    // ---- dX_i = p_i dxs + ds_i w
    if (dX != nullptr) {
        for (int c = VN * tid; c < C; c += VN * SC_THREADS) {
            float gv[VN], wv[VN];
            load_vec(g + c, gv);
            load_vec(w + c, wv);
            for (int i = r0; i < r1; ++i) {
                const float p = probs[i], d = ds[i];
                float o[VN];
#pragma unroll
                for (int q = 0; q < VN; ++q) o[q] = fmaf(p, gv[q], d * wv[q]);
                store_vec(dX + (int64_t)i * C + c, o);
            }
        }
    }
    cl.sync();         // a CTA's `slot` is read by the others until here
}

// Clusters of 16 CTAs need the non-portable-size attribute and a device that can place them;
// decided once per kernel, clusters of 8 otherwise.
template <typename... KArgs>
static int cluster_size_for(void (*kernel)(KArgs...))
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(SC_CLUSTER_MAX); cfg.blockDim = dim3(SC_THREADS);
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = SC_CLUSTER_MAX; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    int n = 0;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
        cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) == cudaSuccess && n >= 1)
        return SC_CLUSTER_MAX;
    (void)cudaGetLastError();
    return 8;
}

template <typename... KArgs, typename... Args>
static cudaError_t launch_cluster(void (*kernel)(KArgs...), int n_seg, cudaStream_t s, Args... args)
{
    static int size_by_dev[SC_MAX_DEVICES];        // per kernel instantiation and device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= SC_MAX_DEVICES) return cudaErrorInvalidDevice;
    if (size_by_dev[dev] == 0) size_by_dev[dev] = cluster_size_for(kernel);
    const int nb = size_by_dev[dev];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_seg * nb); cfg.blockDim = dim3(SC_THREADS); cfg.dynamicSmemBytes = 0; cfg.stream = s;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = nb; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

template <typename T>
static cudaError_t fwd_t(const T *X, const int32_t *off, int n_seg, int64_t n, int C, const T *w, T *xs,
                         float *probs, cudaStream_t s)
{
    (void)n;     // empty segments write zeros
    return launch_cluster(k_summary_fwd<T>, n_seg, s, X, w, off, probs, xs, C);
}

template <typename T>
static cudaError_t bwd_t(const T *X, const int32_t *off, int n_seg, int64_t n, int C, const T *w,
                         const float *probs, const T *dxs, T *dX, void *dw, int dw_fp32, float *scratch,
                         cudaStream_t s)
{
    float *ds = scratch, *part = scratch + ((n + 63) / 64) * 64;
    if (n > 0) {
        cudaError_t e = launch_cluster(k_summary_bwd<T>, n_seg, s, X, w, off, probs, dxs, ds, dX, C);
        if (e != cudaSuccess) return e;
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
