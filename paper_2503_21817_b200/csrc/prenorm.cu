// Pre-norm variant of the Skip-FFN sublayer: out = x + FFN(RMSNorm(x) * gamma) on retained tokens.
// The paper's Eq. 4 writes FFN(h_attn); the decoder blocks of its LLaMA-3 / Vicuna backbones
// normalise the FFN input first, and skipping the FFN skips that normalisation too.
//   forward : rstd = rsqrt(mean_c x^2 + eps);  xn = x * rstd * gamma   (kept rows only)
//   backward: with xh = x * rstd and dy the gradient w.r.t. xn,
//             dgamma = sum_rows dy * xh;  dx = dout + rstd * (gamma * dy - xh * mean_c(gamma * dy * xh))
// All reductions run in fp32 in a fixed order (no atomics).
#include "common.cuh"

namespace skipffn {

constexpr int PN_THREADS = 128;

__device__ __forceinline__ float block_sum(float v, float *red)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();                       // red may still be read from a previous call
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float s = 0.0f;
#pragma unroll
    for (int w = 0; w < PN_THREADS / 32; ++w) s += red[w];
    return s;
}

// Row routing with the normalisation fused in.  Unit u < N is token u: a kept token's row goes,
// raw, to Xk[pos[u]] (the residual stash) and, normalised, to Xn[pos[u]]; a skipped token's row is
// copied to dst_identity[u].  Units u >= N zero the padding rows of Xk and Xn.
template <typename T>
__global__ void __launch_bounds__(PN_THREADS)
k_route_norm(const T *__restrict__ src, T *__restrict__ Xk, T *__restrict__ Xn, T *__restrict__ dst_identity,
             float *__restrict__ rstd_out, const T *__restrict__ gamma, float eps,
             const int32_t *__restrict__ pos, const int32_t *__restrict__ status, int64_t N, int C,
             int copy_identity)
{
    __shared__ float red[PN_THREADS / 32];
    const int64_t u = blockIdx.x;
    if (u >= N) {
        const int nk = status[ST_NK];
        const int64_t r = nk + (u - N);
        const int64_t end = ((int64_t)nk + ROW_PAD - 1) / ROW_PAD * ROW_PAD;
        if (r >= end) return;
        const float z[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        for (int c = 4 * threadIdx.x; c < C; c += 4 * PN_THREADS) {
            store4(Xk + r * C + c, z);
            store4(Xn + r * C + c, z);
        }
        return;
    }
    const int p = pos[u];
    const T *s = src + u * C;
    if (p < 0) {
        if (copy_identity) {
            const uint4 *sv = reinterpret_cast<const uint4 *>(s);
            uint4 *dv = reinterpret_cast<uint4 *>(dst_identity + u * C);
            const int vecs = C * (int)sizeof(T) / 16;
            for (int v = threadIdx.x; v < vecs; v += PN_THREADS) dv[v] = sv[v];
        }
        return;
    }
    float ss = 0.0f;
    for (int c = 4 * threadIdx.x; c < C; c += 4 * PN_THREADS) {
        float v[4];
        load4(s + c, v);
#pragma unroll
        for (int q = 0; q < 4; ++q) ss = fmaf(v[q], v[q], ss);
    }
    ss = block_sum(ss, red);
    const float rstd = rsqrtf(ss / (float)C + eps);
    if (threadIdx.x == 0) rstd_out[p] = rstd;
    T *dk = Xk + (int64_t)p * C, *dn = Xn + (int64_t)p * C;
    for (int c = 4 * threadIdx.x; c < C; c += 4 * PN_THREADS) {
        float v[4], g[4], n[4];
        load4(s + c, v);
        load4(gamma + c, g);
#pragma unroll
        for (int q = 0; q < 4; ++q) n[q] = v[q] * rstd * g[q];
        store4(dk + c, v);      // exact: the values came from T
        store4(dn + c, n);
    }
}

// dx[idx[r]] for kept row r from the fp32 gradient dy[r] w.r.t. the normalised input.
template <typename T>
__global__ void __launch_bounds__(PN_THREADS)
k_norm_bwd_rows(const float *__restrict__ dY, const T *__restrict__ Xk, const T *__restrict__ dOk,
                const float *__restrict__ rstd_in, const T *__restrict__ gamma, T *__restrict__ dx,
                const int32_t *__restrict__ idx, const int32_t *__restrict__ status, int C)
{
    __shared__ float red[PN_THREADS / 32];
    const int64_t r = blockIdx.x;
    if (r >= status[ST_NK]) return;
    const float rstd = rstd_in[r];
    const float *dy = dY + r * C;
    const T *x = Xk + r * C, *dout = dOk + r * C;
    float m = 0.0f;
    for (int c = 4 * threadIdx.x; c < C; c += 4 * PN_THREADS) {
        float g[4], y[4], xv[4];
        load4(gamma + c, g); load4(dy + c, y); load4(x + c, xv);
#pragma unroll
        for (int q = 0; q < 4; ++q) m = fmaf(g[q] * y[q], xv[q] * rstd, m);
    }
    m = block_sum(m, red) / (float)C;
    T *d = dx + (int64_t)idx[r] * C;
    for (int c = 4 * threadIdx.x; c < C; c += 4 * PN_THREADS) {
        float g[4], y[4], xv[4], o[4], res[4];
        load4(gamma + c, g); load4(dy + c, y); load4(x + c, xv); load4(dout + c, o);
#pragma unroll
        for (int q = 0; q < 4; ++q) res[q] = o[q] + rstd * (g[q] * y[q] - xv[q] * rstd * m);
        store4(d + c, res);
    }
}

// dgamma[c] = sum over kept rows of dy[r, c] * x[r, c] * rstd[r], in two stages with a fixed order:
// the kept rows are cut into DG_CHUNKS equal chunks; CTA (column block, chunk) sums its rows with
// eight row lanes (combined in lane order) into part[chunk][c]; the second stage adds the chunks
// in chunk order, then accumulates / converts.
constexpr int DG_COLS = 32, DG_LANES = 8;

template <typename T>
__global__ void __launch_bounds__(DG_COLS * DG_LANES)
k_dgamma_partial(const float *__restrict__ dY, const T *__restrict__ Xk, const float *__restrict__ rstd_in,
                 float *__restrict__ part, const int32_t *__restrict__ status, int C)
{
    __shared__ float red[DG_LANES][DG_COLS];
    const int nk = status[ST_NK];
    const int per = (nk + DG_CHUNKS - 1) / DG_CHUNKS;
    const int r0 = blockIdx.y * per, r1 = min(nk, r0 + per);
    const int cl = threadIdx.x % DG_COLS, lane = threadIdx.x / DG_COLS;
    const int col = blockIdx.x * DG_COLS + cl;
    float acc = 0.0f;
    if (col < C)
        for (int r = r0 + lane; r < r1; r += DG_LANES)
            acc = fmaf(dY[(int64_t)r * C + col], to_f32(Xk[(int64_t)r * C + col]) * rstd_in[r], acc);
    red[lane][cl] = acc;
    __syncthreads();
    if (lane == 0 && col < C) {
        float s = 0.0f;
#pragma unroll
        for (int l = 0; l < DG_LANES; ++l) s += red[l][cl];
        part[(int64_t)blockIdx.y * C + col] = s;
    }
}

template <typename TO>
__global__ void k_dgamma_final(const float *__restrict__ part, TO *__restrict__ dgamma, int C, int accumulate)
{
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    if (col >= C) return;
    float s = 0.0f;
#pragma unroll 8
    for (int k = 0; k < DG_CHUNKS; ++k) s += part[(int64_t)k * C + col];
    if (accumulate) s += to_f32(dgamma[col]);
    dgamma[col] = from_f32<TO>(s);
}

cudaError_t launch_route_norm(const RouteArgs &a, void *Xn, float *rstd, const void *gamma, float eps,
                              cudaStream_t s)
{
    const int copy_identity = a.dst_identity != nullptr && a.dst_identity != a.src;
    const unsigned grid = (unsigned)(a.N + ROW_PAD);
    if (a.elem_bytes == 2)
        k_route_norm<bf16><<<grid, PN_THREADS, 0, s>>>((const bf16 *)a.src, (bf16 *)a.dst_compact, (bf16 *)Xn,
                                                      (bf16 *)a.dst_identity, rstd, (const bf16 *)gamma, eps,
                                                      a.pos, a.status, a.N, a.C, copy_identity);
    else
        k_route_norm<float><<<grid, PN_THREADS, 0, s>>>((const float *)a.src, (float *)a.dst_compact, (float *)Xn,
                                                       (float *)a.dst_identity, rstd, (const float *)gamma, eps,
                                                       a.pos, a.status, a.N, a.C, copy_identity);
    return cudaGetLastError();
}

cudaError_t launch_norm_bwd(const float *dY, const void *Xk, const void *dOk, const float *rstd,
                            const void *gamma, void *dx, void *dgamma, float *dg_part, const int32_t *idx,
                            const int32_t *status, int64_t max_rows, int C, int elem_bytes,
                            int dgamma_fp32, int accumulate, cudaStream_t s)
{
    if (max_rows > 0) {
        if (elem_bytes == 2)
            k_norm_bwd_rows<bf16><<<(unsigned)max_rows, PN_THREADS, 0, s>>>(dY, (const bf16 *)Xk, (const bf16 *)dOk, rstd,
                                                                           (const bf16 *)gamma, (bf16 *)dx, idx, status, C);
        else
            k_norm_bwd_rows<float><<<(unsigned)max_rows, PN_THREADS, 0, s>>>(dY, (const float *)Xk, (const float *)dOk, rstd,
                                                                            (const float *)gamma, (float *)dx, idx, status, C);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (dgamma) {
        dim3 grid((unsigned)((C + DG_COLS - 1) / DG_COLS), DG_CHUNKS);
        const int thr = DG_COLS * DG_LANES;
        if (elem_bytes == 2)
            k_dgamma_partial<bf16><<<grid, thr, 0, s>>>(dY, (const bf16 *)Xk, rstd, dg_part, status, C);
        else
            k_dgamma_partial<float><<<grid, thr, 0, s>>>(dY, (const float *)Xk, rstd, dg_part, status, C);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        const unsigned g2 = (unsigned)((C + 255) / 256);
        if (elem_bytes == 2 && !dgamma_fp32)
            k_dgamma_final<bf16><<<g2, 256, 0, s>>>(dg_part, (bf16 *)dgamma, C, accumulate);
        else
            k_dgamma_final<float><<<g2, 256, 0, s>>>(dg_part, (float *)dgamma, C, accumulate);
        return cudaGetLastError();
    }
    return cudaSuccess;
}

}  // namespace skipffn
