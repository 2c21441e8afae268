// Token merge of the skipped visual tokens (paper section 4.1, three steps): average cosine
// similarity per token, keep the k tokens with the lowest average (the most distinctive), merge
// every other token into its most similar kept token.
//   average similarity  avg_i = (1/n) sum_j xh_i . xh_j = xh_i . mean_j(xh_j): O(n C), no n x n matrix
//   selection           rank of avg_i under (value, index); kept = ranks < k, listed by token index
//   assignment          sims = Xh_rest Xh_kept^T, a dense (n-k) x k x C contraction (tensor cores
//                       for bf16), then a row arg-max (ties: first kept token)
//   merge               mean of a kept token and everything assigned to it (the paper does not
//                       state the operator; this is the reading), summed in token order
// fp32 statistics; every reduction in a fixed order.
#include <string.h>

#include "common.cuh"
#include "rowops.cuh"

namespace skipffn {

// rn[i] = 1 / |x_i| (0 for a zero row): one warp per row
template <typename T>
__global__ void __launch_bounds__(SM_THREADS)
k_row_rnorm(const T *__restrict__ X, float *__restrict__ rn, int64_t n, int C)
{
    pdl_enter();
    const int64_t i = (int64_t)blockIdx.x * (SM_THREADS / 32) + (threadIdx.x >> 5);
    if (i >= n) return;
    const int lane = threadIdx.x & 31;
    float ss = 0.0f;
    for (int c = 4 * lane; c < C; c += 128) {
        float a[4];
        load4(X + i * C + c, a);
#pragma unroll
        for (int q = 0; q < 4; ++q) ss = fmaf(a[q], a[q], ss);
    }
    ss = warp_sum(ss);
    if (lane == 0) rn[i] = ss > 0.0f ? rsqrtf(ss) : 0.0f;
}

// avg_i = rn[i] * dot[i] / n.  keep[i] = 0 (kept) if fewer than k tokens precede i under (avg, index),
// else 1; rest = 1 - keep
__global__ void __launch_bounds__(256)
k_rank_select(const float *__restrict__ dot, const float *__restrict__ rn, int64_t n, int k,
              uint8_t *__restrict__ drop, uint8_t *__restrict__ drop_inv)
{
    pdl_enter();
    __shared__ float tile[256];
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const float a = i < n ? dot[i] * rn[i] / (float)n : 0.0f;
    int rank = 0;
    for (int64_t j0 = 0; j0 < n; j0 += 256) {
        __syncthreads();
        if (j0 + threadIdx.x < n) tile[threadIdx.x] = dot[j0 + threadIdx.x] * rn[j0 + threadIdx.x] / (float)n;
        __syncthreads();
        const int lim = (int)(n - j0 < 256 ? n - j0 : 256);
        for (int t = 0; t < lim; ++t) {
            const float b = tile[t];
            rank += (b < a || (b == a && j0 + t < i)) ? 1 : 0;
        }
    }
    if (i < n) {
        const uint8_t d = rank < k ? 0 : 1;
        drop[i] = d;
        drop_inv[i] = 1 - d;
    }
}

// Two row sets in one launch: CTAs below rows_a fill dst_a from idx_a, the others dst_b from idx_b.
// dst[r] = x[idx[r]] * rn[idx[r]] for r < count, zeros up to the next multiple of ROW_PAD.
template <typename T>
__global__ void __launch_bounds__(128)
k_gather_unit_rows(const T *__restrict__ X, const float *__restrict__ rn, const int32_t *__restrict__ idx_a,
                   int64_t count_a, int64_t rows_a, T *__restrict__ dst_a, const int32_t *__restrict__ idx_b,
                   int64_t count_b, T *__restrict__ dst_b, int C)
{
    pdl_enter();
    const bool second = (int64_t)blockIdx.x >= rows_a;
    const int64_t r = second ? (int64_t)blockIdx.x - rows_a : (int64_t)blockIdx.x;
    const int32_t *idx = second ? idx_b : idx_a;
    const int64_t count = second ? count_b : count_a;
    T *dst = second ? dst_b : dst_a;
    float v[4];
    if (r < count) {
        const int64_t t = idx[r];
        const float s = rn[t];
        for (int c = 4 * threadIdx.x; c < C; c += 512) {
            load4(X + t * C + c, v);
#pragma unroll
            for (int q = 0; q < 4; ++q) v[q] *= s;
            store4(dst + r * C + c, v);
        }
    } else {
        v[0] = v[1] = v[2] = v[3] = 0.0f;
        for (int c = 4 * threadIdx.x; c < C; c += 512) store4(dst + r * C + c, v);
    }
}

// assign[rest[r]] = arg max_j sims[r, j] (first maximum); assign[kept[j]] = j.  One warp per row.
__global__ void __launch_bounds__(SM_THREADS)
k_assign(const float *__restrict__ sims, int64_t n_rest, int k, const int32_t *__restrict__ rest,
         const int32_t *__restrict__ kept, int32_t *__restrict__ assign)
{
    pdl_enter();
    const int64_t r = (int64_t)blockIdx.x * (SM_THREADS / 32) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r < n_rest) {
        float best = -INFINITY;
        int bj = 0x7fffffff;
        for (int j = lane; j < k; j += 32) {
            const float s = sims[r * k + j];
            if (s > best) { best = s; bj = j; }        // ascending j per lane: first maximum of the lane
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best, d);
            const int oj = __shfl_xor_sync(0xffffffffu, bj, d);
            if (ob > best || (ob == best && oj < bj)) { best = ob; bj = oj; }
        }
        if (lane == 0) assign[rest[r]] = bj == 0x7fffffff ? 0 : bj;
    }
    const int64_t g = (int64_t)blockIdx.x * SM_THREADS + threadIdx.x;
    if (g < k) assign[kept[g]] = (int32_t)g;
}

// merged[j] = mean of the rows t (ascending) with assign[t] == j.  One CTA per kept token; thread
// `tid` owns columns 4 tid + 1024 q .. + 3 for q < 16 (C <= 16384).
template <typename T>
__global__ void __launch_bounds__(256)
k_merge_rows(const T *__restrict__ X, const int32_t *__restrict__ assign, int64_t n, T *__restrict__ merged, int C)
{
    pdl_enter();
    __shared__ int32_t members[256];
    __shared__ int warp_cnt[8];
    const int j = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float acc[64];
#pragma unroll
    for (int q = 0; q < 64; ++q) acc[q] = 0.0f;
    int total = 0;
    for (int64_t t0 = 0; t0 < n; t0 += 256) {
        // the tokens of this block of 256 that belong to group j, in ascending order
        __syncthreads();
        const int64_t t = t0 + threadIdx.x;
        const bool mine = t < n && assign[t] == j;
        const unsigned bal = __ballot_sync(0xffffffffu, mine);
        if (lane == 0) warp_cnt[warp] = __popc(bal);
        __syncthreads();
        int base = 0, cnt = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) { if (w < warp) base += warp_cnt[w]; cnt += warp_cnt[w]; }
        if (mine) members[base + __popc(bal & ((1u << lane) - 1u))] = (int32_t)t;
        __syncthreads();
        for (int m = 0; m < cnt; ++m) {
            const T *row = X + (int64_t)members[m] * C;
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                const int c = 4 * threadIdx.x + 1024 * q;
                if (c < C) {
                    float v[4];
                    load4(row + c, v);
                    acc[4 * q] += v[0]; acc[4 * q + 1] += v[1]; acc[4 * q + 2] += v[2]; acc[4 * q + 3] += v[3];
                }
            }
        }
        total += cnt;
    }
    const float inv = total > 0 ? 1.0f / (float)total : 0.0f;
#pragma unroll
    for (int q = 0; q < 16; ++q) {
        const int c = 4 * threadIdx.x + 1024 * q;
        if (c < C) {
            const float v[4] = {acc[4 * q] * inv, acc[4 * q + 1] * inv, acc[4 * q + 2] * inv, acc[4 * q + 3] * inv};
            store4(merged + (int64_t)j * C + c, v);
        }
    }
}

struct MergeScratch {
    float *rn, *avg, *mean, *part, *sims;
    uint8_t *drop, *drop_inv;
    int32_t *kept, *rest, *pos, *status_k, *status_r;
    void *Xa, *Xb;
    size_t total;
};

static MergeScratch merge_layout(char *base, int64_t n, int C, int k, int es)
{
    MergeScratch m;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (size_t)round_up((int64_t)(off + bytes), 256); return base + o; };
    const int64_t npad = round_up(n, ROW_PAD) + ROW_PAD;
    m.rn = (float *)take((size_t)n * 4);
    m.avg = (float *)take((size_t)n * 4);
    m.mean = (float *)take((size_t)C * 4);
    m.part = (float *)take((size_t)DG_CHUNKS * C * 4);
    m.drop = (uint8_t *)take((size_t)n);
    m.drop_inv = (uint8_t *)take((size_t)n);
    m.kept = (int32_t *)take((size_t)npad * 4);
    m.rest = (int32_t *)take((size_t)npad * 4);
    m.pos = (int32_t *)take((size_t)n * 4);
    m.status_k = (int32_t *)take((ST_WORDS + SK_FLAG_WORDS) * 4);
    m.status_r = (int32_t *)take(ST_WORDS * 4);
    m.Xa = take((size_t)round_up(n - k > 0 ? n - k : 1, ROW_PAD) * C * es);
    m.Xb = take((size_t)round_up(k, ROW_PAD) * C * es);
    m.sims = (float *)take((size_t)(n - k > 0 ? n - k : 1) * k * 4);
    m.total = off;
    return m;
}

// device address of the status block the merge's tensor-core GEMM reports to (inside the scratch)
int32_t *merge_status_ptr(void *scratch, int64_t n, int C, int k, int dtype)
{
    return merge_layout((char *)scratch, n, C, k, dtype == SKIPFFN_BF16 ? 2 : 4).status_k;
}

size_t merge_scratch_bytes(int64_t n, int C, int k, int dtype)
{
    return merge_layout(nullptr, n, C, k, dtype == SKIPFFN_BF16 ? 2 : 4).total + (size_t)SK_MAX_CTAS * SK_SLOT_BYTES;
}

template <typename T>
static cudaError_t merge_t(const T *X, int64_t n, int C, int k, int dtype, int32_t *kept_out, int32_t *assign,
                           T *merged, char *scratch, cudaStream_t s)
{
    MergeScratch m = merge_layout(scratch, n, C, k, (int)sizeof(T));
    void *slots = scratch + m.total;
    const int64_t n_rest = n - k;
    cudaError_t e;
    // 1. average similarity
    launch_pdl(k_row_rnorm<T>, dim3((unsigned)((n + 7) / 8)), dim3(SM_THREADS), s, X, m.rn, n, C);
    dim3 g1((C + SP_COLS - 1) / SP_COLS, DG_CHUNKS);
    launch_pdl(k_weighted_rows<T, float>, dim3(g1), dim3(SP_COLS * SP_LANES), s, X, m.rn, nullptr, 0, n, m.part, C);
    launch_pdl(k_sum_parts<float>, dim3((C + 255) / 256), dim3(256), s, m.part, DG_CHUNKS, m.mean, C);
    launch_pdl(k_row_dots<T, float>, dim3((unsigned)((n + 7) / 8)), dim3(SM_THREADS), s, X, m.mean, nullptr, 0, 0, m.avg, n, C);
    // 2. the k most distinctive tokens, and the others, each as an ascending index list
    launch_pdl(k_rank_select, dim3((unsigned)((n + 255) / 256)), dim3(256), s, m.avg, m.rn, n, k, m.drop, m.drop_inv);
    if ((e = cudaMemsetAsync(m.status_k, 0, (ST_WORDS + SK_FLAG_WORDS) * 4, s)) != cudaSuccess) return e;
    if ((e = launch_compact(m.drop, n, 0, m.kept, m.pos, m.status_k, round_up(n, ROW_PAD) + ROW_PAD, n, s)) != cudaSuccess) return e;
    if ((e = launch_compact(m.drop_inv, n, 0, m.rest, m.pos, m.status_r, round_up(n, ROW_PAD) + ROW_PAD, n, s)) != cudaSuccess) return e;
    if ((e = cudaMemcpyAsync(kept_out, m.kept, (size_t)k * 4, cudaMemcpyDeviceToDevice, s)) != cudaSuccess) return e;
    // 3. assignment: unit rows, similarity GEMM, arg max
    if (n_rest > 0) {
        const int64_t rows_a = round_up(n_rest, ROW_PAD), rows_b = round_up(k, ROW_PAD);
        launch_pdl(k_gather_unit_rows<T>, dim3((unsigned)(rows_a + rows_b)), dim3(128), s, X, m.rn, m.rest, n_rest, rows_a,
                   (T *)m.Xa, m.kept, (int64_t)k, (T *)m.Xb, C);
        GemmArgs g;
        memset(&g, 0, sizeof(g));
        g.A = m.Xa; g.lda_m = C; g.lda_k = 1; g.a_outer = round_up(n_rest, ROW_PAD);
        g.B = m.Xb; g.ldb_n = C; g.ldb_k = 1; g.b_outer = round_up(k, ROW_PAD);
        g.M = (int32_t)n_rest; g.N = k; g.K = C;
        g.status = m.status_k; g.idx = m.kept;
        g.out0 = m.sims; g.ldo = k; g.out_fp32 = 1;
        g.sk_slots = slots; g.sk_flags = m.status_k + ST_WORDS; g.sk_epoch = 1; g.tune_streamk = -1;
        e = dtype == SKIPFFN_BF16 ? launch_umma_gemm(EPI_PLAIN, g, s) : launch_simt_gemm(EPI_DW, dtype, g, s);
        if (e != cudaSuccess) return e;
    }
    launch_pdl(k_assign, dim3((unsigned)((max((int64_t)k, n_rest * 32) + SM_THREADS - 1) / SM_THREADS)), dim3(SM_THREADS), s, 
        m.sims, n_rest, k, m.rest, m.kept, assign);
    // 4. merge
    launch_pdl(k_merge_rows<T>, dim3(k), dim3(256), s, X, assign, n, merged, C);
    return cudaGetLastError();
}

cudaError_t launch_token_merge(const void *X, int64_t n, int C, int k, int dtype, int32_t *kept, int32_t *assign,
                               void *merged, void *scratch, cudaStream_t s)
{
    return dtype == SKIPFFN_BF16
               ? merge_t<bf16>((const bf16 *)X, n, C, k, dtype, kept, assign, (bf16 *)merged, (char *)scratch, s)
               : merge_t<float>((const float *)X, n, C, k, dtype, kept, assign, (float *)merged, (char *)scratch, s);
}

}  // namespace skipffn
