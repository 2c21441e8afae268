// Mask compaction (kept-row index list) and row routing (gather of kept rows, identity copy of
// skipped rows).  Integer / byte work only: results are bit-exact by construction.
#include "common.cuh"

namespace skipffn {

// Mask compaction.  Outputs (all ascending, i.e. a stable compaction):
//   idx[r]  : token index of the r-th kept token, r < Nk; entries Nk .. round_up(Nk, ROW_PAD)-1
//             (inside idx's capacity) are 0, a valid row, so that padded gathers stay in bounds
//   pos[t]  : rank of token t among kept tokens, or -1 if skipped
//   status[ST_NK] = Nk
// If the mask keeps more than `max_kept` tokens (the bound the compacted arrays were sized for), the
// first max_kept of them are kept, the others are treated as skipped, Nk = max_kept, and the status
// word reports SKIPFFN_EWORKSPACE: memory stays safe, the results are not those of the mask.
//
// k_compact: one CTA per block of 4096 tokens, no communication between CTAs.  A CTA first counts
// the kept tokens in front of its block by reading that part of the mask itself (at most N bytes,
// from L2 after the first CTA touched them), then ranks its own 4096 tokens: every thread owns 16
// consecutive tokens, a ballot-free bit count gives its share, a two-level shuffle scan its offset.
// The last CTA also knows the total and writes Nk and the padding entries.  The redundant counting
// grows with N^2 / 8192 bytes, so very long inputs take the single-CTA kernel below instead.
constexpr int CB_THREADS = 256;
constexpr int CB_PER_THREAD = 16;
constexpr int CB_TOKENS = CB_THREADS * CB_PER_THREAD;      // 4096 tokens per CTA
constexpr int64_t CB_MAX_N = 262144;                        // beyond: k_compact_serial

// number of kept tokens among bytes [lo, hi) of the mask, summed over the CTA (valid in every thread)
__device__ __forceinline__ int block_sum(int v, int *warp_tot)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    if (lane == 0) warp_tot[warp] = v;
    __syncthreads();
    int t = 0;
#pragma unroll
    for (int w = 0; w < CB_THREADS / 32; ++w) t += warp_tot[w];
    __syncthreads();
    return t;
}

__global__ void __launch_bounds__(CB_THREADS)
k_compact(const uint8_t *__restrict__ mask, int64_t N, int dense, int32_t *__restrict__ idx,
          int32_t *__restrict__ pos, int32_t *__restrict__ status, int64_t cap, int max_kept)
{
    __shared__ int warp_tot[CB_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t base = (int64_t)blockIdx.x * CB_TOKENS;
    pdl_enter();
    // ---- kept tokens in front of this block
    int before = 0;
    if (dense) {
        before = (int)base;
    } else {
        int cnt = 0;
        const bool vec = (((uintptr_t)mask) & 15u) == 0;
        if (vec) {
            const uint4 *m4 = reinterpret_cast<const uint4 *>(mask);
            for (int64_t v = tid; v < base / 16; v += CB_THREADS) {   // base is a multiple of 16
                const uint4 q = __ldg(m4 + v);
                cnt += (__popc(__vcmpeq4(q.x, 0u)) + __popc(__vcmpeq4(q.y, 0u)) + __popc(__vcmpeq4(q.z, 0u)) +
                        __popc(__vcmpeq4(q.w, 0u))) >> 3;
            }
        } else {
            for (int64_t t = tid; t < base; t += CB_THREADS) cnt += mask[t] == 0;
        }
        before = block_sum(cnt, warp_tot);
    }
    // ---- this thread's 16 tokens
    const int64_t t0 = base + (int64_t)tid * CB_PER_THREAD;
    unsigned keep = 0;
#pragma unroll
    for (int j = 0; j < CB_PER_THREAD; ++j)
        if (t0 + j < N && (dense || mask[t0 + j] == 0)) keep |= 1u << j;
    const int mine = __popc(keep);
    // exclusive scan over the CTA: within the warp, then over the warp totals
    int incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int off = before + incl - mine, total = before;
#pragma unroll
    for (int w = 0; w < CB_THREADS / 32; ++w) {
        if (w < warp) off += warp_tot[w];
        total += warp_tot[w];
    }
    int r = off;
#pragma unroll
    for (int j = 0; j < CB_PER_THREAD; ++j) {
        if (t0 + j < N) {
            if (((keep >> j) & 1u) && r < max_kept) { idx[r] = (int32_t)(t0 + j); pos[t0 + j] = r; }
            else pos[t0 + j] = -1;
            r += (keep >> j) & 1u;
        }
    }
    if (blockIdx.x == gridDim.x - 1) {   // the last block knows the total
        if (total > max_kept) {
            total = max_kept;
            if (tid == 0 && atomicCAS(&status[ST_STATUS], 0, (int)SKIPFFN_EWORKSPACE) == 0) status[ST_SITE] = SITE_KEPT_OVERFLOW;
        }
        if (tid == 0) status[ST_NK] = total;
        int64_t end = ((int64_t)total + ROW_PAD - 1) / ROW_PAD * ROW_PAD;
        if (end > cap) end = cap;
        for (int64_t q = total + tid; q < end; q += CB_THREADS) idx[q] = 0;
    }
}

// One CTA of 1024 threads walks the mask in slabs of 16 x 1024 tokens (inputs too long for the
// redundant counting above).  Within a slab, token (j, warp, lane) = base + j*1024 + warp*32 + lane;
// a warp ballot gives each kept token its rank inside its 32-token segment, and an exclusive scan
// over the 512 segment counts (segments are in ascending token order) gives the segment's offset.
constexpr int CP_THREADS = 1024;
constexpr int CP_J = 16;

__global__ void __launch_bounds__(CP_THREADS)
k_compact_serial(const uint8_t *__restrict__ mask, int64_t N, int dense, int32_t *__restrict__ idx,
                 int32_t *__restrict__ pos, int32_t *__restrict__ status, int64_t cap, int max_kept)
{
    __shared__ int seg[CP_J * 32];
    __shared__ int slab_total;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned lt = (1u << lane) - 1u;
    int carry = 0;
    pdl_enter();
    for (int64_t base = 0; base < N; base += (int64_t)CP_J * CP_THREADS) {
        unsigned bal[CP_J];
#pragma unroll
        for (int j = 0; j < CP_J; ++j) {
            int64_t t = base + (int64_t)j * CP_THREADS + tid;
            bool keep = t < N && (dense || mask[t] == 0);
            bal[j] = __ballot_sync(0xffffffffu, keep);
            if (lane == 0) seg[j * 32 + warp] = __popc(bal[j]);
        }
        __syncthreads();
        if (warp == 0) {   // exclusive scan of the 512 segment counts, 16 per lane
            int loc[CP_J], sum = 0;
#pragma unroll
            for (int q = 0; q < CP_J; ++q) { loc[q] = seg[lane * CP_J + q]; sum += loc[q]; }
            int incl = sum;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                int v = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += v;
            }
            int run = incl - sum;
#pragma unroll
            for (int q = 0; q < CP_J; ++q) { seg[lane * CP_J + q] = run; run += loc[q]; }
            if (lane == 31) slab_total = incl;
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < CP_J; ++j) {
            int64_t t = base + (int64_t)j * CP_THREADS + tid;
            if (t < N) {
                if ((bal[j] >> lane) & 1u) {
                    int r = carry + seg[j * 32 + warp] + __popc(bal[j] & lt);
                    if (r < max_kept) { idx[r] = (int32_t)t; pos[t] = r; }
                    else pos[t] = -1;
                } else {
                    pos[t] = -1;
                }
            }
        }
        carry += slab_total;
        __syncthreads();
    }
    if (carry > max_kept) {
        carry = max_kept;
        if (tid == 0 && atomicCAS(&status[ST_STATUS], 0, (int)SKIPFFN_EWORKSPACE) == 0) status[ST_SITE] = SITE_KEPT_OVERFLOW;
    }
    if (tid == 0) status[ST_NK] = carry;
    int64_t end = ((int64_t)carry + ROW_PAD - 1) / ROW_PAD * ROW_PAD;
    if (end > cap) end = cap;
    for (int64_t r = carry + tid; r < end; r += CP_THREADS) idx[r] = 0;
}

cudaError_t launch_compact(const uint8_t *mask, int64_t N, int32_t dense, int32_t *idx,
                           int32_t *pos, int32_t *status, int64_t cap, int64_t max_kept, cudaStream_t s)
{
    const int mk = (int)(max_kept < N ? max_kept : N);
    if (N > CB_MAX_N)
        return launch_pdl(k_compact_serial, dim3(1), dim3(CP_THREADS), s, mask, N, (int)dense, idx, pos, status, cap, mk);
    const unsigned blocks = (unsigned)((N + CB_TOKENS - 1) / CB_TOKENS);
    return launch_pdl(k_compact, dim3(blocks), dim3(CB_THREADS), s, mask, N, (int)dense, idx, pos, status, cap, mk);
}

// Debug handles: check the kept-row list against its own invariants (in range, strictly ascending,
// consistent with the inverse map) and report a violation through the status word.
__global__ void k_check_kept(const int32_t *__restrict__ idx, const int32_t *__restrict__ pos,
                             int32_t *__restrict__ status, int64_t N)
{
    const int nk = status[ST_NK];
    bool bad = nk < 0 || nk > N;
    for (int64_t r = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; !bad && r < nk; r += (int64_t)gridDim.x * blockDim.x) {
        const int32_t t = idx[r];
        bad = t < 0 || t >= N || (r > 0 && idx[r - 1] >= t) || pos[t] != (int32_t)r;
    }
    if (bad && atomicCAS(&status[ST_STATUS], 0, (int)SKIPFFN_EDEBUG) == 0) status[ST_SITE] = SITE_DEBUG_KEPT_LIST;
}

// Debug handles: every slab of the workspace is followed by a guard band filled with GUARD_BYTE; a
// kernel that wrote past the end of its slab leaves a different byte there.
__global__ void k_check_guards(GuardList g, int32_t *__restrict__ status)
{
    const uint32_t want = 0x01010101u * GUARD_BYTE;
    const uint32_t *p = reinterpret_cast<const uint32_t *>(g.ptr[blockIdx.x]);
    bool bad = false;
    for (int i = threadIdx.x; i < GUARD_BYTES / 4; i += blockDim.x) bad |= p[i] != want;
    if (bad && atomicCAS(&status[ST_STATUS], 0, (int)SKIPFFN_EDEBUG) == 0) status[ST_SITE] = SITE_DEBUG_GUARD_BASE + (int)blockIdx.x;
}

cudaError_t launch_check_kept(const int32_t *idx, const int32_t *pos, int32_t *status, int64_t N, cudaStream_t s)
{
    k_check_kept<<<64, 256, 0, s>>>(idx, pos, status, N);
    return cudaGetLastError();
}

cudaError_t launch_check_guards(const GuardList &g, int32_t *status, cudaStream_t s)
{
    if (g.n <= 0) return cudaSuccess;
    k_check_guards<<<g.n, 128, 0, s>>>(g, status);
    return cudaGetLastError();
}

// Row routing.  Unit u < N is token u: a kept token's row goes to dst_compact[pos[u]], a skipped
// token's row goes to dst_identity[u] (byte copy; omitted when dst_identity is null or the
// source itself).  Units u >= N zero the padding rows Nk .. round_up(Nk, ROW_PAD)-1 of
// dst_compact, which later serve as exact-zero K-padding of the weight-gradient GEMMs.
constexpr int RT_THREADS = 128;

__global__ void __launch_bounds__(RT_THREADS)
k_route(const uint4 *__restrict__ src, uint4 *__restrict__ dst_compact,
        uint4 *__restrict__ dst_identity, const int32_t *__restrict__ pos,
        const int32_t *__restrict__ status, int64_t N, int row_vecs, int copy_identity)
{
    int64_t u = blockIdx.x;
    pdl_enter();
    if (u < N) {
        int p = pos[u];
        const uint4 *s = src + u * row_vecs;
        uint4 *d;
        if (p >= 0) d = dst_compact + (int64_t)p * row_vecs;
        else if (copy_identity) d = dst_identity + u * row_vecs;
        else return;
        // four 16-byte loads in flight per thread before the first store; rows are read once
        for (int v0 = threadIdx.x; v0 < row_vecs; v0 += 4 * RT_THREADS) {
            uint4 t[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (v0 + u * RT_THREADS < row_vecs) t[u] = __ldcs(s + v0 + u * RT_THREADS);
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (v0 + u * RT_THREADS < row_vecs) d[v0 + u * RT_THREADS] = t[u];
        }
    } else {
        int nk = status[ST_NK];
        int64_t r = nk + (u - N);
        int64_t end = ((int64_t)nk + ROW_PAD - 1) / ROW_PAD * ROW_PAD;
        if (r >= end) return;
        uint4 *d = dst_compact + r * row_vecs;
        for (int v = threadIdx.x; v < row_vecs; v += RT_THREADS) d[v] = make_uint4(0, 0, 0, 0);
    }
}

cudaError_t launch_route(const RouteArgs &a, cudaStream_t s)
{
    int row_vecs = (int)((int64_t)a.C * a.elem_bytes / 16);
    int copy_identity = a.dst_identity != nullptr && a.dst_identity != a.src;
    int64_t units = a.N + ROW_PAD;
    return launch_pdl(k_route, dim3((unsigned)units), dim3(RT_THREADS), s, (const uint4 *)a.src,
                      (uint4 *)a.dst_compact, (uint4 *)a.dst_identity, a.pos, a.status, a.N, row_vecs,
                      copy_identity);
}

}  // namespace skipffn
