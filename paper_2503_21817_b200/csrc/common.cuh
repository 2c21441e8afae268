// Shared declarations of the Skip-FFN CUDA library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "skipffn.h"

namespace skipffn {

typedef __nv_bfloat16 bf16;

// Device status block at the start of the workspace (int32 words).
enum : int { ST_NK = 0, ST_STATUS = 1, ST_SITE = 2, ST_ROLE_BASE = 16, ST_WORDS = 64 };   // ST_ROLE_BASE..: optional role cycle counters

// Wait sites reported through the status word when a bounded wait gives up.
enum : int { SITE_PRODUCER_EMPTY = 1, SITE_MMA_FULL = 2, SITE_MMA_TMEM_EMPTY = 3,
             SITE_EPI_TMEM_FULL = 4, SITE_TEARDOWN = 5, SITE_EPI_PARTIAL = 6, SITE_EPI_EXCHANGE = 7, SITE_KEPT_OVERFLOW = 8,
             SITE_DEBUG_KEPT_LIST = 16, SITE_DEBUG_GUARD_BASE = 32 /* + index of the slab whose guard band changed */ };

// Split-K hand-over between CTAs of one tensor-core GEMM launch: a CTA that computes only part
// of a tile's K range leaves its fp32 accumulator in its own slot of the workspace and raises one
// flag per epilogue warp; the CTA that finishes the tile adds the slot to its accumulator.
constexpr int SK_MAX_CTAS = 160;                    // slots (>= CTAs of a persistent launch)
constexpr int SK_SLOT_BYTES = 128 * 256 * 4;        // one CTA's 128 x 256 fp32 accumulator
constexpr int SK_FLAGS_PER_CTA = 8;                 // one per epilogue warp
constexpr int SK_FLAG_WORDS = SK_MAX_CTAS * SK_FLAGS_PER_CTA;

constexpr int ROW_PAD = 256;   // compacted buffers are zero-padded to this many rows past Nk

static inline int64_t round_up(int64_t a, int64_t b) { return (a + b - 1) / b * b; }

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// four consecutive elements (C is a multiple of 8, rows are 16-byte aligned)
__device__ __forceinline__ void load4(const float *p, float (&v)[4])
{
    const float4 t = *reinterpret_cast<const float4 *>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void load4(const bf16 *p, float (&v)[4])
{
    const uint2 t = *reinterpret_cast<const uint2 *>(p);
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162 *>(&t.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162 *>(&t.y);
    v[0] = __low2float(a); v[1] = __high2float(a); v[2] = __low2float(b); v[3] = __high2float(b);
}
__device__ __forceinline__ void store4(float *p, const float (&v)[4])
{
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store4(bf16 *p, const float (&v)[4])
{
    const __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
    uint2 t;
    t.x = *reinterpret_cast<const uint32_t *>(&a);
    t.y = *reinterpret_cast<const uint32_t *>(&b);
    *reinterpret_cast<uint2 *>(p) = t;
}

__device__ __forceinline__ float sigmoidf_(float z) { return 1.0f / (1.0f + expf(-z)); }

// h = silu(g) * u  (Eq. 4's FFN body, SwiGLU)
__device__ __forceinline__ float swiglu(float g, float u) { return g * sigmoidf_(g) * u; }

// Activation backward: given dh and the saved g, u returns dg, du.
//   du = dh * silu(g);  dg = dh * u * silu'(g),  silu'(g) = s (1 + g (1 - s)),  s = sigmoid(g)
__device__ __forceinline__ void swiglu_bwd(float dh, float g, float u, float &dg, float &du)
{
    float s = sigmoidf_(g);
    du = dh * (g * s);
    dg = dh * u * (s * (1.0f + g * (1.0f - s)));
}

// Programmatic dependent launch.  Device side: let the next kernel of the stream start launching,
// then wait until every earlier kernel has completed and its writes are visible (a no-op for a
// kernel launched the ordinary way).  Must precede the kernel's first access to global memory.
__device__ __forceinline__ void pdl_enter()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
// Host side: launch `kernel` so that its launch latency overlaps the tail of the previous kernel.
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t s, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = 0; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---------------------------------------------------------------- launch descriptors (host)
struct RouteArgs {          // row routing: compact copy of kept rows + identity copy of skipped rows
    const void *src;        // [N, C]
    void *dst_compact;      // [cap, C]
    void *dst_identity;     // [N, C] or nullptr / == src for "nothing to copy"
    const int32_t *pos;     // [N] rank of token among kept tokens, or -1
    const int32_t *status;  // status block (Nk)
    int64_t N;
    int32_t C;
    int32_t elem_bytes;
};

// Encoded TMA tensor maps of the arrays a handle keeps seeing (weights, workspace slabs, the
// caller's activations); lives in the handle, filled and searched by the launch code.
constexpr int TMAP_BYTES = 128, TMAP_CACHE_ENTRIES = 48;
struct TmapKey { const void *base; int64_t inner, outer, pitch; int box_outer; int64_t dim2, stride2; };
struct TmapCache {
    int used, next;
    TmapKey key[TMAP_CACHE_ENTRIES];
    alignas(64) unsigned char map[TMAP_CACHE_ENTRIES][TMAP_BYTES];
};

struct GemmArgs {
    // C[m, n] = sum_k A(m, k) * B(n, k)  (+ second segment A2/B2 for dX)
    const void *A, *B, *A2, *B2;
    int64_t lda_m, lda_k, ldb_n, ldb_k;
    int64_t a_outer, b_outer;   // addressable rows of the A / B arrays (tensor-map extents)
    int32_t M, N, K;            // host upper bounds
    int32_t m_from_nk, n_from_nk, k_from_nk;   // 1: the extent is the device-resident kept count
    const int32_t *status;      // status block
    const int32_t *idx;         // kept-row list for scatter epilogues
    // epilogue operands
    void *out0, *out1, *out2;   // meaning depends on the epilogue
    const void *in0, *in1;
    int64_t ldo;                // leading dimension of outputs
    int32_t accumulate;         // DW epilogue: add to the destination
    int32_t out_fp32;           // DW epilogue: destination is float
    // split-K hand-over (tensor-core path): slots, flags and this launch's flag value
    void *sk_slots;
    int32_t *sk_flags;
    int32_t sk_epoch;
    int32_t sk_wait_skew;       // 0; debug handles: make finishing units wait for a value nobody writes
    // tensor-core path: tuning overrides of the handle (0 / -1 = defaults) and its tensor-map cache
    int32_t tune_tile_n, tune_stages, tune_streamk;
    int32_t tune_panel_sync;    // down, dX: -1 choose, 0 never, 1 when cheap, 2 always group workers by weight panel
    int32_t one_box_loads;      // 1: load an operand tile with one 3-D box where the arrays allow it
    int32_t tma_stores;         // 1: weight-gradient tiles leave through TMA tile stores (overwrite mode)
    // gate/up, dH (tensor-core path): non-null = fetch the token operand from this [gather_rows, K]
    // array through the kept-row list instead of from B (its compacted copy)
    const void *gather_src;
    int64_t gather_rows;
    TmapCache *tmaps;
};

// EPI_PLAIN: a plain GEMM with both operands K-major and the weight-gradient store (used by the
// token-merge similarity matrix); the tensor-core path only.
enum Epilogue : int { EPI_GATEUP = 0, EPI_DOWN = 1, EPI_DH = 2, EPI_DW = 3, EPI_DX = 4, EPI_PLAIN = 5 };

// compact.cu
cudaError_t launch_compact(const uint8_t *mask, int64_t N, int32_t dense, int32_t *idx,
                           int32_t *pos, int32_t *status, int64_t cap, int64_t max_kept, cudaStream_t s);
cudaError_t launch_route(const RouteArgs &a, cudaStream_t s);
// debug handles: guard bands behind the workspace slabs, and the invariants of the kept-row list
constexpr int GUARD_BYTES = 1024, GUARD_BYTE = 0xA5, MAX_GUARDS = 24;
struct GuardList { int n; const void *ptr[MAX_GUARDS]; };
cudaError_t launch_check_kept(const int32_t *idx, const int32_t *pos, int32_t *status, int64_t N, cudaStream_t s);
cudaError_t launch_check_guards(const GuardList &g, int32_t *status, cudaStream_t s);
// kvcache.cu
cudaError_t launch_kv_compact(const void *src, void *dst, const int32_t *idx, const int32_t *status,
                              int64_t planes, int64_t N, int64_t dst_rows, int64_t row_bytes,
                              cudaStream_t s);
cudaError_t launch_kept_cu_seqlens(const int32_t *cu, int32_t *new_cu, int n, const int32_t *idx,
                                   const int32_t *status, cudaStream_t s);
// prenorm.cu
cudaError_t launch_route_norm(const RouteArgs &a, void *Xn, float *rstd, const void *gamma, float eps,
                              cudaStream_t s);
cudaError_t launch_norm_bwd(const float *dY, const void *Xk, const void *dOk, const float *rstd,
                            const void *gamma, void *dx, void *dgamma, float *dg_part, const int32_t *idx,
                            const int32_t *status, int64_t max_rows, int C, int elem_bytes,
                            int dgamma_fp32, int accumulate, cudaStream_t s);
constexpr int DG_CHUNKS = 32;   // row chunks of the two-stage dgamma reduction ([DG_CHUNKS, C] fp32 partials)
// summary.cu
cudaError_t launch_summary_forward(const void *X, const int32_t *off, int n_seg, int64_t n, int C, int dtype,
                                   const void *w, void *xs, float *probs, cudaStream_t s);
cudaError_t launch_summary_backward(const void *X, const int32_t *off, int n_seg, int64_t n, int C, int dtype,
                                    const void *w, const float *probs, const void *dxs, void *dX, void *dw,
                                    int dw_fp32, float *scratch, cudaStream_t s);
// merge.cu
size_t merge_scratch_bytes(int64_t n, int C, int k, int dtype);
int32_t *merge_status_ptr(void *scratch, int64_t n, int C, int k, int dtype);
cudaError_t launch_token_merge(const void *X, int64_t n, int C, int k, int dtype, int32_t *kept, int32_t *assign,
                               void *merged, void *scratch, cudaStream_t s);
// simt.cu
cudaError_t launch_simt_gemm(int epi, int dtype, const GemmArgs &a, cudaStream_t s);
// umma.cu (bf16 only)
cudaError_t launch_umma_gemm(int epi, const GemmArgs &a, cudaStream_t s);
// up to three weight-gradient problems (same K; problems 1 and 2 share B) in one launch
cudaError_t launch_umma_dw_group(const GemmArgs *gs, int n, cudaStream_t s);

}  // namespace skipffn
