// Tensor-core GEMM kernels of the Skip-FFN path for sm_100a: TMA-fed shared-memory pipeline,
// tcgen05.mma with fp32 accumulators in tensor memory, fused Skip-FFN epilogues.
//
// One persistent kernel template serves every contraction of the path:
//   C[m, n] = sum_k A(m, k) * B(n, k),   bf16 in, fp32 accumulate, K step 64.
// Either operand may be K-major (global array [rows = M or N, cols = K]) or MN-major (global array
// [rows = K, cols = M or N]); the latter is what the backward pass needs for W_down (dH), for
// W_gate / W_up (dX) and for both operands of the weight-gradient GEMMs, whose reduction axis is the
// compacted token axis.
//
// Two launch shapes share the code:
//   PAIR   two CTAs of a cluster (an SM pair) compute one 256 x bn tile with cta_group::2 MMAs.
//          Each CTA stages its own 128 rows of A and HALF of the B tile, so an SM pulls 32 KiB
//          from L2 per K step for a 128 x 256 x 64 block of work (128 flop/byte); six stages.
//   SINGLE one CTA computes a 128 x bn tile (48 KiB per K step, 85 flop/byte); four stages.
//          Used when the device cannot co-schedule pairs.
//
// Warp roles (320 threads per CTA, one CTA per SM):
//   warp 0      TMA producer: fills the stage ring (128-byte swizzle)
//   warp 1      MMA issuer (the pair's leader CTA issues for both SMs): owns the tensor-memory
//               allocation (512 columns = two 128 x 256 fp32 accumulators per SM), issues four K=16
//               tcgen05.mma per stage, releases stages and publishes finished accumulators through
//               tcgen05.commit
//   warps 2..9  epilogue: read one accumulator (tcgen05.ld, one row per thread) while the MMA warp
//               fills the other, apply the fused epilogue, write global memory
//
// The kept-token count Nk lives in device memory, so tile counts are derived on the device and no
// host synchronisation sits between mask compaction and the GEMMs.  Every wait (mbarrier or
// hand-over flag) is bounded: on expiry the CTA records SKIPFFN_ETIMEOUT plus a site code and
// leaves normally.
//
// Work distribution.  A launch has T output tiles of KB K-blocks each and W tile workers (CTAs or
// CTA pairs, all co-resident).  Whole waves of W tiles are handed out tile by tile; the tiles of
// the last one-to-two waves (T mod W of them, plus W more when there are that many) are instead
// cut along K into W equal, contiguous runs of K-blocks, one per worker, so that every worker
// carries the same number of K-blocks whatever T mod W is.  A run that stops short of its last
// tile's final K-block leaves that tile's fp32 partial accumulator in the worker's slot of the
// workspace (each worker has at most one such run and processes it first); the worker whose run
// contains the tile's final K-block adds the slots of its predecessors, in a fixed order, and
// runs the epilogue.  The summation order depends only on the shapes, so results are
// reproducible from run to run.
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#include "sched.cuh"

namespace skipffn {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int MAX_STAGES = 6;
constexpr int A_BYTES = BM * BK * 2;             // 16 KiB: this CTA's 128 rows of A
constexpr int CHUNK_BYTES = 64 * BK * 2;         // one 64-wide slab of B (or MN-major A): 8 KiB
constexpr int ACC_COLS = 256;                    // fp32 columns per accumulator
constexpr int TMEM_COLS = 512;
constexpr int EPI_WARPS = 8;
constexpr int EPI_BUF_BYTES = 2048;              // per-warp staging: 32 rows x 64 B
constexpr int UMMA_THREADS = 64 + 32 * EPI_WARPS;
template <bool PAIR> struct Shape {
    static constexpr int STAGES = PAIR ? 6 : 4;
    static constexpr int B_BYTES = PAIR ? 128 * BK * 2 : 256 * BK * 2;   // B rows staged per CTA
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * EPI_BUF_BYTES +
                                      1024 /*alignment slack*/ + 256 /*barriers*/;
};
constexpr unsigned long long WAIT_LIMIT_NS = 1000000000ull;   // 1 s

// ------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One probe of the barrier.  The suspend-time hint (nanoseconds) lets the hardware park the thread
// until the phase completes instead of returning at once: waiting warps then stop competing for
// issue slots (measured: 4 % off every GEMM of the path).  It only bounds one probe; the bounded
// wait around it keeps its own 1 s limit.
constexpr uint32_t TRY_WAIT_HINT_NS = 20000u;
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(TRY_WAIT_HINT_NS)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false if the CTA is aborting (this wait or another one ran out of time).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                            int32_t *status, int site)
{
    unsigned long long t0 = globaltimer_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 0xf) == 0) {     // a probe may take up to TRY_WAIT_HINT_NS
            if (*abort_flag) return false;
            if (globaltimer_ns() - t0 > WAIT_LIMIT_NS) {
                *abort_flag = 1;
                if (atomicCAS(&status[ST_STATUS], 0, (int)SKIPFFN_ETIMEOUT) == 0)
                    status[ST_SITE] = site;
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          int32_t *status, int site)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, status, site);
}

// Bounded wait of one warp for a hand-over flag written by another CTA of this launch.
__device__ __noinline__ bool flag_wait(const int32_t *flag, int32_t want, int lane,
                                       volatile int *abort_flag, int32_t *status)
{
    int ok = 1;
    if (lane == 0) {
        unsigned long long t0 = 0;
        for (uint32_t it = 1;; ++it) {
            int32_t v;
            asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
            if (v == want) break;
            if ((it & 0x3f) == 0) {
                if (*abort_flag) { ok = 0; break; }
                if (t0 == 0) t0 = globaltimer_ns();
                else if (globaltimer_ns() - t0 > WAIT_LIMIT_NS) {
                    *abort_flag = 1;
                    if (atomicCAS(&status[ST_STATUS], 0, (int)SKIPFFN_ETIMEOUT) == 0)
                        status[ST_SITE] = SITE_EPI_PARTIAL;
                    ok = 0;
                    break;
                }
            }
        }
    }
    ok = __shfl_sync(0xffffffffu, ok, 0);
    return ok != 0;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst),
                 "r"(cols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols)
                 : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]; one thread issues for the CTA
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// mbarrier arrives once every tcgen05 operation issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives row (lane base + i)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
          "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),
          "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- cluster (SM pair) variants
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into this CTA's shared memory whose bytes are counted on the pair leader's mbarrier
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int c0, int c1,
                                                 uint32_t leader_bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(c0), "r"(c1), "r"(leader_bar)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst),
                 "r"(cols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols)
                 : "memory");
}
// one MMA spanning both SMs of the pair: 256 rows (128 per SM), issued by the leader CTA
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                               uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrive on the mbarrier at this offset in BOTH CTAs of the pair once the MMAs issued so far retire
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
        "h"((uint16_t)3)
        : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout code 2), descriptor version 1.
// K-major tile:  rows of 64 bf16 (128 B); 8-row groups 1024 B apart (stride byte offset).
// MN-major tile: 64-wide slabs of BK rows x 128 B; 8-row groups 1024 B apart (stride byte offset),
//                next 64-wide slab CHUNK_BYTES further (leading byte offset).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fff);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fff) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = m (128, or 256 across an SM pair), N = n (a
// multiple of 16, at most 256).
__host__ __device__ constexpr uint32_t make_idesc(int a_mn_major, int b_mn_major, int m, int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) |
           ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------------------------ kernel
struct UmmaParams {
    int32_t M, N, K;                 // host upper bounds
    int32_t m_from_nk, k_from_nk;    // extent is the device-resident kept count
    int32_t segments;                // 2: second K segment reads tmA2 / tmB2 (dX)
    int32_t force_bn;                // > 0: tile width override (tuning)
    int32_t force_stages;            // > 0: use fewer ring stages (tuning)
    int32_t *status;
    const int32_t *idx;
    void *out0, *out1, *out2;
    const void *in0, *in1;
    int64_t ldo;
    int32_t accumulate, out_fp32;
    float4 *sk_slots;                // per-CTA partial-accumulator slots
    int32_t *sk_flags;               // SK_FLAGS_PER_CTA flags per slot
    int32_t sk_epoch;                // flag value of this launch
    int32_t sk_wait_skew;            // 0; test hook: finishing units wait for a value nobody writes
    // grouped launch (weight gradients): up to three independent problems sharing K; problem g has
    // extents gM[g] x gN[g], operands (tmA, tmB) / (tmA2, tmB2) / (tmA3, tmB2), output gout[g]
    int32_t groups;
    int32_t gM[3], gN[3];
    void *gout[3];
    int64_t gldo[3];
    int32_t streamk;                 // 0: whole tiles only; else the least number of K-blocks per worker
                                     // that cutting the last waves along K must save to be used
};

struct alignas(8) SmemCtl {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ void unpack_bf16(uint32_t w, float &lo, float &hi)
{
    __nv_bfloat162 v = *reinterpret_cast<__nv_bfloat162 *>(&w);
    lo = __low2float(v);
    hi = __high2float(v);
}

// sigmoid from the hardware exp2 / reciprocal approximations (relative error ~1e-6, far below the
// bf16 rounding of everything it feeds)
__device__ __forceinline__ float fast_sigmoid(float z) { return __fdividef(1.0f, 1.0f + __expf(-z)); }
__device__ __forceinline__ float fast_swiglu(float g, float u) { return g * fast_sigmoid(g) * u; }
__device__ __forceinline__ void fast_swiglu_bwd(float dh, float g, float u, float &dg, float &du)
{
    float s = fast_sigmoid(g);
    du = dh * (g * s);
    dg = dh * u * (s * (1.0f + g * (1.0f - s)));
}

// Epilogue staging.  A warp owns 32 accumulator rows (one per lane).  For a 32-column bf16 chunk
// each lane holds its row as 16 packed words (64 B).  The rows are written to a 2 KiB per-warp
// shared-memory buffer (16-byte slots XOR-swizzled by row pair: conflict-free both ways), then read
// back so that four consecutive lanes cover one row's 64 contiguous bytes: every global store
// instruction writes eight full 64-byte row segments instead of 32 scattered 16-byte pieces.
// `my_row` is this lane's destination (row pointer at the chunk's first column) or null for a row
// that must not be written; `valid_slots` = number of 16-byte slots inside the column range.
__device__ __forceinline__ void store_rows_64B(uint32_t sbuf, int lane, const uint32_t (&w)[16],
                                               char *my_row, int valid_slots)
{
    const int sw = (lane >> 1) & 3;
#pragma unroll
    for (int c = 0; c < 4; ++c)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sbuf + lane * 64 + ((c ^ sw) << 4)),
                     "r"(w[4 * c]), "r"(w[4 * c + 1]), "r"(w[4 * c + 2]), "r"(w[4 * c + 3])
                     : "memory");
    __syncwarp();
    const int c = lane & 3;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int row = it * 8 + (lane >> 2);
        uint4 v;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                     : "r"(sbuf + row * 64 + ((c ^ ((row >> 1) & 3)) << 4))
                     : "memory");
        char *dst = (char *)__shfl_sync(0xffffffffu, (unsigned long long)my_row, row);
        if (dst != nullptr && c < valid_slots) *reinterpret_cast<uint4 *>(dst + c * 16) = v;
    }
    __syncwarp();
}
// The reverse for epilogue inputs.  `v[it]` holds the 16 bytes this lane loaded from row
// it * 8 + lane / 4, slot lane % 4 (four consecutive lanes cover one row's 64 bytes, so a warp
// load touches eight full 64-byte segments instead of 32 scattered 16-byte pieces); the same
// staging buffer turns them into this lane's own row as 16 packed words.
__device__ __forceinline__ void rows_from_coalesced(uint32_t sbuf, int lane, const uint4 (&v)[4],
                                                    uint32_t (&w)[16])
{
    const int c = lane & 3;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int row = it * 8 + (lane >> 2);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sbuf + row * 64 + ((c ^ ((row >> 1) & 3)) << 4)),
                     "r"(v[it].x), "r"(v[it].y), "r"(v[it].z), "r"(v[it].w)
                     : "memory");
    }
    __syncwarp();
    const int sw = (lane >> 1) & 3;
#pragma unroll
    for (int q = 0; q < 4; ++q)
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(w[4 * q]), "=r"(w[4 * q + 1]), "=r"(w[4 * q + 2]), "=r"(w[4 * q + 3])
                     : "r"(sbuf + lane * 64 + ((q ^ sw) << 4))
                     : "memory");
    __syncwarp();
}
// fp32 variant with read-modify-write (dW accumulation): same staging, 16 columns per call
__device__ __forceinline__ void store_rows_64B_f32(uint32_t sbuf, int lane, const uint32_t (&w)[16],
                                                   char *my_row, int valid_slots, int accumulate)
{
    const int sw = (lane >> 1) & 3;
#pragma unroll
    for (int c = 0; c < 4; ++c)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sbuf + lane * 64 + ((c ^ sw) << 4)),
                     "r"(w[4 * c]), "r"(w[4 * c + 1]), "r"(w[4 * c + 2]), "r"(w[4 * c + 3])
                     : "memory");
    __syncwarp();
    const int c = lane & 3;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int row = it * 8 + (lane >> 2);
        float4 v;
        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                     : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                     : "r"(sbuf + row * 64 + ((c ^ ((row >> 1) & 3)) << 4))
                     : "memory");
        char *dst = (char *)__shfl_sync(0xffffffffu, (unsigned long long)my_row, row);
        if (dst != nullptr && c < valid_slots) {
            float4 *d = reinterpret_cast<float4 *>(dst + c * 16);
            if (accumulate) { float4 o = *d; v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w; }
            *d = v;
        }
    }
    __syncwarp();
}

template <int EPI, bool A_MN, bool B_MN, bool PAIR>
__global__ void __launch_bounds__(UMMA_THREADS, 1)
k_umma_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2,
            const __grid_constant__ CUtensorMap tmA3, const UmmaParams p)
{
    constexpr bool GATEUP = (EPI == EPI_GATEUP);
    constexpr int STAGES = Shape<PAIR>::STAGES;
    constexpr int STAGE_BYTES = Shape<PAIR>::STAGE_BYTES;
    constexpr int SPLIT = PAIR ? 2 : 1;           // CTAs sharing one tile
    constexpr int TILE_M = BM * SPLIT;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t epi_bufs = tiles + STAGES * STAGE_BYTES;
    SmemCtl *ctl = reinterpret_cast<SmemCtl *>(smem_raw + (tiles - raw) + STAGES * STAGE_BYTES +
                                               EPI_WARPS * EPI_BUF_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;   // position in the SM pair; 0 leads
    const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int num_workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    // ---- set-up that touches no global memory: barriers, tensor memory
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 1);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&ctl->tmem_full[s]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[s]), EPI_WARPS * SPLIT);
        }
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        if (PAIR) { tmem_alloc_pair(smem_u32(&ctl->tmem_base), TMEM_COLS); tmem_relinquish_pair(); }
        else      { tmem_alloc(smem_u32(&ctl->tmem_base), TMEM_COLS); tmem_relinquish(); }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();   // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    volatile int *abort_flag = &ctl->abort_flag;
    // Programmatic dependent launch: the next kernel of the stream may start its own set-up while
    // this one runs; everything below reads what earlier kernels wrote, so wait for them first.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int nk = p.status[ST_NK];
    const int M = p.m_from_nk ? nk : p.M;
    const int K = p.k_from_nk ? nk : p.K;
    // accumulator columns per tile (256 unless overridden); gate and up halves share a tile, so its
    // output is half as wide
    const int bn = (GATEUP || p.force_bn <= 0) ? BN : p.force_bn;
    const int n_tile = GATEUP ? BN / 2 : bn;
    // tiles of problem g: ids [g_first[g], g_first[g+1]), the row-tile index running fastest
    const int groups = (EPI == EPI_DW) ? p.groups : 1;
    int g_m[3], g_n[3], g_num_m[3], g_first[4];
    g_first[0] = 0;
#pragma unroll
    for (int g = 0; g < 3; ++g) {
        g_m[g] = g < groups ? ((EPI == EPI_DW) ? p.gM[g] : M) : 0;
        g_n[g] = g < groups ? ((EPI == EPI_DW) ? p.gN[g] : p.N) : 0;
        g_num_m[g] = (g_m[g] + TILE_M - 1) / TILE_M;
        g_first[g + 1] = g_first[g] + g_num_m[g] * ((g_n[g] + n_tile - 1) / n_tile);
    }
    const int num_tiles = g_first[3];
    auto pick = [](const int (&a)[3], int g) { return g == 2 ? a[2] : (g == 1 ? a[1] : a[0]); };
    struct TileLoc { int g, m0, n0; };
    auto locate = [&](int tile) {
        TileLoc t;
        t.g = (EPI == EPI_DW) ? (tile >= g_first[2] ? 2 : (tile >= g_first[1] ? 1 : 0)) : 0;
        const int local = tile - (t.g == 2 ? g_first[2] : (t.g == 1 ? g_first[1] : 0)), nm = pick(g_num_m, t.g);
        t.m0 = (local % nm) * TILE_M;
        t.n0 = (local / nm) * n_tile;
        return t;
    };
    const int kb_per_seg = (K + BK - 1) / BK;
    const int num_kb = kb_per_seg * p.segments;
    const bool zero_acc = (num_kb == 0);   // empty reduction: the accumulator is exactly zero
    Sched sched;
    // Cutting the last waves costs every worker about two extra epilogues (one hand-over, one
    // finish with the slot added); it pays when the idle time it removes, (W - T mod W) / W of a
    // tile's main loop, is longer than that.
    const int rem_tiles = num_tiles % num_workers;
    const bool split_k = p.streamk > 0 && rem_tiles != 0 &&
                         (long long)(num_workers - rem_tiles) * num_kb >= (long long)p.streamk * num_workers;
    sched.init(worker, num_workers, num_tiles, num_kb, split_k);
    const int num_segs = sched.count();
    const int bn_cta = bn / SPLIT;         // B rows (tile columns) this CTA stages
    const int b_slabs = (bn_cta + 63) / 64;
    const uint32_t nst = (p.force_stages > 0 && p.force_stages < STAGES) ? p.force_stages : STAGES;


    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && !zero_acc) {
            prefetch_tmap(&tmA);
            prefetch_tmap(&tmB);
            if (GATEUP || p.segments == 2 || groups > 1) prefetch_tmap(&tmB2);
            if (p.segments == 2 || groups > 1) prefetch_tmap(&tmA2);
            if (groups > 2) prefetch_tmap(&tmA3);
            // bytes landing on the (leader's) full barrier per stage, from every CTA of the tile
            const uint32_t stage_tx = SPLIT * (A_BYTES + b_slabs * CHUNK_BYTES);
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            // TMA loads of one K-block of one run into ring stage `stage`
            auto issue = [&](const Seg &sg, int kb) {
                const int tile = sg.tile;
                const TileLoc tl = locate(tile);
                const int m0 = tl.m0 + (int)rank * BM, n0 = tl.n0;
                const int nb0 = GATEUP ? n0 : n0 + (int)rank * bn_cta;   // first B row of this CTA
                const int seg = kb >= kb_per_seg ? 1 : 0;
                const int k0 = (kb - seg * kb_per_seg) * BK;
                const CUtensorMap *mA = tl.g == 2 ? &tmA3 : ((tl.g == 1 || seg) ? &tmA2 : &tmA);
                const CUtensorMap *mB = (tl.g >= 1 || seg) ? &tmB2 : &tmB;
                const uint32_t own_bar = smem_u32(&ctl->full[stage]);
                const uint32_t bar = PAIR ? mapa_rank(own_bar, 0) : own_bar;
                const uint32_t sa = tiles + stage * STAGE_BYTES, sb = sa + A_BYTES;
                auto load = [&](uint32_t dst, const CUtensorMap *map, int c0, int c1) {
                    if (PAIR) tma_load_2d_pair(dst, map, c0, c1, bar);
                    else tma_load_2d(dst, map, c0, c1, bar);
                };
                if (rank == 0) mbar_expect_tx(own_bar, stage_tx);
                if (A_MN) {
#pragma unroll
                    for (int j = 0; j < BM / 64; ++j) load(sa + j * CHUNK_BYTES, mA, m0 + 64 * j, k0);
                } else {
                    load(sa, mA, k0, m0);
                }
                if (B_MN) {          // 64-column slabs of BK rows
                    for (int j = 0; j < b_slabs; ++j) load(sb + j * CHUNK_BYTES, mB, nb0 + 64 * j, k0);
                } else if (GATEUP && PAIR) {   // leader stages the 128 gate rows, its peer the up rows
#pragma unroll
                    for (int j = 0; j < 2; ++j)
                        load(sb + j * CHUNK_BYTES, rank == 0 ? &tmB : &tmB2, k0, n0 + 64 * j);
                } else if (GATEUP) { // 128 gate rows, then 128 up rows, in 64-row pieces
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        load(sb + j * CHUNK_BYTES, &tmB, k0, n0 + 64 * j);
                        load(sb + (2 + j) * CHUNK_BYTES, &tmB2, k0, n0 + 64 * j);
                    }
                } else {             // 64-row pieces of a K-major tile are contiguous in smem
                    for (int j = 0; j < b_slabs; ++j) load(sb + j * CHUNK_BYTES, mB, k0, nb0 + 64 * j);
                }
            };
            for (int si = 0; ok && si < num_segs; ++si) {
                const Seg sg = sched.get(si);
                for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
                    ok = mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1, abort_flag, p.status,
                                   SITE_PRODUCER_EMPTY);
                    if (!ok) break;
                    issue(sg, kb);
                    if (++stage == nst) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && !zero_acc && rank == 0) {
            const uint32_t idesc = make_idesc(A_MN ? 1 : 0, B_MN ? 1 : 0, TILE_M, bn);
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int si = 0; ok && si < num_segs; ++si) {
                const Seg sg = sched.get(si);
                ok = mbar_wait(smem_u32(&ctl->tmem_empty[acc]), acc_phase ^ 1, abort_flag, p.status,
                               SITE_MMA_TMEM_EMPTY);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * ACC_COLS;
                for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
                    ok = mbar_wait(smem_u32(&ctl->full[stage]), phase, abort_flag, p.status,
                                   SITE_MMA_FULL);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sa = tiles + stage * STAGE_BYTES, sb = sa + A_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        const uint64_t da = A_MN ? make_desc(sa + k * (UMMA_K * 128), CHUNK_BYTES, 1024)
                                                 : make_desc(sa + k * (UMMA_K * 2), 16, 1024);
                        const uint64_t db = B_MN ? make_desc(sb + k * (UMMA_K * 128), CHUNK_BYTES, 1024)
                                                 : make_desc(sb + k * (UMMA_K * 2), 16, 1024);
                        const uint32_t accumulate = (kb != sg.kb0 || k != 0);   // first MMA of a run overwrites
                        if (PAIR) umma_bf16_pair(d_tmem, da, db, idesc, accumulate);
                        else umma_bf16(d_tmem, da, db, idesc, accumulate);
                    }
                    // the stage is reusable (in both CTAs) once these MMAs retire
                    if (PAIR) umma_commit_pair(smem_u32(&ctl->empty[stage]));
                    else umma_commit(smem_u32(&ctl->empty[stage]));
                    if (++stage == nst) { stage = 0; phase ^= 1; }
                }
                if (ok) {
                    if (PAIR) umma_commit_pair(smem_u32(&ctl->tmem_full[acc]));
                    else umma_commit(smem_u32(&ctl->tmem_full[acc]));
                }
                if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        // Two warps share each 32-lane quarter of tensor memory and alternate over 32-column chunks.
        const int ew = warp - 2;
        const int quarter = warp & 3;
        const int half = ew >> 2;
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t sbuf = epi_bufs + ew * EPI_BUF_BYTES;
        const int esz = p.out_fp32 ? 4 : 2;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        // accumulators are handed back on the leader's barrier, which its MMA warp waits on
        const uint32_t empty_bar0 = smem_u32(&ctl->tmem_empty[0]);
        // hand-over slots: a warp reads back exactly the words the same warp of the producing CTA wrote
        const int my_slot = (int)blockIdx.x;
        auto slot_ptr = [&](int cta_slot, int j) {
            return p.sk_slots + (size_t)cta_slot * (SK_SLOT_BYTES / 16) + ((size_t)(ew * 4 + j) * 8) * 32 + lane;
        };
        for (int si = 0; ok && si < num_segs; ++si) {
            const Seg sg = sched.get(si);
            const int tile = sg.tile;
            const TileLoc tl = locate(tile);
            const int m0 = tl.m0 + (int)rank * BM, n0 = tl.n0;
            if (sg.partial) {
                // ---- this run ends before the tile does: park the raw accumulator in this CTA's slot
                ok = mbar_wait(smem_u32(&ctl->tmem_full[acc]), acc_phase, abort_flag, p.status,
                               SITE_EPI_TMEM_FULL);
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * ACC_COLS;
#pragma unroll 1
                for (int col = half * 32, j = 0; col < bn; col += 64, ++j) {
                    uint32_t r[32];
                    tmem_ld32(t_acc + col, r);
                    tmem_ld_wait();
                    float4 *dst = slot_ptr(my_slot, j);
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        __stcg(dst + v * 32, make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                         __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3])));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    __threadfence();
                    asm volatile("st.release.gpu.global.b32 [%0], %1;" ::"l"(p.sk_flags + my_slot * SK_FLAGS_PER_CTA + ew),
                                 "r"(p.sk_epoch)
                                 : "memory");
                    const uint32_t bar = empty_bar0 + acc * 8;
                    if (PAIR) mbar_arrive_cluster(mapa_rank(bar, 0));
                    else mbar_arrive(bar);
                }
                if (++acc == 2) { acc = 0; acc_phase ^= 1; }
                continue;
            }
            const bool add_slots = sg.kb0 > 0;
            const int m = m0 + row_in_tile;
            const int n_end = min(n0 + n_tile, pick(g_n, tl.g));
            const bool row_valid = m < pick(g_m, tl.g);
            int64_t tok = 0;
            if ((EPI == EPI_DOWN || EPI == EPI_DX) && row_valid) tok = p.idx[m];
            // prefetch of the per-row epilogue inputs of the first chunk (overlaps the accumulator wait)
            uint4 pa[4], pb[4];
            auto prefetch = [&](int n) {
                // compact rows m0 + quarter * 32 .. + 31 of in0 / in1, loaded eight rows per instruction
                if ((EPI == EPI_DH || EPI == EPI_DOWN || EPI == EPI_DX) && p.in0 != nullptr) {
                    const int c = lane & 3;
#pragma unroll
                    for (int it = 0; it < 4; ++it) {
                        const int mr = m0 + quarter * 32 + it * 8 + (lane >> 2);
                        pa[it] = make_uint4(0, 0, 0, 0);
                        pb[it] = make_uint4(0, 0, 0, 0);
                        if (mr < pick(g_m, tl.g) && n + c * 8 < n_end) {
                            const int64_t o = (int64_t)mr * p.ldo + n + c * 8;
                            pa[it] = __ldcs(reinterpret_cast<const uint4 *>((const bf16 *)p.in0 + o));
                            if (EPI == EPI_DH) pb[it] = __ldcs(reinterpret_cast<const uint4 *>((const bf16 *)p.in1 + o));
                        }
                    }
                }
            };
            prefetch(n0 + half * 32);
            if (!zero_acc) {
                ok = mbar_wait(smem_u32(&ctl->tmem_full[acc]), acc_phase, abort_flag, p.status,
                               SITE_EPI_TMEM_FULL);
                if (!ok) break;
                tc_fence_after();
            }
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * ACC_COLS;
            if (add_slots) {
                // the rest of this tile's K range sits in the slots of workers src_lo .. worker-1
                for (int q = sg.src_lo; ok && q < worker; ++q) {
                    if (sched.bound(q + 1) == sched.bound(q)) continue;   // that worker had no run
                    ok = flag_wait(p.sk_flags + (q * SPLIT + (int)rank) * SK_FLAGS_PER_CTA + ew,
                                   p.sk_epoch + p.sk_wait_skew, lane, abort_flag, p.status);
                }
                if (!ok) break;
            }

#pragma unroll 1
            for (int n = n0 + half * 32; n < n_end; n += 64) {
                const int col = n - n0;
                uint32_t r[32], r2[GATEUP ? 32 : 1];
                if (!zero_acc) {
                    tmem_ld32(t_row + col, r);
                    if (GATEUP) tmem_ld32(t_row + BN / 2 + col, *reinterpret_cast<uint32_t(*)[32]>(&r2));
                } else {
#pragma unroll
                    for (int q = 0; q < 32; ++q) r[q] = 0u;
                }
                uint4 ca[4], cb[4];
#pragma unroll
                for (int v = 0; v < 4; ++v) { ca[v] = pa[v]; cb[v] = pb[v]; }
                if (n + 64 < n_end) prefetch(n + 64);
                if (!zero_acc) tmem_ld_wait();
                if (add_slots) {
                    const int j = col >> 6;   // this warp's j-th 32-column chunk of the accumulator
                    for (int q = sg.src_lo; q < worker; ++q) {
                        if (sched.bound(q + 1) == sched.bound(q)) continue;
                        const float4 *src = slot_ptr(q * SPLIT + (int)rank, j);
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            const float4 a = __ldcg(src + v * 32);
                            r[4 * v] = __float_as_uint(__uint_as_float(r[4 * v]) + a.x);
                            r[4 * v + 1] = __float_as_uint(__uint_as_float(r[4 * v + 1]) + a.y);
                            r[4 * v + 2] = __float_as_uint(__uint_as_float(r[4 * v + 2]) + a.z);
                            r[4 * v + 3] = __float_as_uint(__uint_as_float(r[4 * v + 3]) + a.w);
                        }
                        if (GATEUP) {   // the up half of the accumulator: columns 128 + col
                            const float4 *src2 = slot_ptr(q * SPLIT + (int)rank, j + 2);
#pragma unroll
                            for (int v = 0; v < 8; ++v) {
                                const float4 a = __ldcg(src2 + v * 32);
                                r2[GATEUP ? 4 * v : 0] = __float_as_uint(__uint_as_float(r2[GATEUP ? 4 * v : 0]) + a.x);
                                r2[GATEUP ? 4 * v + 1 : 0] = __float_as_uint(__uint_as_float(r2[GATEUP ? 4 * v + 1 : 0]) + a.y);
                                r2[GATEUP ? 4 * v + 2 : 0] = __float_as_uint(__uint_as_float(r2[GATEUP ? 4 * v + 2 : 0]) + a.z);
                                r2[GATEUP ? 4 * v + 3 : 0] = __float_as_uint(__uint_as_float(r2[GATEUP ? 4 * v + 3 : 0]) + a.w);
                            }
                        }
                    }
                }
                const int valid_slots = min(4, (n_end - n) / 8);
                uint32_t w[16];
                if (EPI == EPI_GATEUP) {
                    // compacted G, U, H; rows past Nk inside the tile are written as zeros
                    const int64_t o = (int64_t)m * p.ldo + n;
                    char *rowG = (char *)((bf16 *)p.out0 + o), *rowU = (char *)((bf16 *)p.out1 + o),
                         *rowH = (char *)((bf16 *)p.out2 + o);
                    if (!row_valid) {
#pragma unroll
                        for (int q = 0; q < 32; ++q) { r[q] = 0u; r2[GATEUP ? q : 0] = 0u; }
                    }
#pragma unroll
                    for (int q = 0; q < 16; ++q) w[q] = pack_bf16(__uint_as_float(r[2 * q]), __uint_as_float(r[2 * q + 1]));
                    store_rows_64B(sbuf, lane, w, rowG, valid_slots);
#pragma unroll
                    for (int q = 0; q < 16; ++q)
                        w[q] = pack_bf16(__uint_as_float(r2[GATEUP ? 2 * q : 0]), __uint_as_float(r2[GATEUP ? 2 * q + 1 : 0]));
                    store_rows_64B(sbuf, lane, w, rowU, valid_slots);
#pragma unroll
                    for (int q = 0; q < 16; ++q)
                        w[q] = pack_bf16(fast_swiglu(__uint_as_float(r[2 * q]), __uint_as_float(r2[GATEUP ? 2 * q : 0])),
                                         fast_swiglu(__uint_as_float(r[2 * q + 1]), __uint_as_float(r2[GATEUP ? 2 * q + 1 : 0])));
                    store_rows_64B(sbuf, lane, w, rowH, valid_slots);
                } else if (EPI == EPI_DX && p.out_fp32) {
                    // pre-norm variant: the raw fp32 gradient w.r.t. the normalised rows, compact,
                    // no residual (the normalisation's backward runs afterwards, row-wide)
                    char *row = row_valid ? (char *)p.out0 + ((int64_t)m * p.ldo + n) * 4 : nullptr;
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                        for (int q = 0; q < 16; ++q) w[q] = r[hh * 16 + q];
                        store_rows_64B_f32(sbuf, lane, w, row ? row + hh * 64 : nullptr,
                                           min(4, max(0, (n_end - n - hh * 16) / 4)), 0);
                    }
                } else if (EPI == EPI_DOWN || EPI == EPI_DX) {
                    // residual add in fp32, one rounding, scatter to the token's row
                    uint32_t rw[16];
                    rows_from_coalesced(sbuf, lane, ca, rw);
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        float a0, a1;
                        unpack_bf16(rw[q], a0, a1);
                        w[q] = pack_bf16(a0 + __uint_as_float(r[2 * q]), a1 + __uint_as_float(r[2 * q + 1]));
                    }
                    char *row = row_valid ? (char *)((bf16 *)p.out0 + tok * p.ldo + n) : nullptr;
                    store_rows_64B(sbuf, lane, w, row, valid_slots);
                } else if (EPI == EPI_DH) {
                    uint32_t gw[16], uw[16];
                    rows_from_coalesced(sbuf, lane, ca, gw);
                    rows_from_coalesced(sbuf, lane, cb, uw);
                    uint32_t w2[16];
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        float g0, g1, u0, u1, dg0, dg1, du0, du1;
                        unpack_bf16(gw[q], g0, g1);
                        unpack_bf16(uw[q], u0, u1);
                        fast_swiglu_bwd(__uint_as_float(r[2 * q]), g0, u0, dg0, du0);
                        fast_swiglu_bwd(__uint_as_float(r[2 * q + 1]), g1, u1, dg1, du1);
                        if (!row_valid) { dg0 = dg1 = du0 = du1 = 0.0f; }
                        w[q] = pack_bf16(dg0, dg1);
                        w2[q] = pack_bf16(du0, du1);
                    }
                    const int64_t o = (int64_t)m * p.ldo + n;
                    store_rows_64B(sbuf, lane, w, (char *)((bf16 *)p.out0 + o), valid_slots);
                    store_rows_64B(sbuf, lane, w2, (char *)((bf16 *)p.out1 + o), valid_slots);
                } else {   // EPI_DW: weight-gradient tile, overwrite or accumulate
                    const int64_t o = (int64_t)m * p.gldo[tl.g] + n;
                    char *row = row_valid ? (char *)p.gout[tl.g] + o * esz : nullptr;
                    if (p.out_fp32) {
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                            for (int q = 0; q < 16; ++q) w[q] = r[hh * 16 + q];
                            store_rows_64B_f32(sbuf, lane, w, row ? row + hh * 64 : nullptr,
                                               min(4, max(0, (n_end - n - hh * 16) / 4)), p.accumulate);
                        }
                    } else if (!p.accumulate) {
#pragma unroll
                        for (int q = 0; q < 16; ++q) w[q] = pack_bf16(__uint_as_float(r[2 * q]), __uint_as_float(r[2 * q + 1]));
                        store_rows_64B(sbuf, lane, w, row, valid_slots);
                    } else if (row_valid) {   // bf16 accumulation: add in fp32, round once (per-row path)
                        uint4 *dst = reinterpret_cast<uint4 *>(row);
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            if (v >= valid_slots) break;
                            uint4 old = dst[v];
                            uint32_t oldw[4] = {old.x, old.y, old.z, old.w}, ow[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                float a0, a1;
                                unpack_bf16(oldw[q], a0, a1);
                                ow[q] = pack_bf16(a0 + __uint_as_float(r[v * 8 + 2 * q]),
                                                  a1 + __uint_as_float(r[v * 8 + 2 * q + 1]));
                            }
                            dst[v] = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                        }
                    }
                }
            }
            if (!zero_acc) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    const uint32_t bar = empty_bar0 + acc * 8;
                    if (PAIR) mbar_arrive_cluster(mapa_rank(bar, 0));
                    else mbar_arrive(bar);
                }
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();   // neither SM leaves while the other may still touch its memory
    if (warp == 1) {
        tc_fence_after();
        if (PAIR) tmem_dealloc_pair(tmem_base, TMEM_COLS);
        else tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------ host
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)sym;
    }
    return fn;
}

// 2-D bf16 row-major array [outer, inner] with row pitch `pitch` elements; box = [box_outer, 64].
// Out-of-range parts of a box read as zero.
static bool make_map(CUtensorMap *m, const void *base, int64_t inner, int64_t outer, int64_t pitch,
                     int box_outer)
{
    EncodeTiledFn enc = get_encode();
    if (!enc || !base) return false;
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)pitch * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)box_outer};
    cuuint32_t es[2] = {1u, 1u};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides,
                     box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

static int g_num_sms = 0;

// Launch one instantiation.  PAIR kernels run as clusters of two CTAs; `workers` counts tiles
// processed concurrently (CTAs, or CTA pairs).
template <int EPI, bool A_MN, bool B_MN, bool PAIR>
static cudaError_t launch_k(const CUtensorMap &a, const CUtensorMap &b, const CUtensorMap &a2,
                            const CUtensorMap &b2, const CUtensorMap &a3, const UmmaParams &p,
                            int64_t max_tiles, cudaStream_t s)
{
    constexpr int SMEM = Shape<PAIR>::SMEM_BYTES;
    static int max_workers = -1;   // -1 not yet queried; 0 unavailable
    auto kern = k_umma_gemm<EPI, A_MN, B_MN, PAIR>;
    if (max_workers < 0) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        if (PAIR) {
            cudaLaunchConfig_t q = {};
            q.gridDim = dim3(2 * g_num_sms);
            q.blockDim = dim3(UMMA_THREADS);
            q.dynamicSmemBytes = SMEM;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            q.attrs = at; q.numAttrs = 1;
            int n = 0;
            e = cudaOccupancyMaxActiveClusters(&n, kern, &q);
            if (e != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
            max_workers = n;
        } else {
            max_workers = g_num_sms;
        }
    }
    if (max_workers <= 0) return cudaErrorNotSupported;
    // `max_tiles` = upper bound of the work items the launch can be cut into (tiles, or groups of
    // K-blocks when tiles are split along K); every worker has its own hand-over slot
    int workers = (int)(max_tiles < max_workers ? max_tiles : max_workers);
    if (workers > SK_MAX_CTAS / (PAIR ? 2 : 1)) workers = SK_MAX_CTAS / (PAIR ? 2 : 1);
    if (workers <= 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(PAIR ? 2 * workers : workers);
    cfg.blockDim = dim3(UMMA_THREADS);
    cfg.dynamicSmemBytes = SMEM;
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = PAIR ? 2 : 1; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    // let this kernel's set-up overlap the tail of the previous kernel on the stream (the kernel
    // itself waits for its predecessors before it reads global memory)
    static int pdl = -1;
    if (pdl < 0) { const char *e = getenv("SKIPFFN_PDL"); pdl = (e && atoi(e) == 0) ? 0 : 1; }
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = pdl ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kern, a, b, a2, b2, a3, p);
}

template <bool PAIR>
static cudaError_t dispatch(int epi, const CUtensorMap &a, const CUtensorMap &b, const CUtensorMap &a2,
                            const CUtensorMap &b2, const CUtensorMap &a3, const UmmaParams &p,
                            int64_t max_tiles, cudaStream_t s)
{
    switch (epi) {
    case EPI_GATEUP: return launch_k<EPI_GATEUP, false, false, PAIR>(a, b, a2, b2, a3, p, max_tiles, s);
    case EPI_DOWN:   return launch_k<EPI_DOWN, false, false, PAIR>(a, b, a2, b2, a3, p, max_tiles, s);
    case EPI_DH:     return launch_k<EPI_DH, false, true, PAIR>(a, b, a2, b2, a3, p, max_tiles, s);
    case EPI_DW:     return launch_k<EPI_DW, true, true, PAIR>(a, b, a2, b2, a3, p, max_tiles, s);
    case EPI_DX:     return launch_k<EPI_DX, false, true, PAIR>(a, b, a2, b2, a3, p, max_tiles, s);
    case EPI_PLAIN:  return launch_k<EPI_DW, false, false, PAIR>(a, b, a2, b2, a3, p, max_tiles, s);
    default: return cudaErrorInvalidValue;
    }
}

// GemmArgs conventions: an operand with ld_k == 1 is K-major ([outer = M or N rows, inner = K]),
// otherwise MN-major with ld_mn == 1 ([outer = K rows, inner = M or N]).  a_outer / b_outer give the
// number of addressable rows of each array.
// `n` > 1 (weight gradients only): up to three independent problems with the same K in one launch;
// problems 1 and 2 share their B operand.
static cudaError_t launch_problems(int epi, const GemmArgs *gs, int n, cudaStream_t s)
{
    if (n < 1 || n > 3 || (n > 1 && epi != EPI_DW) || epi < 0 || epi > EPI_PLAIN) return cudaErrorInvalidValue;
    if (n == 3 && (gs[2].B != gs[1].B || gs[2].ldb_k != gs[1].ldb_k || gs[2].N != gs[1].N))
        return cudaErrorInvalidValue;
    if (g_num_sms == 0) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
    }
    const GemmArgs &g = gs[0];
    const bool gateup = epi == EPI_GATEUP;
    CUtensorMap mA, mB, mA2, mB2, mA3;
    bool ok = true;
    auto mk = [&](CUtensorMap *m, const GemmArgs &q, const void *base, bool is_a) {
        const int64_t ld_mn = is_a ? q.lda_m : q.ldb_n, ld_k = is_a ? q.lda_k : q.ldb_k;
        const int64_t outer = is_a ? q.a_outer : q.b_outer;
        if (ld_k != 1) return make_map(m, base, is_a ? q.M : q.N, outer, ld_k, BK);   // MN-major
        return make_map(m, base, (int64_t)q.K, outer, ld_mn, is_a ? BM : 64);          // K-major
    };
    ok &= mk(&mA, g, g.A, true);
    ok &= mk(&mB, g, g.B, false);
    if (n > 1) {
        ok &= mk(&mA2, gs[1], gs[1].A, true);
        ok &= mk(&mB2, gs[1], gs[1].B, false);
    } else {
        if (g.A2) ok &= mk(&mA2, g, g.A2, true); else mA2 = mA;
        if (g.B2) ok &= mk(&mB2, g, g.B2, false); else mB2 = mB;
    }
    if (n > 2) ok &= mk(&mA3, gs[2], gs[2].A, true); else mA3 = mA;
    if (!ok) return cudaErrorInvalidValue;

    UmmaParams p;
    p.M = g.M; p.N = g.N; p.K = g.K;
    p.m_from_nk = g.m_from_nk; p.k_from_nk = g.k_from_nk;
    p.segments = epi == EPI_DX ? 2 : 1;
    p.force_bn = 0;
    p.force_stages = 0;
    if (const char *e = getenv("SKIPFFN_STAGES")) p.force_stages = atoi(e);
    if (const char *e = getenv("SKIPFFN_TILE_N")) {   // tuning override: accumulator columns per tile
        int v = atoi(e);
        if (v >= 32 && v <= BN && v % 32 == 0) p.force_bn = v;
    }
    p.status = const_cast<int32_t *>(g.status);
    p.idx = g.idx;
    p.out0 = g.out0; p.out1 = g.out1; p.out2 = g.out2;
    p.in0 = g.in0; p.in1 = g.in1;
    p.ldo = g.ldo; p.accumulate = g.accumulate; p.out_fp32 = g.out_fp32;
    p.groups = n;
    for (int i = 0; i < 3; ++i) {
        const GemmArgs &q = gs[i < n ? i : 0];
        p.gM[i] = i < n ? q.M : 0; p.gN[i] = i < n ? q.N : 0;
        p.gout[i] = q.out0; p.gldo[i] = q.ldo;
    }
    p.sk_slots = (float4 *)g.sk_slots;
    p.sk_flags = g.sk_flags;
    p.sk_epoch = g.sk_epoch;
    // Test hook for the failure path: with SKIPFFN_TEST_LOST_HANDOVER set, units that finish a tile
    // wait for a hand-over flag value that no producer writes, so their bounded wait runs out, the
    // kernel records SKIPFFN_ETIMEOUT (site SITE_EPI_PARTIAL) and returns normally after about 1 s.
    p.sk_wait_skew = 0;
    if (const char *e = getenv("SKIPFFN_TEST_LOST_HANDOVER")) { if (atoi(e) != 0) p.sk_wait_skew = 0x40000000; }
    // K-blocks of main loop (about 512 cycles each) that two extra epilogues of this kind cost
    static const int sk_threshold[6] = {/*GATEUP*/ 64, /*DOWN*/ 40, /*DH*/ 96, /*DW*/ 32, /*DX*/ 40, /*PLAIN*/ 32};
    p.streamk = (g.sk_slots && g.sk_flags) ? sk_threshold[epi] : 0;
    if (const char *e = getenv("SKIPFFN_STREAMK")) { int v = atoi(e); if (v >= 0) p.streamk = v; }

    // SM pairs by default; SKIPFFN_SINGLE_CTA=1 (or a device that cannot co-schedule pairs) selects
    // the one-CTA-per-tile shape
    static int single = -1;
    if (single < 0) { const char *e = getenv("SKIPFFN_SINGLE_CTA"); single = (e && atoi(e) != 0) ? 1 : 0; }
    const int n_tile = gateup ? BN / 2 : (p.force_bn > 0 ? p.force_bn : BN);   // output columns per tile
    // with K splitting a tile can be shared by several workers: allow one worker per 4 K-blocks
    const int64_t kb = ((int64_t)g.K + BK - 1) / BK * p.segments;
    const int64_t per_tile = p.streamk ? (kb >= 8 ? kb / 4 : 1) : 1;
    auto max_items = [&](int tile_m) {
        int64_t t = 0;
        for (int i = 0; i < n; ++i)
            t += (((int64_t)gs[i].M + tile_m - 1) / tile_m) * (((int64_t)gs[i].N + n_tile - 1) / n_tile);
        return t * per_tile;
    };
    if (!single) {
        cudaError_t e = dispatch<true>(epi, mA, mB, mA2, mB2, mA3, p, max_items(2 * BM), s);
        if (e != cudaErrorNotSupported) return e;
        (void)cudaGetLastError();
        single = 1;
    }
    return dispatch<false>(epi, mA, mB, mA2, mB2, mA3, p, max_items(BM), s);
}

cudaError_t launch_umma_gemm(int epi, const GemmArgs &g, cudaStream_t s)
{
    return launch_problems(epi, &g, 1, s);
}

cudaError_t launch_umma_dw_group(const GemmArgs *gs, int n, cudaStream_t s)
{
    return launch_problems(EPI_DW, gs, n, s);
}

}  // namespace skipffn
