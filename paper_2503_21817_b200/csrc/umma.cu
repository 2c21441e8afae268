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
// Token problems (gate/up, down, dH, dX) put the WEIGHT rows on the accumulator rows (A operand,
// MMA M = 256 per SM pair) and the kept TOKENS on the accumulator columns (B operand, MMA N = any
// multiple of 16 up to 256): the kept count is padded to 16 instead of 256.  Their outputs are
// token-major, the transpose of the accumulator; the epilogue works in MMA-fragment layout and
// transposes through shared memory (tcgen05.ld 16x256b, stmatrix / ldmatrix .trans).
//
// Two launch shapes share the code:
//   PAIR   two CTAs of a cluster (an SM pair) compute one 256 x bn tile with cta_group::2 MMAs.
//          Each CTA stages its own 128 rows of A and HALF of the B tile, so an SM pulls 32 KiB
//          from L2 per K step for a 128 x 256 x 64 block of work (128 flop/byte); six stages.
//   SINGLE one CTA computes a 128 x bn tile (48 KiB per K step, 85 flop/byte); four stages.
//          Used when the device cannot co-schedule pairs.
//
// Warp roles (320 threads per CTA, one CTA per SM):
//   warp 0      TMA producer: fills the stage ring (128-byte swizzle), two or three box loads per stage
//   warp 1      MMA issuer (the pair's leader CTA issues for both SMs): owns the tensor-memory
//               allocation (512 columns = two 128 x 256 fp32 accumulators per SM), issues four K=16
//               tcgen05.mma per stage, releases stages and publishes finished accumulators through
//               tcgen05.commit
//   warps 2..9  epilogue: read one accumulator (tcgen05.ld) while the MMA warp fills the other,
//               apply the fused epilogue, write global memory (16-byte accesses, or TMA tile
//               stores for the weight gradients)
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
// reproducible from run to run.  The down and dX launches at a high skip ratio (few tiles, hundreds
// of K-blocks each) use the same schedule one level up: the workers form groups of one member per
// token tile, a group takes the place of a worker and a weight panel (all token tiles of one row
// block) the place of a tile, so the members of a group read the same weight bytes at the same time
// and DRAM delivers them once.
#include <cuda.h>
#include <stdlib.h>
#include <string.h>

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
constexpr int X_BUF_BYTES = 4096;                // gate/up: fp32 exchange buffer of a warp pair (32 x 32 words)
constexpr int UMMA_THREADS = 64 + 32 * EPI_WARPS;
template <bool PAIR> struct Shape {
    static constexpr int STAGES = PAIR ? 6 : 4;
    static constexpr int B_BYTES = PAIR ? 128 * BK * 2 : 256 * BK * 2;   // B rows staged per CTA
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * EPI_BUF_BYTES + 4 * X_BUF_BYTES +
                                      1024 /*alignment slack*/ + 256 /*barriers*/;
};
constexpr unsigned long long WAIT_LIMIT_NS = 1000000000ull;   // 1 s

// Optional per-role cycle counters (build with -DSKIPFFN_ROLE_CYCLES; never in the default build):
// every launch adds, per epilogue kind, the cycles its MMA issuers spent waiting for operand
// stages and for a free accumulator, the producers' waits for free stages, and one epilogue
// warp's wait and busy time, into status words ST_ROLE_BASE + 8 * EPI + {0..7}.
#ifdef SKIPFFN_ROLE_CYCLES
#define ROLE_CLOCK() clock64()
#define ROLE_ADD(var, t0) (var) += clock64() - (t0)
#else
#define ROLE_CLOCK() 0ll
#define ROLE_ADD(var, t0) (void)(t0)
#endif

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
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
        "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
// Four rows of a 2-D tensor (row indices r0..r3, 64 elements from column c0) into four consecutive
// 128-byte rows of shared memory; the tensor map's box is one row high.  A row index outside the
// tensor reads as zeros.
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap *map, int c0, int4 r, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];" ::"r"(dst),
        "l"(map), "r"(c0), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_gather4_pair(uint32_t dst, const CUtensorMap *map, int c0, int4 r, uint32_t leader_bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes.cta_group::2 "
        "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];" ::"r"(dst),
        "l"(map), "r"(c0), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w), "r"(leader_bar)
        : "memory");
}
// Tile store shared -> global (clipped at the tensor's edges), tracked in the issuing thread's bulk groups
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src),
                 "r"(c0), "r"(c1)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// wait until at most N of this thread's bulk groups still READ their shared-memory source
template <int N> __device__ __forceinline__ void tma_store_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
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
// 16 lanes x 32 consecutive fp32 columns in the layout of an MMA accumulator fragment: for each
// group g of 8 columns, thread t receives row t/4, columns 8g + 2(t%4) and +1 in r[4g], r[4g+1] and
// row t/4 + 8, same columns, in r[4g+2], r[4g+3]
__device__ __forceinline__ void tmem_ld_frag16(uint32_t taddr, uint32_t *r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
          "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
// four 8x8 matrices of 16-bit elements between fragment registers and shared memory, transposed:
// thread t holds elements (row t/4, columns 2(t%4), +1) of each matrix; shared-memory row R (16
// bytes at the address given by thread 8k + R for matrix k) holds COLUMN R of the matrix
__device__ __forceinline__ void stsm_x4_trans(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a),
                 "r"(b), "r"(c), "r"(d)
                 : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t &a, uint32_t &b, uint32_t &c, uint32_t &d)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(a), "=r"(b), "=r"(c), "=r"(d)
                 : "r"(addr)
                 : "memory");
}

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
// Arrive without memory ordering.  Handing an accumulator back orders only tensor-memory reads, which
// the tcgen05 wait / fence before the arrive already does; a releasing arrive would in addition wait
// until the epilogue's outstanding global stores are visible (measured: about 2400 cycles per tile).
__device__ __forceinline__ void mbar_arrive_cluster_relaxed(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
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
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2,
                                                 uint32_t leader_bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
        "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(leader_bar)
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
    int32_t n_from_nk, k_from_nk;    // extent is the device-resident kept count
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
    int32_t sk_wait_skew;            // 0; debug handles: finishing units wait for a value nobody writes
    // grouped launch (weight gradients): up to three independent problems sharing K; problem g has
    // extents gM[g] x gN[g], operands (tmA, tmB) / (tmA2, tmB2) / (tmA3, tmB2), output gout[g]
    int32_t groups;
    int32_t gM[3], gN[3];
    void *gout[3];
    int64_t gldo[3];
    int32_t streamk;                 // 0: whole tiles only; else the least number of K-blocks per worker
                                     // that cutting the last waves along K must save to be used
    int32_t panel_sync;              // down, dX: 1 = the token tiles of a weight panel run side by side (see kernel)
    // one-instruction operand loads (see TmapSet): which of them the host could encode
    int32_t a_one, b_one;            // MN-major operand: both 64-wide slabs of a CTA's 128 in one 3-D box
    int32_t gu_one;                  // gate/up: gate and up rows in one 3-D box; 2 = the up rows come first
    int32_t dw_tma;                  // weight gradients (overwrite mode): tiles leave through TMA stores (maps O[g])
    // gate/up and dH: fetch the token operand straight from the caller's [tokens, C] array with
    // tile::gather4 loads driven by the kept-row list (map Bg) instead of from the compacted copy
    int32_t gather;
    int32_t n_rows;                  // rows of the gathered array (an index >= n_rows reads as zeros)
};

// Tensor maps of one launch.  A, B, A2, B2, A3: 2-D maps (box = 64 elements of the contiguous
// axis x 64 or 128 rows).  Bw, B2w: the same K-major B arrays with 128-row boxes, so that a CTA's
// whole half of a full-width token tile arrives with one instruction.  A1, A21, A31, B1, B21: 3-D views
// of MN-major arrays [K rows, 64-wide slab, 64 columns] whose box holds two slabs (128 columns); for
// gate/up A1 is the 3-D view [K, weight row, {gate, up}] of the two weight matrices.
// O[g]: the output matrix of weight-gradient problem g, box = 32 rows x 64 bytes, 64-byte swizzle.
struct alignas(64) TmapSet {
    CUtensorMap A, B, A2, B2, A3, Bw, B2w, A1, A21, A31, B1, B21, O[3], Bg;
};

struct alignas(8) SmemCtl {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], tmem_full[2], tmem_empty[2];
    uint64_t xfull[4], xempty[4];    // gate/up epilogue: up-warp -> gate-warp exchange, per warp pair
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
__device__ __forceinline__ unsigned short bf16_bits(float v)
{
    return __bfloat16_as_ushort(__float2bfloat16_rn(v));
}
__device__ __forceinline__ float bf16_from_bits(unsigned short b) { return __uint_as_float((uint32_t)b << 16); }

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

// Epilogue staging of the weight-gradient tiles.  A warp owns 32 accumulator rows (one per lane).
// For a 32-column bf16 chunk each lane holds its row as 16 packed words (64 B).  The rows are
// written to a 2 KiB per-warp shared-memory buffer (16-byte slots XOR-swizzled by row pair:
// conflict-free both ways), then read back so that four consecutive lanes cover one row's 64
// contiguous bytes: every global store instruction writes eight full 64-byte row segments instead
// of 32 scattered 16-byte pieces.  `my_row` is this lane's destination (row pointer at the chunk's
// first column) or null for a row that must not be written; `valid_slots` = number of 16-byte
// slots inside the column range.
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

// ---- Epilogue staging of the token problems.
// A warp owns 32 accumulator rows (weight rows) and works on chunks of 32 columns (tokens).  Its
// accumulator chunk sits in registers as two 16-row MMA fragments: r[16 hb + 4 g + 2 s + e] is row
// 16 hb + 8 s + t/4, column 8 g + 2 (t%4) + e.  The outputs are token-major ([token, weight row]),
// i.e. the transpose: one token's 32 weight rows are 64 contiguous bytes.  The transposition runs
// through a 2 KiB per-warp staging buffer laid out like the output ([32 tokens][64 bytes], 16-byte
// pieces XOR-swizzled by token pair): stmatrix / ldmatrix with .trans move whole 8x8 blocks
// between fragments and the buffer, and global memory is touched with 16-byte accesses, four
// consecutive lanes covering one token's 64 bytes.
__device__ __forceinline__ uint32_t stage_addr(uint32_t sbuf, int token, int piece)
{
    return sbuf + token * 64 + ((piece ^ ((token >> 1) & 3)) << 4);
}
// packed fragment P[8 hb + 2 g + s] = (column 8g + 2(t%4) low half, +1 high half) of row block (hb, s)
__device__ __forceinline__ void frag_to_stage(uint32_t sbuf, int lane, const uint32_t (&P)[16])
{
    const int k = lane >> 3, rr = lane & 7;
#pragma unroll
    for (int hb = 0; hb < 2; ++hb)
#pragma unroll
        for (int g0 = 0; g0 < 4; g0 += 2) {
            const int token = 8 * (g0 + (k >> 1)) + rr, piece = 2 * hb + (k & 1);
            stsm_x4_trans(stage_addr(sbuf, token, piece), P[8 * hb + 2 * g0], P[8 * hb + 2 * g0 + 1],
                          P[8 * hb + 2 * g0 + 2], P[8 * hb + 2 * g0 + 3]);
        }
}
__device__ __forceinline__ void stage_to_frag(uint32_t sbuf, int lane, uint32_t (&P)[16])
{
    const int k = lane >> 3, rr = lane & 7;
#pragma unroll
    for (int hb = 0; hb < 2; ++hb)
#pragma unroll
        for (int g0 = 0; g0 < 4; g0 += 2) {
            const int token = 8 * (g0 + (k >> 1)) + rr, piece = 2 * hb + (k & 1);
            ldsm_x4_trans(stage_addr(sbuf, token, piece), P[8 * hb + 2 * g0], P[8 * hb + 2 * g0 + 1],
                          P[8 * hb + 2 * g0 + 2], P[8 * hb + 2 * g0 + 3]);
        }
}
// Staging buffer -> global: lane L moves, for it = 0..3, the 16-byte piece L%4 of token 8 it + L/4 to
// dst[it] (this lane's address inside that token's row, or null).
__device__ __forceinline__ void stage_to_global(uint32_t sbuf, int lane, char *const (&dst)[4])
{
    __syncwarp();
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int token = it * 8 + (lane >> 2);
        uint4 v;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                     : "r"(stage_addr(sbuf, token, lane & 3))
                     : "memory");
        if (dst[it] != nullptr) *reinterpret_cast<uint4 *>(dst[it]) = v;
    }
    __syncwarp();
}
// Four 16-byte pieces per lane (as stage_to_global moves them) -> staging buffer -> fragment registers.
__device__ __forceinline__ void pieces_to_frag(uint32_t sbuf, int lane, const uint4 *v, uint32_t (&P)[16])
{
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int token = it * 8 + (lane >> 2);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage_addr(sbuf, token, lane & 3)), "r"(v[it].x),
                     "r"(v[it].y), "r"(v[it].z), "r"(v[it].w)
                     : "memory");
    }
    __syncwarp();
    stage_to_frag(sbuf, lane, P);
    __syncwarp();
}
// Global -> staging buffer (zeros where src[it] is null), then into fragment registers.
__device__ __forceinline__ void global_to_frag(uint32_t sbuf, int lane, const char *const (&src)[4], uint32_t (&P)[16])
{
    uint4 v[4];
#pragma unroll
    for (int it = 0; it < 4; ++it)
        v[it] = src[it] != nullptr ? __ldcs(reinterpret_cast<const uint4 *>(src[it])) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int token = it * 8 + (lane >> 2);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stage_addr(sbuf, token, lane & 3)), "r"(v[it].x),
                     "r"(v[it].y), "r"(v[it].z), "r"(v[it].w)
                     : "memory");
    }
    __syncwarp();
    stage_to_frag(sbuf, lane, P);
    __syncwarp();
}

// Two kinds of problems share the kernel.
//   Token problems (gate/up, down, dH, dX): the WEIGHT rows run along the accumulator rows (MMA M,
//   256 per SM pair) and the kept TOKENS along the accumulator columns (MMA N, any multiple of 16
//   up to 256), so a kept count that is not a multiple of the tile width costs at most 15 padded
//   columns instead of up to 255 padded rows.  A = weights (K-major or MN-major), B = compacted
//   token rows (K-major).  The outputs are token-major arrays [token, weight row]: for one token
//   the 32 lanes of a warp hold 32 consecutive weight rows, i.e. 64 contiguous bytes of its
//   output row, so every epilogue load / store instruction moves one full 64-byte segment.
//   Weight-gradient problems (and the plain GEMM of the token merge): both axes are weight axes,
//   K is the kept count; tiles are 256 x 256 and rows are staged through shared memory.
template <int EPI, bool A_MN, bool B_MN, bool PAIR>
__global__ void __launch_bounds__(UMMA_THREADS, 1)
k_umma_gemm(const __grid_constant__ TmapSet tm, const UmmaParams p)
{
    const CUtensorMap &tmA = tm.A, &tmB = tm.B, &tmA2 = tm.A2, &tmB2 = tm.B2, &tmA3 = tm.A3;
    constexpr bool GATEUP = (EPI == EPI_GATEUP);
    constexpr bool TOK = (EPI != EPI_DW);         // token problem: tokens on the accumulator columns
    constexpr int STAGES = Shape<PAIR>::STAGES;
    constexpr int STAGE_BYTES = Shape<PAIR>::STAGE_BYTES;
    constexpr int SPLIT = PAIR ? 2 : 1;           // CTAs sharing one tile
    constexpr int TILE_M = BM * SPLIT;            // accumulator rows of one tile
    // gate/up: each CTA's 128 rows are 64 gate rows followed by the 64 up rows of the same
    // intermediate indices, so a tile covers TILE_M / 2 indices
    constexpr int M_UNIT = GATEUP ? TILE_M / 2 : TILE_M;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t epi_bufs = tiles + STAGES * STAGE_BYTES;
    SmemCtl *ctl = reinterpret_cast<SmemCtl *>(smem_raw + (tiles - raw) + STAGES * STAGE_BYTES +
                                               EPI_WARPS * EPI_BUF_BYTES + 4 * X_BUF_BYTES);

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
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_u32(&ctl->xfull[s]), 1);
            mbar_init(smem_u32(&ctl->xempty[s]), 1);
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
    const int K = p.k_from_nk ? nk : p.K;
    // token problems: the column extent is the kept count rounded up to the MMA's N granularity;
    // columns nk .. n_tot-1 exist only as padding (their operand rows are zero)
    const int n_tot = TOK ? (p.n_from_nk ? ((nk + 15) & ~15) : p.N) : 0;
    // accumulator columns per tile: 256 unless overridden; token problems cut the token range into
    // the same number of tiles but of equal width (320 tokens: 160 + 160 instead of 256 + 64), which
    // balances the workers and avoids a sliver whose operand loads would cost as much as a full tile's
    int tile_w = p.force_bn > 0 ? p.force_bn : BN;
    if constexpr (TOK) {
        if (p.force_bn <= 0 && n_tot > 0) {
            const int n_tiles = (n_tot + BN - 1) / BN;
            tile_w = ((n_tot / 16 + n_tiles - 1) / n_tiles) * 16;
        }
    }
    // tiles of problem g: ids [g_first[g], g_first[g+1]); token problems run the column (token)
    // tile index fastest, so that tiles sharing a weight panel run at the same time
    const int groups = TOK ? 1 : p.groups;
    int g_m[3], g_n[3], g_num_m[3], g_first[4];
    g_first[0] = 0;
#pragma unroll
    for (int g = 0; g < 3; ++g) {
        g_m[g] = g < groups ? (TOK ? p.M : p.gM[g]) : 0;
        g_n[g] = g < groups ? (TOK ? n_tot : p.gN[g]) : 0;
        g_num_m[g] = (g_m[g] + M_UNIT - 1) / M_UNIT;
        g_first[g + 1] = g_first[g] + g_num_m[g] * ((g_n[g] + tile_w - 1) / tile_w);
    }
    const int num_tiles = g_first[3];
    const int num_n0 = (g_n[0] + tile_w - 1) / tile_w;
    auto pick = [](const int (&a)[3], int g) { return g == 2 ? a[2] : (g == 1 ? a[1] : a[0]); };
    struct TileLoc { int g, m0, n0, bn; };   // m0 in units of output rows (gate/up: intermediate indices)
    // Order of the tiles of one problem: `nf` tiles along the fast axis, visited in bands of `band`
    // of them; inside a band the fast index runs fastest, then the slow index.  A wave of W tiles
    // then covers about band x W/band tiles, so the operand panels it touches (band + W/band of them,
    // each K long) stay within L2 when K is large; with nf <= band it is the plain order.
    auto raster = [](int t, int nf, int ns, int band, int &f, int &sl) {
        const int per_band = band * ns;
        const int b = t / per_band, f0 = b * band;
        const int width = min(band, nf - f0);
        const int r = t - b * per_band;
        f = f0 + r % width;
        sl = r / width;
    };
    auto locate = [&](int tile) {
        TileLoc t;
        int f, sl;
        if (TOK) {   // token tiles fastest (tiles sharing a weight panel run together), in bands of 16
            t.g = 0;
            raster(tile, num_n0, g_num_m[0], 16, f, sl);
            t.m0 = sl * M_UNIT;
            t.n0 = f * tile_w;
            t.bn = min(tile_w, n_tot - t.n0);
        } else {     // weight gradients: row tiles fastest, in bands of 8
            t.g = tile >= g_first[2] ? 2 : (tile >= g_first[1] ? 1 : 0);
            const int local = tile - (t.g == 2 ? g_first[2] : (t.g == 1 ? g_first[1] : 0)), nm = pick(g_num_m, t.g);
            const int nn = (pick(g_n, t.g) + tile_w - 1) / tile_w;
            raster(local, nm, nn, 8, f, sl);
            t.m0 = f * TILE_M;
            t.n0 = sl * tile_w;
            t.bn = tile_w;
        }
        return t;
    };
    const int kb_per_seg = (K + BK - 1) / BK;
    const int num_kb = kb_per_seg * p.segments;
    const bool zero_acc = (num_kb == 0);   // empty reduction: the accumulator is exactly zero
    // Work distribution (sched.cuh).  Cutting the last waves along K costs every worker about two
    // extra epilogues (one hand-over, one finish with the slot added); it pays when the idle time it
    // removes is longer than that (p.streamk K-blocks per worker).  Few tiles with a long K (down,
    // dX at a high skip ratio): with one run per worker the token tiles that share a weight panel
    // would sit at different K offsets and read the panel at different times, each time from DRAM;
    // there the workers form groups that walk a panel's K-blocks side by side, so that a panel byte
    // is fetched from DRAM once and hit in L2 by the other members.
    Plan sched;
    if (TOK) sched.init(worker, num_workers, g_num_m[0], num_n0, num_kb, p.streamk,
                        (EPI == EPI_DOWN || EPI == EPI_DX) ? p.panel_sync : 0);
    else sched.init(worker, num_workers, num_tiles, 1, num_kb, p.streamk, 0);
    const int num_segs = sched.count();
    auto seg_at = [&](int i) { return sched.get(i); };
    // CTA slot of schedule worker q (same token tile, same CTA rank as this one)
    auto slot_cta = [&](int q) { return sched.slot_worker(q) * SPLIT + (int)rank; };
    const uint32_t nst = (p.force_stages > 0 && p.force_stages < STAGES) ? p.force_stages : STAGES;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if ((EPI == EPI_GATEUP || EPI == EPI_DH) && p.gather && !zero_acc) {
            // Gathering variant: the whole warp takes part.  Lane l fetches rows 4l .. 4l+3 of this
            // CTA's token rows with one gather4 load per K-block; lane 0 also posts the byte count and
            // loads the weight tile.
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int si = 0; ok && si < num_segs; ++si) {
                const Seg sg = seg_at(si);
                const TileLoc tl = locate(sg.tile);
                const int bn_cta = tl.bn / SPLIT;
                const int rows4 = (bn_cta + 3) >> 2;                     // gather4 loads of this CTA per K-block
                const uint32_t stage_tx = SPLIT * (A_BYTES + rows4 * 512);
                const int m0 = GATEUP ? tl.m0 + (int)rank * (BM / 2) : tl.m0 + (int)rank * BM;
                const int nb0 = tl.n0 + (int)rank * bn_cta;
                int4 rows = make_int4(p.n_rows, p.n_rows, p.n_rows, p.n_rows);
                if (lane < rows4) {
                    const int r0 = nb0 + 4 * lane;
                    if (r0 + 0 < nk) rows.x = p.idx[r0 + 0];
                    if (r0 + 1 < nk) rows.y = p.idx[r0 + 1];
                    if (r0 + 2 < nk) rows.z = p.idx[r0 + 2];
                    if (r0 + 3 < nk) rows.w = p.idx[r0 + 3];
                }
                for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
                    ok = mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1, abort_flag, p.status, SITE_PRODUCER_EMPTY);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    const int k0 = kb * BK;
                    const uint32_t own_bar = smem_u32(&ctl->full[stage]);
                    const uint32_t bar = PAIR ? mapa_rank(own_bar, 0) : own_bar;
                    const uint32_t sa = tiles + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    if (lane == 0) {
                        if (rank == 0) mbar_expect_tx(own_bar, stage_tx);
                        if (GATEUP) {
                            if (p.gu_one) {
                                if (PAIR) tma_load_3d_pair(sa, &tm.A1, k0, m0, 0, bar); else tma_load_3d(sa, &tm.A1, k0, m0, 0, bar);
                            } else {
                                if (PAIR) { tma_load_2d_pair(sa, &tmA, k0, m0, bar); tma_load_2d_pair(sa + CHUNK_BYTES, &tmA2, k0, m0, bar); }
                                else { tma_load_2d(sa, &tmA, k0, m0, bar); tma_load_2d(sa + CHUNK_BYTES, &tmA2, k0, m0, bar); }
                            }
                        } else {   // dH: the transposed weight operand in two 64-wide slabs
#pragma unroll
                            for (int j = 0; j < BM / 64; ++j) {
                                if (PAIR) tma_load_2d_pair(sa + j * CHUNK_BYTES, &tmA, m0 + 64 * j, k0, bar);
                                else tma_load_2d(sa + j * CHUNK_BYTES, &tmA, m0 + 64 * j, k0, bar);
                            }
                        }
                    }
                    if (lane < rows4) {
                        if (PAIR) tma_gather4_pair(sb + lane * 512, &tm.Bg, k0, rows, bar);
                        else tma_gather4(sb + lane * 512, &tm.Bg, k0, rows, bar);
                    }
                    if (++stage == nst) { stage = 0; phase ^= 1; }
                }
            }
        } else if (lane == 0 && !zero_acc) {
            prefetch_tmap(&tmA);
            prefetch_tmap(&tmB);
            if (p.segments == 2 || groups > 1) prefetch_tmap(&tmB2);
            if (GATEUP || p.segments == 2 || groups > 1) prefetch_tmap(&tmA2);
            if (groups > 2) prefetch_tmap(&tmA3);
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            [[maybe_unused]] long long role_a = 0;
            for (int si = 0; ok && si < num_segs; ++si) {
                const Seg sg = seg_at(si);
                const TileLoc tl = locate(sg.tile);
                const int bn_cta = tl.bn / SPLIT;          // B rows (tile columns) this CTA stages
                const int b_slabs = (bn_cta + 63) / 64;
                // bytes landing on the (leader's) full barrier per stage, from every CTA of the tile
                const uint32_t stage_tx = SPLIT * (A_BYTES + b_slabs * CHUNK_BYTES);
                const int m0 = GATEUP ? tl.m0 + (int)rank * (BM / 2) : tl.m0 + (int)rank * BM;
                const int nb0 = tl.n0 + (int)rank * bn_cta;   // first B row of this CTA
                for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
                    const long long tw = ROLE_CLOCK();
                    ok = mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1, abort_flag, p.status,
                                   SITE_PRODUCER_EMPTY);
                    ROLE_ADD(role_a, tw);
                    if (!ok) break;
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
                    auto load3 = [&](uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2) {
                        if (PAIR) tma_load_3d_pair(dst, map, c0, c1, c2, bar);
                        else tma_load_3d(dst, map, c0, c1, c2, bar);
                    };
                    if (rank == 0) mbar_expect_tx(own_bar, stage_tx);
                    if (GATEUP) {        // 64 gate rows and the 64 up rows of the same indices
                        if (p.gu_one) {
                            load3(sa, &tm.A1, k0, m0, 0);
                        } else {
                            load(sa, &tmA, k0, m0);
                            load(sa + CHUNK_BYTES, &tmA2, k0, m0);
                        }
                    } else if (A_MN) {
                        if (p.a_one) {
                            load3(sa, tl.g == 2 ? &tm.A31 : ((tl.g == 1 || seg) ? &tm.A21 : &tm.A1), 0, k0, m0 >> 6);
                        } else {
#pragma unroll
                            for (int j = 0; j < BM / 64; ++j) load(sa + j * CHUNK_BYTES, mA, m0 + 64 * j, k0);
                        }
                    } else {
                        load(sa, mA, k0, m0);
                    }
                    if (B_MN) {          // 64-column slabs of BK rows
                        if (p.b_one && bn_cta == 128) {
                            load3(sb, (tl.g >= 1 || seg) ? &tm.B21 : &tm.B1, 0, k0, nb0 >> 6);
                        } else {
                            for (int j = 0; j < b_slabs; ++j) load(sb + j * CHUNK_BYTES, mB, nb0 + 64 * j, k0);
                        }
                    } else if (TOK) {    // K-major token rows: boxes of 128 rows, then one of 64 if 64 are left
                        int j = 0;
                        for (; b_slabs - j > 1; j += 2) load(sb + j * CHUNK_BYTES, seg ? &tm.B2w : &tm.Bw, k0, nb0 + 64 * j);
                        if (j < b_slabs) load(sb + j * CHUNK_BYTES, mB, k0, nb0 + 64 * j);
                    } else {             // 64-row pieces of a K-major tile are contiguous in smem
                        for (int j = 0; j < b_slabs; ++j) load(sb + j * CHUNK_BYTES, mB, k0, nb0 + 64 * j);
                    }
                    if (++stage == nst) { stage = 0; phase ^= 1; }
                }
            }
#ifdef SKIPFFN_ROLE_CYCLES
            if (rank == 0) atomicAdd(&p.status[ST_ROLE_BASE + 8 * EPI + 3], (int)(role_a >> 4));
#endif
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && !zero_acc && rank == 0) {
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            // shared-memory descriptors of ring stage 0; a K step of 16 elements advances the address
            // field by 32 bytes (K-major) or by 16 rows of 128 bytes (MN-major)
            constexpr uint32_t KINC_A = A_MN ? (UMMA_K * 128) >> 4 : (UMMA_K * 2) >> 4;
            constexpr uint32_t KINC_B = B_MN ? (UMMA_K * 128) >> 4 : (UMMA_K * 2) >> 4;
            const uint64_t da0 = A_MN ? make_desc(tiles, CHUNK_BYTES, 1024) : make_desc(tiles, 16, 1024);
            const uint64_t db0 = B_MN ? make_desc(tiles + A_BYTES, CHUNK_BYTES, 1024) : make_desc(tiles + A_BYTES, 16, 1024);
            const int k_tail = K - (kb_per_seg - 1) * BK;   // elements in the last K-block
            const int k_steps_last = k_tail < BK ? (k_tail + UMMA_K - 1) / UMMA_K : BK / UMMA_K;
            [[maybe_unused]] long long role_full = 0, role_acc = 0;
            [[maybe_unused]] const long long role_t0 = ROLE_CLOCK();
            for (int si = 0; ok && si < num_segs; ++si) {
                const Seg sg = seg_at(si);
                const TileLoc tl = locate(sg.tile);
                const uint32_t idesc = make_idesc(A_MN ? 1 : 0, B_MN ? 1 : 0, TILE_M, tl.bn);
                const long long ta = ROLE_CLOCK();
                ok = mbar_wait(smem_u32(&ctl->tmem_empty[acc]), acc_phase ^ 1, abort_flag, p.status,
                               SITE_MMA_TMEM_EMPTY);
                ROLE_ADD(role_acc, ta);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * ACC_COLS;
                for (int kb = sg.kb0; kb < sg.kb1; ++kb) {
                    const long long tf = ROLE_CLOCK();
                    ok = mbar_wait(smem_u32(&ctl->full[stage]), phase, abort_flag, p.status,
                                   SITE_MMA_FULL);
                    ROLE_ADD(role_full, tf);
                    if (!ok) break;
                    tc_fence_after();
                    // descriptors of this stage: the ring base descriptors plus the stage offset in the
                    // 14-bit address field (shared memory ends below 256 KiB, so no carry leaves the field)
                    const uint64_t da = da0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
                    const uint64_t db = db0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
                    // A reduction over kept tokens ends inside its last K-block: rows past the
                    // count (rounded up to 16, zero up to there) hold stale data and stay unread
                    int k_steps = BK / UMMA_K;
                    if (!TOK && p.k_from_nk && kb == kb_per_seg - 1) k_steps = k_steps_last;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        if (k < k_steps) {
                            const uint32_t accumulate = (kb != sg.kb0 || k != 0);   // first MMA of a run overwrites
                            if (PAIR) umma_bf16_pair(d_tmem, da + (uint64_t)(k * KINC_A), db + (uint64_t)(k * KINC_B), idesc, accumulate);
                            else umma_bf16(d_tmem, da + (uint64_t)(k * KINC_A), db + (uint64_t)(k * KINC_B), idesc, accumulate);
                        }
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
#ifdef SKIPFFN_ROLE_CYCLES
            atomicAdd(&p.status[ST_ROLE_BASE + 8 * EPI + 0], (int)(role_full >> 4));
            atomicAdd(&p.status[ST_ROLE_BASE + 8 * EPI + 1], (int)(role_acc >> 4));
            atomicAdd(&p.status[ST_ROLE_BASE + 8 * EPI + 2], (int)((clock64() - role_t0) >> 4));
            atomicAdd(&p.status[ST_ROLE_BASE + 8 * EPI + 7], 1);
#endif
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
        [[maybe_unused]] long long role_wait = 0;
        [[maybe_unused]] const long long role_e0 = ROLE_CLOCK();
        // gate/up: warps of quarters 0, 1 hold gate rows, quarters 2, 3 the up rows of the same
        // indices; pair x = (quarter & 1) + 2 * half exchanges the up values through shared memory
        const int xpair = (quarter & 1) + 2 * half;
        const uint32_t xbuf = epi_bufs + EPI_WARPS * EPI_BUF_BYTES + xpair * X_BUF_BYTES;
        const uint32_t xfull_bar = smem_u32(&ctl->xfull[xpair]), xempty_bar = smem_u32(&ctl->xempty[xpair]);
        uint32_t xcount = 0;            // chunks exchanged so far by this warp
        uint32_t tbuf = 0;              // weight gradients: staging buffers handed to TMA stores so far
        // accumulators are handed back on the leader's barrier, which its MMA warp waits on
        const uint32_t empty_bar0 = smem_u32(&ctl->tmem_empty[0]);
        // hand-over slots: a warp reads back exactly the words the same warp of the producing CTA wrote
        const int my_slot = (int)blockIdx.x;
        auto slot_ptr = [&](int cta_slot, int j) {
            return p.sk_slots + (size_t)cta_slot * (SK_SLOT_BYTES / 16) + ((size_t)(ew * 4 + j) * 8) * 32 + lane;
        };
        for (int si = 0; ok && si < num_segs; ++si) {
            const Seg sg = seg_at(si);
            const TileLoc tl = locate(sg.tile);
            const int n0 = tl.n0, bn = tl.bn;
            if (sg.partial) {
                // ---- this run ends before the tile does: park the raw accumulator in this CTA's slot
                const long long tw = ROLE_CLOCK();
                ok = mbar_wait(smem_u32(&ctl->tmem_full[acc]), acc_phase, abort_flag, p.status,
                               SITE_EPI_TMEM_FULL);
                ROLE_ADD(role_wait, tw);
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_acc = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * ACC_COLS;
#pragma unroll 1
                for (int col = half * 32, j = 0; col < bn; col += 64, ++j) {
                    uint32_t r[32];
                    if (TOK) { tmem_ld_frag16(t_acc + col, r); tmem_ld_frag16(t_acc + (16u << 16) + col, r + 16); }
                    else tmem_ld32(t_acc + col, r);
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
            // this lane's output row: a weight row of the problem (token problems) or a row of the
            // weight gradient
            const bool is_up = GATEUP && ((quarter >= 2) != (p.gu_one == 2));
            const int m = GATEUP ? tl.m0 + (int)rank * (BM / 2) + (quarter & 1) * 32 + lane
                                 : tl.m0 + (int)rank * BM + row_in_tile;
            const bool row_valid = m < pick(g_m, tl.g);
            const int n_end = TOK ? n0 + bn : min(n0 + bn, pick(g_n, tl.g));
            // token problems: 16-byte pieces, lane moves piece lane%4 (8 weight rows) of tokens 8 it + lane/4
            const int m_warp = m - lane;                  // first weight row of this warp
            const bool piece_ok = m_warp + 8 * (lane & 3) < pick(g_m, tl.g);
            const int64_t piece_off = (int64_t)m_warp + 8 * (lane & 3);
            // down, dX: the epilogue's own global inputs (residual rows, scatter indices) are requested
            // one chunk ahead -- for a tile's first chunk before the accumulator is even waited for --
            // so their latency overlaps the tensor-memory loads and the arithmetic of the chunk before
            // (down -2.3 %, dX -1.7 %; the same for G and U in dH ran out of registers: +4 %).
            constexpr bool PRE = TOK && (EPI == EPI_DOWN || EPI == EPI_DX);
            [[maybe_unused]] uint4 pre[4];
            [[maybe_unused]] int pre_idx[4];
            auto issue_pre = [&](int nc) {
                if constexpr (PRE) {
                    if (EPI == EPI_DX && p.out_fp32) return;
                    const int real_c = max(0, min(min(32, n_end - nc), nk - nc));
#pragma unroll
                    for (int it = 0; it < 4; ++it) {
                        const int tok = it * 8 + (lane >> 2);
                        const bool v = tok < real_c && piece_ok;
                        const int64_t off = ((int64_t)(nc + tok) * p.ldo + piece_off) * 2;
                        pre[it] = v ? __ldcs(reinterpret_cast<const uint4 *>((const char *)p.in0 + off)) : make_uint4(0, 0, 0, 0);
                        pre_idx[it] = v ? p.idx[nc + tok] : 0;
                    }
                }
            };
            if (n0 + half * 32 < n_end) issue_pre(n0 + half * 32);
            if (!zero_acc) {
                const long long tw = ROLE_CLOCK();
                ok = mbar_wait(smem_u32(&ctl->tmem_full[acc]), acc_phase, abort_flag, p.status,
                               SITE_EPI_TMEM_FULL);
                ROLE_ADD(role_wait, tw);
                if (!ok) break;
                tc_fence_after();
            }
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * ACC_COLS;
            if (add_slots) {
                // the rest of this tile's K range sits in the slots of workers src_lo .. worker-1
                for (int q = sg.src_lo; ok && q < sched.self(); ++q) {
                    if (!sched.had_run(q)) continue;
                    ok = flag_wait(p.sk_flags + slot_cta(q) * SK_FLAGS_PER_CTA + ew,
                                   p.sk_epoch + p.sk_wait_skew, lane, abort_flag, p.status);
                }
                if (!ok) break;
            }

#pragma unroll 1
            for (int n = n0 + half * 32; n < n_end; n += 64) {
                const int col = n - n0;
                uint32_t r[32];
                if (!zero_acc) {
                    if (TOK) { tmem_ld_frag16(t_row + col, r); tmem_ld_frag16(t_row + (16u << 16) + col, r + 16); }
                    else tmem_ld32(t_row + col, r);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int q = 0; q < 32; ++q) r[q] = 0u;
                }
                if (add_slots) {
                    const int j = col >> 6;   // this warp's j-th 32-column chunk of the accumulator
                    for (int q = sg.src_lo; q < sched.self(); ++q) {
                        if (!sched.had_run(q)) continue;
                        const float4 *src = slot_ptr(slot_cta(q), j);
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            const float4 a = __ldcg(src + v * 32);
                            r[4 * v] = __float_as_uint(__uint_as_float(r[4 * v]) + a.x);
                            r[4 * v + 1] = __float_as_uint(__uint_as_float(r[4 * v + 1]) + a.y);
                            r[4 * v + 2] = __float_as_uint(__uint_as_float(r[4 * v + 2]) + a.z);
                            r[4 * v + 3] = __float_as_uint(__uint_as_float(r[4 * v + 3]) + a.w);
                        }
                    }
                }
                if (TOK) {
                    // ---- token problems: column c of the chunk is token n + c.  Tokens below nk are
                    // real; tokens nk .. n_end-1 are the padding of the last tile (stored as zeros
                    // where a later reduction over tokens reads them).  r[] is in fragment layout:
                    // r[16 hb + 4 g + 2 s + e] = row 16 hb + 8 s + lane/4, column 8 g + 2 (lane%4) + e.
                    const int cols = min(32, n_end - n);          // columns of this chunk inside the tile
                    const int real = max(0, min(cols, nk - n));   // of which real tokens
                    const int fc = (lane & 3) * 2;                // this thread's first column in a group of 8
                    auto tok_of = [&](int it) { return it * 8 + (lane >> 2); };
                    // zero the accumulator columns that are padding (so every derived value is zero)
                    if (real < cols) {
#pragma unroll
                        for (int q = 0; q < 32; ++q)
                            if (8 * ((q >> 2) & 3) + fc + (q & 1) >= real) r[q] = 0u;
                    }
                    if (EPI == EPI_GATEUP) {
                        char *dst[4];
                        const uint32_t xslot = xbuf + lane * 16;
                        if (is_up) {
                            // hand the fp32 up values to the gate warp (same fragment layout there), then store U
                            ok = mbar_wait(xempty_bar, (xcount & 1) ^ 1, abort_flag, p.status, SITE_EPI_EXCHANGE);
                            if (!ok) break;
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(xslot + v * 512), "r"(r[4 * v]),
                                             "r"(r[4 * v + 1]), "r"(r[4 * v + 2]), "r"(r[4 * v + 3])
                                             : "memory");
                            __syncwarp();
                            if (lane == 0) mbar_arrive(xfull_bar);
                            if (p.out1 != nullptr) {
                                uint32_t P[16];
#pragma unroll
                                for (int q = 0; q < 16; ++q) P[q] = pack_bf16(__uint_as_float(r[2 * q]), __uint_as_float(r[2 * q + 1]));
                                frag_to_stage(sbuf, lane, P);
#pragma unroll
                                for (int it = 0; it < 4; ++it)
                                    dst[it] = (tok_of(it) < cols && piece_ok)
                                                  ? (char *)((bf16 *)p.out1 + (int64_t)(n + tok_of(it)) * p.ldo + piece_off) : nullptr;
                                stage_to_global(sbuf, lane, dst);
                            }
                        } else {
                            ok = mbar_wait(xfull_bar, xcount & 1, abort_flag, p.status, SITE_EPI_EXCHANGE);
                            if (!ok) break;
                            uint32_t u[32];
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                             : "=r"(u[4 * v]), "=r"(u[4 * v + 1]), "=r"(u[4 * v + 2]), "=r"(u[4 * v + 3])
                                             : "r"(xslot + v * 512)
                                             : "memory");
                            __syncwarp();
                            if (lane == 0) mbar_arrive(xempty_bar);
                            uint32_t P[16];
                            if (p.out0 != nullptr) {
#pragma unroll
                                for (int q = 0; q < 16; ++q) P[q] = pack_bf16(__uint_as_float(r[2 * q]), __uint_as_float(r[2 * q + 1]));
                                frag_to_stage(sbuf, lane, P);
#pragma unroll
                                for (int it = 0; it < 4; ++it)
                                    dst[it] = (tok_of(it) < cols && piece_ok)
                                                  ? (char *)((bf16 *)p.out0 + (int64_t)(n + tok_of(it)) * p.ldo + piece_off) : nullptr;
                                stage_to_global(sbuf, lane, dst);
                            }
#pragma unroll
                            for (int q = 0; q < 16; ++q)
                                P[q] = pack_bf16(fast_swiglu(__uint_as_float(r[2 * q]), __uint_as_float(u[2 * q])),
                                                 fast_swiglu(__uint_as_float(r[2 * q + 1]), __uint_as_float(u[2 * q + 1])));
                            frag_to_stage(sbuf, lane, P);
#pragma unroll
                            for (int it = 0; it < 4; ++it)
                                dst[it] = (tok_of(it) < cols && piece_ok)
                                              ? (char *)((bf16 *)p.out2 + (int64_t)(n + tok_of(it)) * p.ldo + piece_off) : nullptr;
                            stage_to_global(sbuf, lane, dst);
                        }
                        ++xcount;
                    } else if (EPI == EPI_DX && p.out_fp32) {
                        // pre-norm variant: the raw fp32 gradient w.r.t. the normalised rows, compact,
                        // no residual (the normalisation's backward runs afterwards, row-wide); two
                        // consecutive tokens per thread, 4-byte stores
                        float *Y = (float *)p.out0 + (int64_t)n * p.ldo + m_warp;
#pragma unroll
                        for (int q = 0; q < 32; ++q) {
                            const int row = 16 * (q >> 4) + 8 * ((q >> 1) & 1) + (lane >> 2);
                            const int c = 8 * ((q >> 2) & 3) + fc + (q & 1);
                            if (c < real && m_warp + row < pick(g_m, tl.g)) Y[(int64_t)c * p.ldo + row] = __uint_as_float(r[q]);
                        }
                    } else if (EPI == EPI_DOWN || EPI == EPI_DX) {
                        // residual add in fp32, one rounding, scatter to the token's row
                        char *dst[4];
#pragma unroll
                        for (int it = 0; it < 4; ++it) {
                            const bool v = tok_of(it) < real && piece_ok;
                            dst[it] = v ? (char *)((bf16 *)p.out0 + (int64_t)pre_idx[it] * p.ldo + piece_off) : nullptr;
                        }
                        uint32_t R[16], P[16];
                        pieces_to_frag(sbuf, lane, pre, R);
                        if (n + 64 < n_end) issue_pre(n + 64);
#pragma unroll
                        for (int q = 0; q < 16; ++q) {
                            float a0, a1;
                            unpack_bf16(R[q], a0, a1);
                            P[q] = pack_bf16(a0 + __uint_as_float(r[2 * q]), a1 + __uint_as_float(r[2 * q + 1]));
                        }
                        frag_to_stage(sbuf, lane, P);
                        stage_to_global(sbuf, lane, dst);
                    } else if (EPI == EPI_DH) {
                        const char *src[4];
                        char *dst[4];
                        int64_t off[4];
#pragma unroll
                        for (int it = 0; it < 4; ++it) off[it] = ((int64_t)(n + tok_of(it)) * p.ldo + piece_off) * 2;
                        uint32_t Gf[16], Uf[16], P[16], Q[16];
#pragma unroll
                        for (int it = 0; it < 4; ++it) src[it] = (tok_of(it) < real && piece_ok) ? (const char *)p.in0 + off[it] : nullptr;
                        global_to_frag(sbuf, lane, src, Gf);
#pragma unroll
                        for (int it = 0; it < 4; ++it) src[it] = (tok_of(it) < real && piece_ok) ? (const char *)p.in1 + off[it] : nullptr;
                        global_to_frag(sbuf, lane, src, Uf);
#pragma unroll
                        for (int q = 0; q < 16; ++q) {
                            float g0, g1, u0, u1, dg0, dg1, du0, du1;
                            unpack_bf16(Gf[q], g0, g1);
                            unpack_bf16(Uf[q], u0, u1);
                            fast_swiglu_bwd(__uint_as_float(r[2 * q]), g0, u0, dg0, du0);
                            fast_swiglu_bwd(__uint_as_float(r[2 * q + 1]), g1, u1, dg1, du1);
                            P[q] = pack_bf16(dg0, dg1);
                            Q[q] = pack_bf16(du0, du1);
                        }
                        frag_to_stage(sbuf, lane, P);
#pragma unroll
                        for (int it = 0; it < 4; ++it) dst[it] = (tok_of(it) < cols && piece_ok) ? (char *)p.out0 + off[it] : nullptr;
                        stage_to_global(sbuf, lane, dst);
                        frag_to_stage(sbuf, lane, Q);
#pragma unroll
                        for (int it = 0; it < 4; ++it) dst[it] = (tok_of(it) < cols && piece_ok) ? (char *)p.out1 + off[it] : nullptr;
                        stage_to_global(sbuf, lane, dst);
                    }
                } else {
                    // ---- weight-gradient tile, overwrite or accumulate
                    const int valid_slots = min(4, (n_end - n) / 8);
                    uint32_t w[16];
                    const int64_t o = (int64_t)m * p.gldo[tl.g] + n;
                    char *row = row_valid ? (char *)p.gout[tl.g] + o * esz : nullptr;
                    if (p.dw_tma) {
                        // overwrite mode: the 32-row x 64-byte chunk is staged (same XOR layout as the
                        // 64-byte TMA swizzle) and leaves as one tile store, which also clips at the
                        // matrix edges; two staging buffers per warp, so a store still reading one of
                        // them overlaps the next chunk
                        const CUtensorMap *mo = tl.g == 2 ? &tm.O[2] : (tl.g == 1 ? &tm.O[1] : &tm.O[0]);
                        const int m_warp = m - lane;
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            if (!p.out_fp32 && hh == 1) break;
                            if (p.out_fp32) {
#pragma unroll
                                for (int q = 0; q < 16; ++q) w[q] = r[hh * 16 + q];
                            } else {
#pragma unroll
                                for (int q = 0; q < 16; ++q) w[q] = pack_bf16(__uint_as_float(r[2 * q]), __uint_as_float(r[2 * q + 1]));
                            }
                            const uint32_t sb2 = (tbuf & 1) ? sbuf + EPI_WARPS * EPI_BUF_BYTES : sbuf;
                            ++tbuf;
                            if (lane == 0) tma_store_wait_read<1>();   // the store that last used this buffer has read it
                            __syncwarp();
                            const int sw = (lane >> 1) & 3;
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sb2 + lane * 64 + ((c ^ sw) << 4)),
                                             "r"(w[4 * c]), "r"(w[4 * c + 1]), "r"(w[4 * c + 2]), "r"(w[4 * c + 3])
                                             : "memory");
                            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                            __syncwarp();
                            if (lane == 0) {
                                tma_store_2d(mo, sb2, n + hh * 16, m_warp);
                                tma_store_commit();
                            }
                        }
                    } else if (p.out_fp32) {
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
            if (!ok) break;
            if (add_slots && lane == 0) {
                // this warp has consumed the hand-overs of the tile: clear their flags, so that a replay
                // of the launch with the same flag value (a captured graph) never takes an old flag for
                // a new one
                for (int q = sg.src_lo; q < sched.self(); ++q)
                    if (sched.had_run(q)) p.sk_flags[slot_cta(q) * SK_FLAGS_PER_CTA + ew] = 0;
            }
            if (!zero_acc) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    const uint32_t bar = empty_bar0 + acc * 8;
                    if (PAIR) mbar_arrive_cluster_relaxed(mapa_rank(bar, 0));
                    else mbar_arrive(bar);
                }
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        if (!TOK && lane == 0) tma_store_wait_read<0>();   // the staging buffers are free before the CTA gives them up
#ifdef SKIPFFN_ROLE_CYCLES
        if (ew == 0 && lane == 0 && rank == 0) {
            atomicAdd(&p.status[ST_ROLE_BASE + 8 * EPI + 4], (int)(role_wait >> 4));
            atomicAdd(&p.status[ST_ROLE_BASE + 8 * EPI + 5], (int)((clock64() - role_e0 - role_wait) >> 4));
        }
#endif
    }

    // ---------------------------------------------------------------------- teardown
    // After a wait ran out, copies or MMAs of this CTA may still be in flight: give them time to
    // land (bounded) before the shared and tensor memory they target is given up.
    if (*abort_flag) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
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
// Out-of-range parts of a box read as zero.  With dim2 > 0 the map has a third, outermost
// dimension of dim2 entries `stride2_bytes` apart (which may be smaller than the row pitch: the
// 64-column slabs of an MN-major array) and the box spans two of them.  Encoded maps are kept in
// the caller's cache (a handle sees the same few arrays call after call), looked up by every field
// that enters the map.
static_assert(sizeof(CUtensorMap) == TMAP_BYTES, "tensor map size");
static bool make_map(CUtensorMap *m, TmapCache *cache, const void *base, int64_t inner, int64_t outer,
                     int64_t pitch, int box_outer, int64_t dim2 = 0, int64_t stride2_bytes = 0)
{
    if (!base) return false;
    if (cache) {
        for (int i = 0; i < cache->used; ++i) {
            const TmapKey &k = cache->key[i];
            if (k.base == base && k.inner == inner && k.outer == outer && k.pitch == pitch && k.box_outer == box_outer &&
                k.dim2 == dim2 && k.stride2 == stride2_bytes) {
                memcpy(m, cache->map[i], TMAP_BYTES);
                return true;
            }
        }
    }
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)dim2};
    cuuint64_t strides[2] = {(cuuint64_t)pitch * 2, (cuuint64_t)stride2_bytes};
    cuuint32_t box[3] = {64u, (cuuint32_t)box_outer, 2u};
    cuuint32_t es[3] = {1u, 1u, 1u};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, dim2 > 0 ? 3 : 2, const_cast<void *>(base), dims, strides,
                     box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (cache) {
        const int i = cache->used < TMAP_CACHE_ENTRIES ? cache->used++ : (cache->next++ % TMAP_CACHE_ENTRIES);
        cache->key[i] = TmapKey{base, inner, outer, pitch, box_outer, dim2, stride2_bytes};
        memcpy(cache->map[i], m, TMAP_BYTES);
    }
    return true;
}

// Output matrix of a weight-gradient problem for TMA tile stores: row-major [rows, cols] with row
// pitch `pitch` elements of 2 or 4 bytes; box = 32 rows x 64 bytes, 64-byte swizzle (the layout of the
// epilogue's staging buffers).
static bool make_out_map(CUtensorMap *m, TmapCache *cache, const void *base, int64_t rows, int64_t cols, int64_t pitch,
                         bool fp32)
{
    if (!base) return false;
    const int kind = fp32 ? -2 : -1;   // kept apart from operand maps in the cache
    if (cache) {
        for (int i = 0; i < cache->used; ++i) {
            const TmapKey &k = cache->key[i];
            if (k.base == base && k.inner == cols && k.outer == rows && k.pitch == pitch && k.box_outer == 32 && k.dim2 == kind) {
                memcpy(m, cache->map[i], TMAP_BYTES);
                return true;
            }
        }
    }
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const int esz = fp32 ? 4 : 2;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)pitch * esz};
    cuuint32_t box[2] = {(cuuint32_t)(64 / esz), 32u};
    cuuint32_t es[2] = {1u, 1u};
    CUresult r = enc(m, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                     const_cast<void *>(base), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (cache) {
        const int i = cache->used < TMAP_CACHE_ENTRIES ? cache->used++ : (cache->next++ % TMAP_CACHE_ENTRIES);
        cache->key[i] = TmapKey{base, cols, rows, pitch, 32, kind, 0};
        memcpy(cache->map[i], m, TMAP_BYTES);
    }
    return true;
}

// What the launch code has to know about a device, looked up once per device.
constexpr int MAX_DEVICES = 64;
struct DeviceInfo { int num_sms; };
static DeviceInfo g_dev[MAX_DEVICES];
// Process-wide switches, read from the environment once: SKIPFFN_PDL=0 launches without
// programmatic dependent launch; SKIPFFN_SINGLE_CTA=1 selects the one-CTA-per-tile shape.
struct Switches { int pdl, single; };
static const Switches &switches()
{
    static const Switches sw = [] {
        Switches v;
        const char *e = getenv("SKIPFFN_PDL");
        v.pdl = (e && atoi(e) == 0) ? 0 : 1;
        e = getenv("SKIPFFN_SINGLE_CTA");
        v.single = (e && atoi(e) != 0) ? 1 : 0;
        return v;
    }();
    return sw;
}

// Launch one instantiation.  PAIR kernels run as clusters of two CTAs; `workers` counts tiles
// processed concurrently (CTAs, or CTA pairs).
template <int EPI, bool A_MN, bool B_MN, bool PAIR>
static cudaError_t launch_k(int dev, const TmapSet &tm, const UmmaParams &p, int64_t max_tiles, cudaStream_t s)
{
    constexpr int SMEM = Shape<PAIR>::SMEM_BYTES;
    static int max_workers_p1[MAX_DEVICES];   // per device: 0 not yet queried, else workers + 1
    auto kern = k_umma_gemm<EPI, A_MN, B_MN, PAIR>;
    if (max_workers_p1[dev] == 0) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
        if (e != cudaSuccess) return e;
        int n = g_dev[dev].num_sms;
        if (PAIR) {
            cudaLaunchConfig_t q = {};
            q.gridDim = dim3(2 * g_dev[dev].num_sms);
            q.blockDim = dim3(UMMA_THREADS);
            q.dynamicSmemBytes = SMEM;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            q.attrs = at; q.numAttrs = 1;
            e = cudaOccupancyMaxActiveClusters(&n, kern, &q);
            if (e != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
        }
        max_workers_p1[dev] = n + 1;
    }
    const int max_workers = max_workers_p1[dev] - 1;
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
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = switches().pdl ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kern, tm, p);
}

template <bool PAIR>
static cudaError_t dispatch(int dev, int epi, const TmapSet &tm, const UmmaParams &p, int64_t max_tiles, cudaStream_t s)
{
    switch (epi) {
    case EPI_GATEUP: return launch_k<EPI_GATEUP, false, false, PAIR>(dev, tm, p, max_tiles, s);
    case EPI_DOWN:   return launch_k<EPI_DOWN, false, false, PAIR>(dev, tm, p, max_tiles, s);
    case EPI_DH:     return launch_k<EPI_DH, true, false, PAIR>(dev, tm, p, max_tiles, s);
    case EPI_DW:     return launch_k<EPI_DW, true, true, PAIR>(dev, tm, p, max_tiles, s);
    case EPI_DX:     return launch_k<EPI_DX, true, false, PAIR>(dev, tm, p, max_tiles, s);
    case EPI_PLAIN:  return launch_k<EPI_DW, false, false, PAIR>(dev, tm, p, max_tiles, s);
    default: return cudaErrorInvalidValue;
    }
}

// GemmArgs conventions: C[m, n] = sum_k A(m, k) * B(n, k).  An operand with ld_k == 1 is K-major
// ([outer = M or N rows, inner = K]), otherwise MN-major with ld_mn == 1 ([outer = K rows, inner =
// M or N]).  a_outer / b_outer give the number of addressable rows of each array.
// Token problems (gate/up, down, dH, dX) arrive with the WEIGHTS as A (M = weight rows) and the
// compacted token rows as B (N = token bound, the device-resident kept count when n_from_nk);
// their outputs and epilogue inputs are token-major arrays [token, ldo].  gate/up: A = W_gate,
// A2 = W_up.  dX: second K segment A2 = W_up, B2 = dU.
// `n` > 1 (weight gradients only): up to three independent problems with the same K in one launch;
// problems 1 and 2 share their B operand.
static cudaError_t launch_problems(int epi, const GemmArgs *gs, int n, cudaStream_t s)
{
    if (n < 1 || n > 3 || (n > 1 && epi != EPI_DW) || epi < 0 || epi > EPI_PLAIN) return cudaErrorInvalidValue;
    if (n == 3 && (gs[2].B != gs[1].B || gs[2].ldb_k != gs[1].ldb_k || gs[2].N != gs[1].N))
        return cudaErrorInvalidValue;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    if (g_dev[dev].num_sms == 0) {
        e = cudaDeviceGetAttribute(&g_dev[dev].num_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
    }
    const GemmArgs &g = gs[0];
    const bool gateup = epi == EPI_GATEUP;
    const bool tok = epi != EPI_DW && epi != EPI_PLAIN;
    TmapSet tm;
    bool ok = true;
    auto mk = [&](CUtensorMap *m, const GemmArgs &q, const void *base, bool is_a) {
        const int64_t ld_mn = is_a ? q.lda_m : q.ldb_n, ld_k = is_a ? q.lda_k : q.ldb_k;
        const int64_t outer = is_a ? q.a_outer : q.b_outer;
        if (ld_k != 1) return make_map(m, q.tmaps, base, is_a ? q.M : q.N, outer, ld_k, BK);   // MN-major
        // K-major: A arrives in one box of 128 rows (gate/up: 64 gate + 64 up rows), B in 64-row pieces
        return make_map(m, q.tmaps, base, (int64_t)q.K, outer, ld_mn, is_a ? (gateup ? BM / 2 : BM) : 64);
    };
    // 3-D view of an MN-major array: [K rows][extent / 64 slabs][64 columns]; only when the slabs tile
    // the extent exactly (a ragged last slab would reach into the next row)
    auto mk_slabs = [&](CUtensorMap *m, const GemmArgs &q, const void *base, bool is_a) {
        const int64_t ext = is_a ? q.M : q.N, ld_k = is_a ? q.lda_k : q.ldb_k, outer = is_a ? q.a_outer : q.b_outer;
        if (ld_k == 1 || ext % 64 != 0) return false;
        return make_map(m, q.tmaps, base, 64, outer, ld_k, BK, ext / 64, 128);
    };
    ok &= mk(&tm.A, g, g.A, true);
    ok &= mk(&tm.B, g, g.B, false);
    if (n > 1) {
        ok &= mk(&tm.A2, gs[1], gs[1].A, true);
        ok &= mk(&tm.B2, gs[1], gs[1].B, false);
    } else {
        if (g.A2) ok &= mk(&tm.A2, g, g.A2, true); else tm.A2 = tm.A;
        if (g.B2) ok &= mk(&tm.B2, g, g.B2, false); else tm.B2 = tm.B;
    }
    if (n > 2) ok &= mk(&tm.A3, gs[2], gs[2].A, true); else tm.A3 = tm.A;
    if (!ok) return cudaErrorInvalidValue;
    tm.Bw = tm.B; tm.B2w = tm.B2;
    tm.A1 = tm.A; tm.A21 = tm.A2; tm.A31 = tm.A3; tm.B1 = tm.B; tm.B21 = tm.B2;
    int a_one = 0, b_one = 0, gu_one = 0;
    if (tok) {   // token rows (K-major B) in 128-row boxes
        ok &= make_map(&tm.Bw, g.tmaps, g.B, (int64_t)g.K, g.b_outer, g.ldb_n, 128);
        if (g.B2) ok &= make_map(&tm.B2w, g.tmaps, g.B2, (int64_t)g.K, g.b_outer, g.ldb_n, 128); else tm.B2w = tm.Bw;
        if (!ok) return cudaErrorInvalidValue;
    }
    if (g.one_box_loads) {
        if (gateup) {   // gate and up rows as the two entries of a third dimension
            const char *lo = (const char *)g.A, *hi = (const char *)g.A2;
            gu_one = 1;
            if (hi < lo) { const char *t = lo; lo = hi; hi = t; gu_one = 2; }
            const int64_t delta = hi - lo;
            if (delta <= 0 || delta % 16 != 0 || delta >= ((int64_t)1 << 40) ||
                !make_map(&tm.A1, g.tmaps, lo, (int64_t)g.K, g.a_outer, g.lda_m, BM / 2, 2, delta))
                gu_one = 0;
        } else if (g.lda_k != 1) {
            // (measured: weight gradients -6 %, dH -6 %, dX -4 % against one box per slab)
            a_one = mk_slabs(&tm.A1, g, g.A, true) ? 1 : 0;
            if (a_one && n > 1) a_one = mk_slabs(&tm.A21, gs[1], gs[1].A, true) ? 1 : 0;
            if (a_one && n == 1 && g.A2) a_one = mk_slabs(&tm.A21, g, g.A2, true) ? 1 : 0;
            if (a_one && n > 2) a_one = mk_slabs(&tm.A31, gs[2], gs[2].A, true) ? 1 : 0;
        }
        if (g.ldb_k != 1) {
            b_one = mk_slabs(&tm.B1, g, g.B, false) ? 1 : 0;
            if (b_one && n > 1) b_one = mk_slabs(&tm.B21, gs[1], gs[1].B, false) ? 1 : 0;
        }
    }

    UmmaParams p;
    p.M = g.M; p.N = g.N; p.K = g.K;
    p.n_from_nk = g.n_from_nk; p.k_from_nk = g.k_from_nk;
    p.segments = epi == EPI_DX ? 2 : 1;
    p.force_stages = g.tune_stages > 0 ? g.tune_stages : 0;
    // tile width override: any multiple of 16 for token problems, of 32 for the weight gradients
    p.force_bn = 0;
    if (g.tune_tile_n >= 32 && g.tune_tile_n <= BN && g.tune_tile_n % (tok ? 16 : 32) == 0) p.force_bn = g.tune_tile_n;
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
    p.sk_wait_skew = g.sk_wait_skew;
    p.a_one = a_one; p.b_one = b_one; p.gu_one = gu_one;
    // gate/up, dH: token rows gathered from the caller's array by the kept-row list (SM-pair shape only)
    p.gather = 0; p.n_rows = 0;
    tm.Bg = tm.B;
    if ((epi == EPI_GATEUP || epi == EPI_DH) && g.gather_src && g.idx &&
        make_map(&tm.Bg, g.tmaps, g.gather_src, (int64_t)g.K, g.gather_rows, g.ldb_n, 1)) {
        p.gather = 1; p.n_rows = (int32_t)g.gather_rows;
    }
    // weight gradients that overwrite their destination leave through TMA tile stores
    p.dw_tma = 0;
    tm.O[0] = tm.O[1] = tm.O[2] = tm.A;
    if (!tok && !g.accumulate && g.tma_stores) {
        p.dw_tma = 1;
        for (int i = 0; i < n && p.dw_tma; ++i)
            if (!make_out_map(&tm.O[i], gs[i].tmaps, gs[i].out0, gs[i].M, gs[i].N, gs[i].ldo, gs[i].out_fp32 != 0)) p.dw_tma = 0;
    }
    // K-blocks of main loop (about 512 cycles each) that two extra epilogues of this kind cost
    static const int sk_threshold[6] = {/*GATEUP*/ 16, /*DOWN*/ 40, /*DH*/ 48, /*DW*/ 64, /*DX*/ 40, /*PLAIN*/ 32};
    p.streamk = (g.sk_slots && g.sk_flags) ? (g.tune_streamk >= 0 ? g.tune_streamk : sk_threshold[epi]) : 0;
    p.panel_sync = g.tune_panel_sync < 0 ? 1 : g.tune_panel_sync;

    const int tile_w = p.force_bn > 0 ? p.force_bn : BN;   // accumulator columns per tile
    // with K splitting a tile can be shared by several workers: allow one worker per 4 K-blocks
    const int64_t kb = ((int64_t)g.K + BK - 1) / BK * p.segments;
    const int64_t per_tile = p.streamk ? (kb >= 8 ? kb / 4 : 1) : 1;
    auto max_items = [&](int tile_m) {
        int64_t t = 0;
        const int m_unit = gateup ? tile_m / 2 : tile_m;
        for (int i = 0; i < n; ++i) {
            const int64_t cols = tok ? (((int64_t)gs[i].N + 15) & ~(int64_t)15) : (int64_t)gs[i].N;
            t += (((int64_t)gs[i].M + m_unit - 1) / m_unit) * ((cols + tile_w - 1) / tile_w);
        }
        return t * per_tile;
    };
    // SM pairs by default; the one-CTA-per-tile shape when asked for or when the device cannot
    // co-schedule pairs
    static int no_pairs[MAX_DEVICES];
    if (!switches().single && !no_pairs[dev]) {
        e = dispatch<true>(dev, epi, tm, p, max_items(2 * BM), s);
        if (e != cudaErrorNotSupported) return e;
        (void)cudaGetLastError();
        no_pairs[dev] = 1;
    }
    p.gather = 0;   // the one-CTA shape stages up to 256 token rows per CTA: compacted copy only
    return dispatch<false>(dev, epi, tm, p, max_items(BM), s);
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
