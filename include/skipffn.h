/*
 * skipffn.h -- C ABI of libskipffn: the Skip-FFN decoder sublayer on NVIDIA B200 (sm_100a).
 *
 * Operation (paper section 4.2, "Training speed-up: skip FFN"):
 *     retained / text tokens  (Eq. 4):   out[t] = x[t] + FFN(x[t])
 *     skipped visual tokens   (Eq. 5):   out[t] = x[t]                    (exact identity)
 * with the bias-free SwiGLU feed-forward network of the paper's LLaMA-3 / Vicuna backbones
 * (three C x I matrices; section 6.2 cost model 3*N*C*M and Table 1):
 *     FFN(x) = ( silu(x W_gate^T) * (x W_up^T) ) W_down^T ,   silu(z) = z * sigmoid(z).
 * The backward pass is the exact vector-Jacobian product of that definition: skipped rows
 * pass dout through unchanged, kept rows add the FFN's vjp, and the weight gradients are sums
 * over kept rows only.
 *
 * Conventions common to every entry point
 *   - Every tensor pointer is a DEVICE pointer owned by the caller; tensors are contiguous and
 *     row-major, base addresses 16-byte aligned.  The library allocates no device memory, never
 *     synchronises the stream and never aborts: every problem is reported as a status code.
 *   - x, out, dout, dx : [N, C] with N = B*S tokens;  skip_mask : [N] bytes, nonzero = skipped.
 *   - W_gate, W_up : [I, C];  W_down : [C, I]   (out_features x in_features).
 *   - Element type is cfg.dtype (bf16: fp32 accumulation on tensor cores; fp32: plain FMA).
 *   - C and I must be multiples of 8, else SKIPFFN_EUNSUPPORTED.
 *   - All work is enqueued on `stream`; the kept-token count stays on the device.
 *   - Device-side problems (a pipeline wait that exceeded its limit) set a status word in the
 *     workspace; the kernel then exits normally and skipffn_poll reports it.
 *   - Stream capture: skipffn_plan, skipffn_forward and skipffn_backward only enqueue kernels and
 *     asynchronous memsets on `stream`, so a forward + backward may be captured into a CUDA graph
 *     after one un-captured call of the same sequence on the same handle (which does the one-time
 *     work: kernel attributes, tensor-map encoding, clearing the status block).  A replay repeats
 *     the captured kernel arguments, including the buffers the capture was given, and gives the
 *     bits of the un-captured call; skipffn_poll and skipffn_profile_read synchronise and stay
 *     outside a capture.
 */
#ifndef SKIPFFN_H_
#define SKIPFFN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SKIPFFN_OK = 0,
    SKIPFFN_EINVAL = 1,       /* null pointer, bad shape, misaligned pointer, forward missing */
    SKIPFFN_EUNSUPPORTED = 2, /* shape outside what the kernels handle */
    SKIPFFN_EWORKSPACE = 3,   /* workspace too small for max_tokens / max_kept; reported by skipffn_poll
                                 when a mask kept more than max_kept tokens */
    SKIPFFN_ECUDA = 4,        /* a CUDA runtime / driver call failed */
    SKIPFFN_ETIMEOUT = 5,     /* a device-side wait hit its limit (reported by skipffn_poll) */
    SKIPFFN_EDEBUG = 6        /* debug handles: a device-side consistency check failed (skipffn_poll) */
} skipffn_status;

typedef enum { SKIPFFN_BF16 = 0, SKIPFFN_FP32 = 1 } skipffn_dtype;

/* Which kernels serve the GEMMs.  DEFAULT: tcgen05 tensor-core kernels for bf16, plain-FMA
 * kernels for fp32.  SIMT: plain-FMA kernels for either dtype (an on-device second opinion). */
typedef enum { SKIPFFN_PATH_DEFAULT = 0, SKIPFFN_PATH_SIMT = 1 } skipffn_path;

typedef struct {
    int32_t C;               /* hidden size */
    int32_t I;               /* intermediate size */
    int32_t dtype;           /* skipffn_dtype of x, weights, out, dx */
    int32_t dense;           /* 1: ignore skip_mask, every token takes the FFN (comparator) */
    int32_t grad_dtype_fp32; /* 1: dW_* are fp32 regardless of dtype */
    int32_t accumulate_dw;   /* 1: dW += ..., 0: dW is overwritten */
    int32_t path;            /* skipffn_path */
    int32_t prenorm;         /* 1: pre-norm variant (skipffn_forward_prenorm / _backward_prenorm) */
    int32_t debug;           /* 1: debug handle: extra device-side checks (see skipffn_poll), test hooks */
    int32_t recompute;       /* 1: the forward keeps no G, U, H; the backward computes them again */
} skipffn_config;

/* Host-side handle linking one forward call to its backward call.  It points into the caller's
 * workspace, where the kept-row index list, the compacted rows of x and the SwiGLU
 * intermediates G, U, H (and dG, dU during backward) live. */
typedef struct skipffn_saved skipffn_saved;

/* Device memory of a handle.  It has two parts:
 *   saved    what must survive from a forward call to its backward call: the kept-row list, the kept
 *            rows of x and -- unless cfg.recompute -- the SwiGLU intermediates G, U, H;
 *   scratch  what only lives inside one call (dG, dU, the kept rows of dout, K-split hand-over slots,
 *            and G, U, H of a recomputing handle).  Handles whose calls never overlap on the GPU (the
 *            layers of one model, run one after the other) may share one scratch buffer.
 * max_tokens bounds B*S of any call; max_kept (<= max_tokens) bounds the number of kept tokens and
 * sizes every compacted array, so a model that skips 75 % of its visual tokens does not pay for the
 * rows it never sends through the FFN.  A mask that keeps more than max_kept tokens is not an
 * out-of-bounds access: the first max_kept kept tokens take the FFN, the others are treated as
 * skipped, and skipffn_poll reports SKIPFFN_EWORKSPACE.
 * Recompute mode trades time for memory (the idea of not storing what the backward can rebuild):
 * the forward stores only H, transiently, for the down projection; the backward runs the gate/up
 * GEMM again (one more launch, +4 Nk C I flops).  Results are the same bits in both modes.
 * All sizes are 0 if the arguments are invalid; buffers must be 1024-byte aligned. */
size_t skipffn_saved_bytes(const skipffn_config *cfg, int64_t max_tokens, int64_t max_kept);
size_t skipffn_scratch_bytes(const skipffn_config *cfg, int64_t max_tokens, int64_t max_kept);
/* saved + scratch in one buffer */
size_t skipffn_workspace_bytes_kept(const skipffn_config *cfg, int64_t max_tokens, int64_t max_kept);
/* the same with max_kept = max_tokens */
size_t skipffn_workspace_bytes(const skipffn_config *cfg, int64_t max_tokens);

/* Create a handle.  Host-only: nothing is launched.  EWORKSPACE if a buffer is too small.
 *   skipffn_saved_create_split : separate saved and scratch buffers;
 *   skipffn_saved_create_kept  : one buffer of skipffn_workspace_bytes_kept bytes;
 *   skipffn_saved_create       : one buffer of skipffn_workspace_bytes bytes (max_kept = max_tokens). */
skipffn_status skipffn_saved_create_split(skipffn_saved **saved, const skipffn_config *cfg,
                                          void *saved_mem, size_t saved_bytes, void *scratch_mem,
                                          size_t scratch_bytes, int64_t max_tokens, int64_t max_kept);
skipffn_status skipffn_saved_create_kept(skipffn_saved **saved, const skipffn_config *cfg,
                                         void *workspace, size_t workspace_bytes, int64_t max_tokens,
                                         int64_t max_kept);
skipffn_status skipffn_saved_create(skipffn_saved **saved, const skipffn_config *cfg,
                                    void *workspace, size_t workspace_bytes, int64_t max_tokens);
void skipffn_saved_destroy(skipffn_saved *saved);

/* Tuning and test knobs of a handle (host-only; none is needed in normal use).  They affect the
 * tensor-core GEMM launches that follow.
 *   TILE_N          accumulator columns per tile instead of 256: a multiple of 16 (token problems)
 *                   or 32 (weight gradients) in 32 .. 256; 0 = default
 *   STREAMK         least number of K-blocks per worker that cutting the tail tiles along K must
 *                   save for the cut to be used: 0 never cut, 1 cut whenever the tiles do not fill
 *                   a wave, -1 = default per kernel
 *   STAGES          use only this many stages of the shared-memory ring (1 .. 5); 0 = all
 *   ONE_BOX         1 (default): an operand tile that consists of two 64-wide pieces (the two slabs
 *                   of a transposed operand; the gate and the up rows) is fetched with one 3-D
 *                   TMA box where the arrays allow it; 0: always one 2-D box per piece
 *   TMA_STORES      1 (default): weight-gradient tiles that overwrite their destination are written
 *                   with TMA tile stores from shared memory; 0: with per-lane 16-byte stores
 *   GATHER          1: the gate/up and dH GEMMs fetch their token rows straight from x / dout with
 *                   tile::gather4 TMA loads driven by the kept-row list, instead of from the
 *                   compacted copy (which is still made: the weight gradients and the residual
 *                   read it).  0 (default): compacted copy, which measured faster
 *   PANEL_SYNC      down and dX GEMMs with few tiles and a long reduction: -1 (default) or 1: when it
 *                   costs under 6 % more K-blocks per worker, the workers form groups of one per
 *                   token tile and each group walks the K-blocks of a weight panel side by side,
 *                   so that a panel is fetched from DRAM once (its loads carry an L2 evict-first
 *                   policy, so that the token operand stays cached); 2: always; 0: every worker
 *                   takes its own contiguous run of K-blocks; add 4 to 1 or 2 to leave the
 *                   eviction policy off
 *   LOSE_HANDOVER   debug handles only (EINVAL otherwise): nonzero makes the finishing units of a
 *                   K-split launch wait for a hand-over that never comes, so that the bounded wait
 *                   runs out and skipffn_poll reports SKIPFFN_ETIMEOUT -- the failure path can be
 *                   exercised without any fault */
typedef enum { SKIPFFN_TUNE_TILE_N = 0, SKIPFFN_TUNE_STREAMK = 1, SKIPFFN_TUNE_STAGES = 2,
               SKIPFFN_TUNE_LOSE_HANDOVER = 3, SKIPFFN_TUNE_ONE_BOX = 4, SKIPFFN_TUNE_TMA_STORES = 5, SKIPFFN_TUNE_GATHER = 6,
               SKIPFFN_TUNE_PANEL_SYNC = 7, SKIPFFN_TUNE_COUNT = 8 } skipffn_tunable;
skipffn_status skipffn_tune(skipffn_saved *saved, int32_t what, int32_t value);

/* Mask compaction alone (the retained / skipped split is the same for every decoder layer, so a
 * caller may build it once): writes the ascending kept-row index list and its length into the
 * workspace.  A later skipffn_forward with skip_mask == NULL reuses it. */
skipffn_status skipffn_plan(skipffn_saved *saved, const uint8_t *skip_mask, int64_t N,
                            void *stream);

/* Forward, Eq. 4 / Eq. 5.  x, out: [B*S, C] (out may alias x); skip_mask: [B*S] bytes or NULL to
 * reuse the list of the last skipffn_plan / skipffn_forward on this handle (same B*S required);
 * cu_seqlens: optional int32 HOST array of n_seq+1 offsets of a packed batch (B == 1), checked
 * for monotonicity and total only -- the FFN is token-wise.  Kept rows of `out` are the fp32 sum
 * x + FFN(x) rounded once; skipped rows are byte copies of x.  The handle borrows the three
 * weight pointers until skipffn_backward returns. */
skipffn_status skipffn_forward(skipffn_saved *saved, const void *x, const uint8_t *skip_mask,
                               int64_t B, int64_t S, const int32_t *cu_seqlens,
                               int32_t n_seq, const void *W_gate, const void *W_up,
                               const void *W_down, void *out, void *stream);

/* Backward of the forward last run on `saved`.  dout, dx: [B*S, C] (dx may alias dout);
 * dW_gate, dW_up: [I, C]; dW_down: [C, I] in cfg.dtype (fp32 if grad_dtype_fp32), overwritten or
 * accumulated per cfg.accumulate_dw; any dW pointer may be NULL to skip that gradient.
 * Skipped rows of dx are byte copies of dout.  With zero kept tokens dW is zero (or untouched
 * when accumulating). */
skipffn_status skipffn_backward(const void *dout, skipffn_saved *saved, void *dx, void *dW_gate,
                                void *dW_up, void *dW_down, void *stream);

/* Pre-norm variant (cfg.prenorm = 1).  Eq. 4 writes FFN(h_attn); the decoder blocks of the paper's
 * LLaMA-3 / Vicuna backbones (section 6.4 training setup) normalise the FFN input, so this variant
 * computes, for retained tokens,
 *     out[t] = x[t] + FFN( RMSNorm(x[t]) * gamma ),   RMSNorm(x) = x / sqrt(mean_c x[c]^2 + eps),
 * and out[t] = x[t] for skipped tokens (Eq. 5): skipping the FFN skips its normalisation too.
 * gamma: [C] in cfg.dtype (borrowed until the backward returns); eps >= 0.  The normalised rows
 * are rounded once to cfg.dtype before the projections; statistics are fp32.
 * Backward additionally returns dgamma [C] (cfg.dtype, fp32 with grad_dtype_fp32; overwritten or
 * accumulated like the weight gradients; may be NULL).  All other arguments as in
 * skipffn_forward / skipffn_backward, which reject a handle created with prenorm = 1 (and these
 * two reject one created without). */
skipffn_status skipffn_forward_prenorm(skipffn_saved *saved, const void *x, const uint8_t *skip_mask,
                                       int64_t B, int64_t S, const int32_t *cu_seqlens, int32_t n_seq,
                                       const void *gamma, float eps, const void *W_gate,
                                       const void *W_up, const void *W_down, void *out, void *stream);
skipffn_status skipffn_backward_prenorm(const void *dout, skipffn_saved *saved, void *dx, void *dgamma,
                                        void *dW_gate, void *dW_up, void *dW_down, void *stream);

/* Adaptive summary token (paper section 4.2, Eq. 6):  x_s = softmax(X w^T)^T X, where X holds the
 * retained or the skipped visual tokens of one sample and w [C] is the layer's weight.  Needs no
 * handle.  Several samples are processed at once as segments of a packed X:
 *   X           : [n_rows, C] device, dtype = skipffn_dtype, C a multiple of 8
 *   seg_offsets : DEVICE int32 [n_seg + 1], ascending, first 0, last n_rows
 *   xs          : [n_seg, C] out (an empty segment gives zeros);  probs : [n_rows] fp32 out, the
 *                 softmax weights, which the backward needs.
 * Backward for upstream gradient dxs [n_seg, C]: dX [n_rows, C] (may be NULL), dw [C] (may be NULL;
 * fp32 if dw_fp32 or dtype is fp32), both overwritten.  scratch: device memory of
 * skipffn_summary_scratch_bytes(n_rows, C) bytes, 16-byte aligned (EWORKSPACE if smaller).
 * X, w, xs, dxs and dX start on 16-byte boundaries (EINVAL otherwise).
 * Scores, weights and all sums are fp32 in a fixed order; outputs are rounded once. */
size_t skipffn_summary_scratch_bytes(int64_t n_rows, int32_t C);
skipffn_status skipffn_summary_forward(const void *X, const int32_t *seg_offsets, int32_t n_seg,
                                       int64_t n_rows, int32_t C, int32_t dtype, const void *w,
                                       void *xs, float *probs, void *stream);
skipffn_status skipffn_summary_backward(const void *X, const int32_t *seg_offsets, int32_t n_seg,
                                        int64_t n_rows, int32_t C, int32_t dtype, const void *w,
                                        const float *probs, const void *dxs, void *dX, void *dw,
                                        int32_t dw_fp32, void *scratch, size_t scratch_bytes,
                                        void *stream);

/* Token merge of the skipped visual tokens (paper section 4.1): (1) cosine similarity between every
 * pair of the n tokens and an average similarity per token, (2) the k tokens with the LOWEST average
 * are kept, (3) each other token is merged into its most similar kept token.
 *   X      : [n, C] device, dtype = skipffn_dtype; C a multiple of 8, at most 16384; n <= 65536
 *   k      : tokens to keep, a multiple of 4, 1 <= k <= n
 *   kept   : [k] int32 out, the kept tokens' indices in ascending order
 *   assign : [n] int32 out, for every token the position in `kept` of the token it goes to (a kept
 *            token goes to itself)
 *   merged : [k, C] out, dtype as X
 *   scratch: device memory of skipffn_token_merge_scratch_bytes(...) bytes, 256-byte aligned.
 * Where the paper is silent: the average includes the token itself (leaving it out would not change
 * the order); equal averages go to the lower index; equal similarities in (3) go to the first kept
 * token; a zero row has similarity 0 with everything; the MERGE OPERATOR IS NOT STATED in the paper
 * and is taken as the mean of a kept token and the tokens merged into it, summed in token order.
 * The average is computed as the dot product with the mean unit vector (no n x n matrix); the
 * (n-k) x k similarity matrix of step (3) runs on the tensor cores for bf16, on unit rows rounded
 * to bf16.  Statistics are fp32; decisions between nearly equal values may differ from an
 * exact-arithmetic evaluation. */
size_t skipffn_token_merge_scratch_bytes(int64_t n, int32_t C, int32_t k, int32_t dtype);
skipffn_status skipffn_token_merge(const void *X, int64_t n, int32_t C, int32_t k, int32_t dtype,
                                   int32_t *kept, int32_t *assign, void *merged, void *scratch,
                                   size_t scratch_bytes, void *stream);

/* Synchronises `stream` and reads the status word the last skipffn_token_merge call on this scratch
 * (same n, C, k, dtype) left behind: SKIPFFN_ETIMEOUT with the wait site in *site_out (may be NULL)
 * if its tensor-core kernel gave up on a wait, else SKIPFFN_OK. */
skipffn_status skipffn_token_merge_poll(void *scratch, int64_t n, int32_t C, int32_t k, int32_t dtype,
                                        void *stream, int32_t *site_out);

/* Device addresses of the kept-row index list (int32, ascending) and of its length. */
skipffn_status skipffn_get_kept(const skipffn_saved *saved, const int32_t **idx_dev,
                                const int32_t **nk_dev);

/* Skip KV-cache (paper section 4.3, Eq. 7): after prefill the cache keeps only the keys / values of
 * the retained tokens, K' = K \ K_skip, in their original order.  Uses the kept-row list of the
 * last skipffn_plan / skipffn_forward on `saved` (N = its token count).
 *   src : [planes, N, row_bytes] device bytes: any number of leading dimensions (layer, key/value)
 *         flattened into `planes`, then the token axis, then one token's heads x head_dim values
 *         (the packed "total tokens" layout); row_bytes a multiple of 16.
 *   dst : [planes, dst_rows, row_bytes]; rows 0 .. min(Nk, dst_rows)-1 of every plane receive the
 *         kept rows, byte for byte; other rows are not written.  Must not overlap src (EINVAL).
 *   cu_seqlens / kept_cu_seqlens : optional DEVICE int32 arrays of n_seq+1 entries; when
 *         kept_cu_seqlens is given it receives the sequence offsets of the pruned cache, i.e. the
 *         number of kept tokens before each cu_seqlens[s].
 * Enqueued on `stream`; Nk stays on the device. */
skipffn_status skipffn_kv_compact(const skipffn_saved *saved, const void *src, void *dst,
                                  int64_t planes, int64_t row_bytes, int64_t dst_rows,
                                  const int32_t *cu_seqlens, int32_t n_seq,
                                  int32_t *kept_cu_seqlens, void *stream);

/* Device addresses of the compacted intermediates of the last forward / backward, each
 * [Nk, I] in cfg.dtype (rows Nk .. round_up(Nk,16)-1 are zero, later rows are unspecified):
 * which = 0 G, 1 U, 2 H, 3 dG, 4 dU;
 * 5 = kept rows of x [.., C]; 6 = kept rows of dout [.., C]; 7 = normalised kept rows of x
 * [.., C] (pre-norm variant only). */
skipffn_status skipffn_get_intermediate(const skipffn_saved *saved, int32_t which,
                                        const void **ptr_dev);

/* Synchronises `stream`, then reads the device status word: returns SKIPFFN_ETIMEOUT (and the
 * site code in *site_out, may be NULL) if a kernel gave up on a wait, SKIPFFN_EWORKSPACE if a mask
 * kept more than max_kept tokens, SKIPFFN_ECUDA if the stream reports an error, else SKIPFFN_OK.
 * The word is cleared.
 * Debug handles (cfg.debug = 1) add two checks, both reported as SKIPFFN_EDEBUG: after every mask
 * compaction the kept-row list is verified on the device (in range, strictly ascending, inverse map
 * consistent; site 16), and every slab of the workspace is followed by a 1 KiB guard band whose
 * contents skipffn_poll verifies (site 32 + slab number): a kernel that wrote past its slab shows up
 * here instead of corrupting a neighbour silently.  Debug handles need slightly more workspace. */
skipffn_status skipffn_poll(skipffn_saved *saved, void *stream, int32_t *site_out);

/* Per-launch timing for benchmarks.  While enabled, forward / backward record a CUDA event on the
 * caller's stream before and after each kernel launch (no synchronisation).  skipffn_profile_read
 * waits for those events and writes the elapsed milliseconds of each launch slot into
 * ms[SKIPFFN_PROFILE_SLOTS] (0 for slots that did not run): 0 mask compaction, 1 routing of x,
 * 2 gate/up GEMM, 3 down GEMM, 4 routing of dout, 5 dH GEMM, 6 dW_down, 7 dW_gate, 8 dW_up,
 * 9 dX GEMM.  The tensor-core path computes the requested weight gradients in ONE grouped launch,
 * whose time is reported in the slot of the first of them (6 when dW_down is requested) with the
 * other two slots 0.  Slot 10 (pre-norm variant): the normalisation's backward (dx rows and dgamma).
 * Slot 11 (recomputing handles): the gate/up GEMM run again at the start of the backward. */
#define SKIPFFN_PROFILE_SLOTS 12
skipffn_status skipffn_profile_enable(skipffn_saved *saved, int32_t on);
skipffn_status skipffn_profile_read(skipffn_saved *saved, float *ms);

/* Number of kernels the last forward (which=0) or backward (which=1) call enqueued. */
int32_t skipffn_last_launches(const skipffn_saved *saved, int32_t which);

/* Diagnostic (host only, launches nothing): the work distribution of the tensor-core GEMM kernels.
 * A launch with `tiles` output tiles of `k_blocks` K-blocks each runs on `workers` persistent
 * workers; whole waves of tiles are handed out tile by tile, the tiles of the last one-to-two waves
 * are cut along K into equal runs (split_k != 0).  Returns the number of segments of `worker`'s
 * schedule (-1 on bad arguments) and, for 0 <= i < that number, writes segment i to seg[5] =
 * {tile, first K-block, end K-block, partial, first source worker}: partial = 1 means the run stops
 * before the tile's last K-block and its accumulator is handed over; otherwise the worker finishes
 * the tile after adding the accumulators handed over by workers seg[4] .. worker-1. */
int32_t skipffn_schedule_segment(int32_t workers, int32_t tiles, int32_t k_blocks, int32_t split_k,
                                 int32_t worker, int32_t i, int32_t *seg);

/* Diagnostic (host only, launches nothing): the same for a token problem of `panels` blocks of weight
 * rows x `token_tiles` token tiles (tile = panel * token_tiles + token tile), including the worker
 * groups of the down / dX launches (group_mode as the PANEL_SYNC knob, min_saving as the STREAMK
 * knob: least K-blocks per worker a cut must save, 0 = never cut).  seg[6] = {tile, first K-block,
 * end K-block, partial, first source worker, source stride}: a finishing segment that starts at a
 * K-block > 0 adds the accumulators handed over by workers seg[4], seg[4] + seg[5], ... below
 * `worker` (those that have a partial segment of this tile). */
int32_t skipffn_schedule_plan_segment(int32_t workers, int32_t panels, int32_t token_tiles, int32_t k_blocks,
                                      int32_t min_saving, int32_t group_mode, int32_t worker, int32_t i,
                                      int32_t *seg);

/* Algorithmic floating-point operations of one forward+backward call with n_kept kept tokens:
 * 18 * n_kept * C * I (forward 6: three GEMMs of the section 6.2 cost model; backward 12). */
double skipffn_flops(const skipffn_config *cfg, int64_t n_kept);

const char *skipffn_strerror(skipffn_status status);

/* Kept-row index list without a workspace or a handle, for callers that cannot allocate device
 * memory.  (The paper has no counterpart: it is a packaging of the mask compaction above, useful
 * by itself e.g. to drop the skipped tokens' rows from a key/value cache.)
 *
 * Who needs it: code running where cudaMalloc is not an option -- a process whose framework has
 * already reserved all device memory for its own pool, a latency-critical loop that cannot take
 * cudaMalloc's device-wide synchronisation, or a host application that forbids allocation calls
 * from extensions.  The kernel's scratch (token -> rank map and kept count) lives in a fixed
 * array inside the library image, about 256 KiB per device that loads the library, held until
 * the process exits.  The call allocates nothing, on the device or through any library.
 *
 * skip_mask : [N] bytes on the device, nonzero = skipped.
 * idx       : [N] int32 on the device; entries 0 .. Nk-1 receive the ascending indices of the kept
 *             tokens, the remaining entries are unspecified.
 * nk        : one int32 on the device, receives Nk.
 * Work is enqueued on `stream`; nothing is synchronised.
 *
 * N > SKIPFFN_STATIC_MAX_TOKENS returns SKIPFFN_EUNSUPPORTED and launches nothing.
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call outside any stream capture.
 * All calls on a device share the array: calls that may overlap on the GPU (different streams or
 * host threads) race and must be serialised by the caller.  Nothing in it has to be zero between
 * calls; each call overwrites every word it reads. */
#define SKIPFFN_STATIC_MAX_TOKENS 65536
skipffn_status skipffn_compact_static(const uint8_t *skip_mask, int64_t N, int32_t *idx,
                                      int32_t *nk, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SKIPFFN_H_ */
