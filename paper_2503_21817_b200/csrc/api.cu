// C-ABI entry points of libskipffn: argument checks, workspace layout, launch sequencing.
#include <new>
#include <string.h>

#include <limits.h>

#include "common.cuh"
#include "sched.cuh"

using namespace skipffn;

struct skipffn_saved {
    skipffn_config cfg;
    int64_t max_tokens, cap;   // cap: rows of the token-indexed arrays (idx, pos)
    int64_t max_kept, cap_k;   // cap_k: rows of the compacted arrays (kept rows only)
    size_t ws_bytes;
    int esize;
    // workspace carve-up (device)
    int32_t *status, *sk_flags, *idx, *pos;
    void *sk_slots, *Xk, *dOk, *G, *U, *H, *dG, *dU;
    void *Xn;              // pre-norm variant: normalised kept rows (the FFN input)
    float *rstd, *dY;      //   per-row 1/rms, and the fp32 gradient w.r.t. the normalised rows
    float *dg_part;        //   [DG_CHUNKS, C] partial sums of the gain's gradient
    const void *gamma;     //   gain vector of the last forward (borrowed)
    // state
    int64_t planned_N;     // tokens of the current index list, -1 if none
    int forwarded;
    const void *Wg, *Wu, *Wd;
    int launches[2];
    int32_t sk_epoch;      // flag value of the latest tensor-core GEMM launch (never 0)
    GuardList guards;      // debug handles: addresses of the guard bands
    int32_t tune[SKIPFFN_TUNE_COUNT];   // skipffn_tune values
    TmapCache tmaps;       // encoded tensor maps of the arrays this handle launches on
    // optional per-launch timing (CUDA events on the caller's stream)
    int profiling;
    cudaEvent_t ev[2 * SKIPFFN_PROFILE_SLOTS];
    int ev_recorded[SKIPFFN_PROFILE_SLOTS];
};

namespace {

// Two regions.  `saved` must survive from a forward call to its backward call; `scratch` only lives
// inside one call, so several handles (the layers of a model) may share one scratch buffer as long
// as their calls do not overlap.  With cfg.recompute the SwiGLU intermediates G, U, H move from the
// saved region to the scratch region: the backward pass computes them again.
struct Layout {
    size_t status, idx, pos, Xk, Xn, rstd, saved_total;                  // saved region
    size_t sk_slots, dOk, dG, dU, dY, dg_part, scratch_total;              // scratch region
    size_t G, U, H;                                                        // in saved, or in scratch when recomputing
    int n_guards;                                                          // debug handles: guard bands behind the slabs
    size_t guard_off[MAX_GUARDS];
    bool guard_in_scratch[MAX_GUARDS];
};

bool valid_cfg(const skipffn_config *c)
{
    return c && c->C > 0 && c->I > 0 && (c->dtype == SKIPFFN_BF16 || c->dtype == SKIPFFN_FP32) &&
           (c->path == SKIPFFN_PATH_DEFAULT || c->path == SKIPFFN_PATH_SIMT) &&
           (c->prenorm == 0 || c->prenorm == 1) && (c->debug == 0 || c->debug == 1) &&
           (c->recompute == 0 || c->recompute == 1);
}

Layout make_layout(const skipffn_config *c, int64_t max_tokens, int64_t max_kept)
{
    Layout l;
    const int64_t cap = round_up(max_tokens > 0 ? max_tokens : 1, ROW_PAD);
    const int64_t cap_k = round_up(max_kept > 0 ? max_kept : 1, ROW_PAD);
    const size_t es = c->dtype == SKIPFFN_BF16 ? 2 : 4;
    size_t off = 0;
    bool in_scratch = false;
    l.n_guards = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off = (size_t)round_up((int64_t)(off + bytes), 1024);
        if (c->debug && bytes > 0 && l.n_guards < MAX_GUARDS) {   // guard band right behind the slab
            l.guard_off[l.n_guards] = off;
            l.guard_in_scratch[l.n_guards++] = in_scratch;
            off += GUARD_BYTES;
        }
        return o;
    };
    l.status = take((ST_WORDS + SK_FLAG_WORDS) * 4);   // status block, then the hand-over flags
    l.idx = take((size_t)cap * 4);
    l.pos = take((size_t)cap * 4);
    l.Xk = take((size_t)cap_k * c->C * es);
    l.Xn = take(c->prenorm ? (size_t)cap_k * c->C * es : 0);
    l.rstd = take(c->prenorm ? (size_t)cap_k * 4 : 0);
    if (!c->recompute) {
        l.G = take((size_t)cap_k * c->I * es);
        l.U = take((size_t)cap_k * c->I * es);
        l.H = take((size_t)cap_k * c->I * es);
    }
    l.saved_total = off;
    off = 0;
    in_scratch = true;
    l.sk_slots = take(c->dtype == SKIPFFN_BF16 ? (size_t)SK_MAX_CTAS * SK_SLOT_BYTES : 0);
    l.dOk = take((size_t)cap_k * c->C * es);
    l.dG = take((size_t)cap_k * c->I * es);
    l.dU = take((size_t)cap_k * c->I * es);
    l.dY = take(c->prenorm ? (size_t)cap_k * c->C * 4 : 0);
    l.dg_part = take(c->prenorm ? (size_t)DG_CHUNKS * c->C * 4 : 0);
    if (c->recompute) {
        l.G = take((size_t)cap_k * c->I * es);
        l.U = take((size_t)cap_k * c->I * es);
        l.H = take((size_t)cap_k * c->I * es);
    }
    l.scratch_total = off;
    return l;
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

bool use_umma(const skipffn_saved *s)
{
    return s->cfg.dtype == SKIPFFN_BF16 && s->cfg.path == SKIPFFN_PATH_DEFAULT;
}

// Launch slots (also the order of skipffn_profile_read): forward 0 compaction, 1 routing of x,
// 2 gate/up GEMM, 3 down GEMM; backward 4 routing of dout, 5 dH GEMM, 6 dW_down, 7 dW_gate,
// 8 dW_up, 9 dX GEMM; 10 normalisation backward (pre-norm variant); 11 the gate/up GEMM run again
// by a recomputing handle's backward.
enum : int { SLOT_COMPACT = 0, SLOT_ROUTE_X, SLOT_GATEUP, SLOT_DOWN, SLOT_ROUTE_DOUT, SLOT_DH,
             SLOT_DW_DOWN, SLOT_DW_GATE, SLOT_DW_UP, SLOT_DX, SLOT_NORM_BWD, SLOT_RECOMPUTE };

template <typename F>
cudaError_t timed_launch(skipffn_saved *s, int slot, cudaStream_t st, F &&launch)
{
    s->launches[(slot >= SLOT_ROUTE_DOUT) ? 1 : 0]++;
    if (!s->profiling) return launch();
    cudaError_t e = cudaEventRecord(s->ev[2 * slot], st);
    if (e != cudaSuccess) return e;
    e = launch();
    if (e != cudaSuccess) return e;
    s->ev_recorded[slot] = 1;
    return cudaEventRecord(s->ev[2 * slot + 1], st);
}

cudaError_t run_gemm(skipffn_saved *s, int slot, int epi, GemmArgs &g, cudaStream_t st)
{
    // every launch gets its own flag value, so flags left by earlier launches never match
    if (++s->sk_epoch <= 0) s->sk_epoch = 1;
    g.sk_epoch = s->sk_epoch;
    return timed_launch(s, slot, st, [&] {
        return use_umma(s) ? launch_umma_gemm(epi, g, st) : launch_simt_gemm(epi, s->cfg.dtype, g, st);
    });
}

GemmArgs base_args(skipffn_saved *s)
{
    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.status = s->status;
    g.idx = s->idx;
    g.sk_slots = s->sk_slots;
    g.sk_flags = s->sk_flags;
    g.tune_tile_n = s->tune[SKIPFFN_TUNE_TILE_N];
    g.tune_stages = s->tune[SKIPFFN_TUNE_STAGES];
    g.tune_streamk = s->tune[SKIPFFN_TUNE_STREAMK];
    g.tune_panel_sync = s->tune[SKIPFFN_TUNE_PANEL_SYNC];
    // failure-path hook of debug handles: finishing units of a K-split launch wait for a hand-over
    // flag value that nothing writes, so their bounded wait runs out
    g.sk_wait_skew = (s->cfg.debug && s->tune[SKIPFFN_TUNE_LOSE_HANDOVER]) ? 0x40000000 : 0;
    g.one_box_loads = s->tune[SKIPFFN_TUNE_ONE_BOX];
    g.tma_stores = s->tune[SKIPFFN_TUNE_TMA_STORES];
    g.tmaps = &s->tmaps;
    return g;
}

// first use of a handle: clear the status block and the hand-over flags; debug handles fill their guard bands
cudaError_t first_use(skipffn_saved *s, cudaStream_t st)
{
    if (s->planned_N >= 0) return cudaSuccess;
    cudaError_t e = cudaMemsetAsync(s->status, 0, (ST_WORDS + SK_FLAG_WORDS) * 4, st);
    for (int i = 0; e == cudaSuccess && i < s->guards.n; ++i)
        e = cudaMemsetAsync(const_cast<void *>(s->guards.ptr[i]), GUARD_BYTE, GUARD_BYTES, st);
    return e;
}

skipffn_status do_plan(skipffn_saved *s, const uint8_t *mask, int64_t N, int which, cudaStream_t st)
{
    (void)which;
    if (N > 0) {
        if (timed_launch(s, SLOT_COMPACT, st, [&] {
                return launch_compact(mask, N, s->cfg.dense, s->idx, s->pos, s->status, s->cap, s->max_kept, st);
            }) != cudaSuccess)
            return SKIPFFN_ECUDA;
        if (s->cfg.debug && launch_check_kept(s->idx, s->pos, s->status, N, st) != cudaSuccess) return SKIPFFN_ECUDA;
    } else if (cudaMemsetAsync(s->status, 0, 4, st) != cudaSuccess) {
        return SKIPFFN_ECUDA;
    }
    s->planned_N = N;
    return SKIPFFN_OK;
}

}  // namespace

extern "C" {

size_t skipffn_saved_bytes(const skipffn_config *cfg, int64_t max_tokens, int64_t max_kept)
{
    if (!valid_cfg(cfg) || max_tokens < 0 || max_kept < 0 || max_kept > max_tokens) return 0;
    return make_layout(cfg, max_tokens, max_kept).saved_total;
}

size_t skipffn_scratch_bytes(const skipffn_config *cfg, int64_t max_tokens, int64_t max_kept)
{
    if (!valid_cfg(cfg) || max_tokens < 0 || max_kept < 0 || max_kept > max_tokens) return 0;
    return make_layout(cfg, max_tokens, max_kept).scratch_total;
}

size_t skipffn_workspace_bytes_kept(const skipffn_config *cfg, int64_t max_tokens, int64_t max_kept)
{
    if (!valid_cfg(cfg) || max_tokens < 0 || max_kept < 0 || max_kept > max_tokens) return 0;
    const Layout l = make_layout(cfg, max_tokens, max_kept);
    return l.saved_total + l.scratch_total;
}

size_t skipffn_workspace_bytes(const skipffn_config *cfg, int64_t max_tokens)
{
    return skipffn_workspace_bytes_kept(cfg, max_tokens, max_tokens);
}

skipffn_status skipffn_saved_create_split(skipffn_saved **saved, const skipffn_config *cfg, void *saved_mem,
                                          size_t saved_bytes, void *scratch_mem, size_t scratch_bytes,
                                          int64_t max_tokens, int64_t max_kept)
{
    if (!saved) return SKIPFFN_EINVAL;
    *saved = nullptr;
    if (!valid_cfg(cfg) || !saved_mem || !scratch_mem || max_tokens < 0 || max_kept < 0 || max_kept > max_tokens)
        return SKIPFFN_EINVAL;
    if ((cfg->C % 8) || (cfg->I % 8)) return SKIPFFN_EUNSUPPORTED;
    if (max_tokens > (int64_t)1 << 30) return SKIPFFN_EUNSUPPORTED;
    if (((uintptr_t)saved_mem & 1023u) || ((uintptr_t)scratch_mem & 1023u)) return SKIPFFN_EINVAL;
    Layout l = make_layout(cfg, max_tokens, max_kept);
    if (saved_bytes < l.saved_total || scratch_bytes < l.scratch_total) return SKIPFFN_EWORKSPACE;
    skipffn_saved *s = new (std::nothrow) skipffn_saved;
    if (!s) return SKIPFFN_EINVAL;
    memset(s, 0, sizeof(*s));
    s->cfg = *cfg;
    s->max_tokens = max_tokens;
    s->cap = round_up(max_tokens > 0 ? max_tokens : 1, ROW_PAD);
    s->max_kept = max_kept;
    s->cap_k = round_up(max_kept > 0 ? max_kept : 1, ROW_PAD);
    s->ws_bytes = saved_bytes + scratch_bytes;
    s->esize = cfg->dtype == SKIPFFN_BF16 ? 2 : 4;
    char *w = (char *)saved_mem, *x = (char *)scratch_mem;
    char *gu = cfg->recompute ? x : w;
    s->status = (int32_t *)(w + l.status);
    s->sk_flags = s->status + ST_WORDS;
    s->idx = (int32_t *)(w + l.idx);
    s->pos = (int32_t *)(w + l.pos);
    s->Xk = w + l.Xk;
    s->Xn = w + l.Xn; s->rstd = (float *)(w + l.rstd);
    s->G = gu + l.G; s->U = gu + l.U; s->H = gu + l.H;
    s->sk_slots = x + l.sk_slots;
    s->dOk = x + l.dOk; s->dG = x + l.dG; s->dU = x + l.dU;
    s->dY = (float *)(x + l.dY);
    s->dg_part = (float *)(x + l.dg_part);
    s->planned_N = -1;
    s->tune[SKIPFFN_TUNE_STREAMK] = -1;
    s->tune[SKIPFFN_TUNE_PANEL_SYNC] = -1;
    s->tune[SKIPFFN_TUNE_ONE_BOX] = 1;
    s->tune[SKIPFFN_TUNE_TMA_STORES] = 1;
    s->guards.n = l.n_guards;
    for (int i = 0; i < l.n_guards; ++i) s->guards.ptr[i] = (l.guard_in_scratch[i] ? x : w) + l.guard_off[i];
    *saved = s;
    return SKIPFFN_OK;
}

skipffn_status skipffn_saved_create_kept(skipffn_saved **saved, const skipffn_config *cfg, void *workspace,
                                         size_t workspace_bytes, int64_t max_tokens, int64_t max_kept)
{
    if (!saved) return SKIPFFN_EINVAL;
    *saved = nullptr;
    if (!valid_cfg(cfg) || !workspace || max_tokens < 0 || max_kept < 0 || max_kept > max_tokens) return SKIPFFN_EINVAL;
    const Layout l = make_layout(cfg, max_tokens, max_kept);
    if (workspace_bytes < l.saved_total + l.scratch_total) return SKIPFFN_EWORKSPACE;
    return skipffn_saved_create_split(saved, cfg, workspace, l.saved_total, (char *)workspace + l.saved_total,
                                      workspace_bytes - l.saved_total, max_tokens, max_kept);
}

skipffn_status skipffn_saved_create(skipffn_saved **saved, const skipffn_config *cfg, void *workspace,
                                    size_t workspace_bytes, int64_t max_tokens)
{
    return skipffn_saved_create_kept(saved, cfg, workspace, workspace_bytes, max_tokens, max_tokens);
}

skipffn_status skipffn_tune(skipffn_saved *s, int32_t what, int32_t value)
{
    if (!s || what < 0 || what >= SKIPFFN_TUNE_COUNT) return SKIPFFN_EINVAL;
    if (what == SKIPFFN_TUNE_LOSE_HANDOVER && !s->cfg.debug) return SKIPFFN_EINVAL;
    s->tune[what] = value;
    return SKIPFFN_OK;
}

void skipffn_saved_destroy(skipffn_saved *saved)
{
    if (!saved) return;
    if (saved->profiling)
        for (int i = 0; i < 2 * SKIPFFN_PROFILE_SLOTS; ++i) cudaEventDestroy(saved->ev[i]);
    delete saved;
}

skipffn_status skipffn_profile_enable(skipffn_saved *s, int32_t on)
{
    if (!s) return SKIPFFN_EINVAL;
    if (on && !s->profiling) {
        for (int i = 0; i < 2 * SKIPFFN_PROFILE_SLOTS; ++i)
            if (cudaEventCreate(&s->ev[i]) != cudaSuccess) {
                for (int j = 0; j < i; ++j) cudaEventDestroy(s->ev[j]);
                return SKIPFFN_ECUDA;
            }
        s->profiling = 1;
    } else if (!on && s->profiling) {
        for (int i = 0; i < 2 * SKIPFFN_PROFILE_SLOTS; ++i) cudaEventDestroy(s->ev[i]);
        s->profiling = 0;
    }
    memset(s->ev_recorded, 0, sizeof(s->ev_recorded));
    return SKIPFFN_OK;
}

skipffn_status skipffn_profile_read(skipffn_saved *s, float *ms)
{
    if (!s || !ms || !s->profiling) return SKIPFFN_EINVAL;
    for (int i = 0; i < SKIPFFN_PROFILE_SLOTS; ++i) {
        ms[i] = 0.0f;
        if (!s->ev_recorded[i]) continue;
        if (cudaEventSynchronize(s->ev[2 * i + 1]) != cudaSuccess) return SKIPFFN_ECUDA;
        if (cudaEventElapsedTime(&ms[i], s->ev[2 * i], s->ev[2 * i + 1]) != cudaSuccess) return SKIPFFN_ECUDA;
        s->ev_recorded[i] = 0;
    }
    return SKIPFFN_OK;
}

skipffn_status skipffn_plan(skipffn_saved *s, const uint8_t *skip_mask, int64_t N, void *stream)
{
    if (!s || N < 0 || N > s->max_tokens) return SKIPFFN_EINVAL;
    if (!skip_mask && !s->cfg.dense && N > 0) return SKIPFFN_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    // the status word is cleared together with the first plan of a handle
    if (first_use(s, st) != cudaSuccess) return SKIPFFN_ECUDA;
    s->launches[0] = 0;
    s->forwarded = 0;
    return do_plan(s, skip_mask, N, 0, st);
}

// G = X Wg^T, U = X Wu^T, H = silu(G) * U, with X = the kept rows (normalised in the pre-norm
// variant).  The tensor-core kernels take the weights as the A operand (weight rows along the
// accumulator rows) and the token rows as B; the plain-FMA kernels the other way round.
// `store_gu` = 0 writes H only.
static cudaError_t gate_up(skipffn_saved *s, int slot, int32_t NB, bool store_gu, cudaStream_t st,
                           const void *gather_x = nullptr, int64_t gather_rows = 0)
{
    const int C = s->cfg.C, I = s->cfg.I;
    const void *Xrows = s->cfg.prenorm ? s->Xn : s->Xk;
    GemmArgs g = base_args(s);
    if (use_umma(s)) {
        g.A = s->Wg; g.A2 = s->Wu; g.lda_m = C; g.lda_k = 1; g.a_outer = I;
        g.B = Xrows; g.ldb_n = C; g.ldb_k = 1; g.b_outer = s->cap_k;
        g.M = I; g.N = NB; g.n_from_nk = 1; g.K = C;
        if (s->tune[SKIPFFN_TUNE_GATHER] && !s->cfg.prenorm) { g.gather_src = gather_x; g.gather_rows = gather_rows; }
    } else {
        g.A = Xrows; g.lda_m = C; g.lda_k = 1; g.a_outer = s->cap_k;
        g.B = s->Wg; g.B2 = s->Wu; g.ldb_n = C; g.ldb_k = 1; g.b_outer = I;
        g.M = NB; g.m_from_nk = 1; g.N = I; g.K = C;
    }
    g.out0 = store_gu ? s->G : nullptr; g.out1 = store_gu ? s->U : nullptr; g.out2 = s->H; g.ldo = I;
    return run_gemm(s, slot, EPI_GATEUP, g, st);
}

static skipffn_status forward_impl(skipffn_saved *s, const void *x, const uint8_t *skip_mask, int64_t B,
                                   int64_t S, const int32_t *cu_seqlens, int32_t n_seq,
                                   const void *gamma, float eps, const void *W_gate, const void *W_up,
                                   const void *W_down, void *out, void *stream)
{
    if (!s || B < 0 || S < 0) return SKIPFFN_EINVAL;
    if ((s->cfg.prenorm != 0) != (gamma != nullptr)) return SKIPFFN_EINVAL;   // wrong entry point
    if (gamma && (!aligned16(gamma) || !(eps >= 0.0f))) return SKIPFFN_EINVAL;
    const int64_t N = B * S;
    if (N > s->max_tokens) return SKIPFFN_EINVAL;
    if (!W_gate || !W_up || !W_down || (N > 0 && (!x || !out))) return SKIPFFN_EINVAL;
    if (!aligned16(x) || !aligned16(out) || !aligned16(W_gate) || !aligned16(W_up) || !aligned16(W_down))
        return SKIPFFN_EINVAL;
    if (cu_seqlens) {   // packed batch: offsets must be non-decreasing from 0 to N
        if (n_seq < 0 || cu_seqlens[0] != 0 || cu_seqlens[n_seq] != N) return SKIPFFN_EINVAL;
        for (int i = 0; i < n_seq; ++i)
            if (cu_seqlens[i + 1] < cu_seqlens[i]) return SKIPFFN_EINVAL;
    }
    cudaStream_t st = (cudaStream_t)stream;
    const int C = s->cfg.C, I = s->cfg.I;
    s->forwarded = 0;
    if (skip_mask || s->cfg.dense || N == 0) {
        if (first_use(s, st) != cudaSuccess) return SKIPFFN_ECUDA;
        s->launches[0] = 0;
        skipffn_status r = do_plan(s, skip_mask, N, 0, st);
        if (r != SKIPFFN_OK) return r;
    } else {
        if (s->planned_N != N) return SKIPFFN_EINVAL;   // no list to reuse
        s->launches[0] = 0;
    }
    s->Wg = W_gate; s->Wu = W_up; s->Wd = W_down; s->gamma = gamma;
    if (N == 0) { s->forwarded = 1; return SKIPFFN_OK; }

    // kept rows of x -> Xk (also the residual stash when out aliases x); skipped rows -> out
    RouteArgs r;
    r.src = x; r.dst_compact = s->Xk; r.dst_identity = out; r.pos = s->pos; r.status = s->status;
    r.N = N; r.C = C; r.elem_bytes = s->esize;
    if (timed_launch(s, SLOT_ROUTE_X, st, [&] {
            return gamma ? launch_route_norm(r, s->Xn, s->rstd, gamma, eps, st) : launch_route(r, st);
        }) != cudaSuccess)
        return SKIPFFN_ECUDA;

    const int32_t NB = (int32_t)(N < s->max_kept ? N : s->max_kept);   // host bound of the kept count
    const bool tc = use_umma(s);
    // a recomputing handle keeps only H (for the down projection); its backward computes G, U, H again
    // (with the GATHER knob the launch reads its token rows from x itself; it ends before the down
    // projection writes `out`, so out may still alias x)
    if (gate_up(s, SLOT_GATEUP, NB, !s->cfg.recompute, st, x, N) != cudaSuccess) return SKIPFFN_ECUDA;

    // out[idx[r]] = Xk[r] + H Wd^T
    GemmArgs g = base_args(s);
    if (tc) {
        g.A = W_down; g.lda_m = I; g.lda_k = 1; g.a_outer = C;
        g.B = s->H; g.ldb_n = I; g.ldb_k = 1; g.b_outer = s->cap_k;
        g.M = C; g.N = NB; g.n_from_nk = 1; g.K = I;
    } else {
        g.A = s->H; g.lda_m = I; g.lda_k = 1; g.a_outer = s->cap_k;
        g.B = W_down; g.ldb_n = I; g.ldb_k = 1; g.b_outer = C;
        g.M = NB; g.m_from_nk = 1; g.N = C; g.K = I;
    }
    g.in0 = s->Xk; g.out0 = out; g.ldo = C;
    if (run_gemm(s, SLOT_DOWN, EPI_DOWN, g, st) != cudaSuccess) return SKIPFFN_ECUDA;
    s->forwarded = 1;
    return SKIPFFN_OK;
}

skipffn_status skipffn_forward(skipffn_saved *s, const void *x, const uint8_t *skip_mask, int64_t B,
                               int64_t S, const int32_t *cu_seqlens, int32_t n_seq,
                               const void *W_gate, const void *W_up, const void *W_down, void *out,
                               void *stream)
{
    return forward_impl(s, x, skip_mask, B, S, cu_seqlens, n_seq, nullptr, 0.0f, W_gate, W_up, W_down, out, stream);
}

skipffn_status skipffn_forward_prenorm(skipffn_saved *s, const void *x, const uint8_t *skip_mask, int64_t B,
                                       int64_t S, const int32_t *cu_seqlens, int32_t n_seq,
                                       const void *gamma, float eps, const void *W_gate, const void *W_up,
                                       const void *W_down, void *out, void *stream)
{
    if (!gamma) return SKIPFFN_EINVAL;
    return forward_impl(s, x, skip_mask, B, S, cu_seqlens, n_seq, gamma, eps, W_gate, W_up, W_down, out, stream);
}

static skipffn_status backward_impl(const void *dout, skipffn_saved *s, void *dx, void *dgamma, void *dW_gate,
                                    void *dW_up, void *dW_down, void *stream)
{
    if (!s || !s->forwarded) return SKIPFFN_EINVAL;
    const bool prenorm = s->cfg.prenorm != 0;
    if (!prenorm && dgamma) return SKIPFFN_EINVAL;
    if (!aligned16(dgamma)) return SKIPFFN_EINVAL;
    const int64_t N = s->planned_N;
    if (N > 0 && (!dout || !dx)) return SKIPFFN_EINVAL;
    if (!aligned16(dout) || !aligned16(dx) || !aligned16(dW_gate) || !aligned16(dW_up) || !aligned16(dW_down))
        return SKIPFFN_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    const int C = s->cfg.C, I = s->cfg.I;
    s->launches[1] = 0;
    GemmArgs g;
    const bool tc = use_umma(s);
    const int32_t NB = (int32_t)(N < s->max_kept ? N : s->max_kept);   // host bound of the kept count

    if (N > 0) {
        RouteArgs r;
        r.src = dout; r.dst_compact = s->dOk; r.dst_identity = dx; r.pos = s->pos; r.status = s->status;
        r.N = N; r.C = C; r.elem_bytes = s->esize;
        if (timed_launch(s, SLOT_ROUTE_DOUT, st, [&] { return launch_route(r, st); }) != cudaSuccess)
            return SKIPFFN_ECUDA;

        // a recomputing handle kept no G, U, H: compute them again from the kept rows
        if (s->cfg.recompute && gate_up(s, SLOT_RECOMPUTE, NB, true, st) != cudaSuccess) return SKIPFFN_ECUDA;

        // dH = dOk Wd ; dG, dU through the activation
        g = base_args(s);
        if (tc) {   // dH^T[i, t] = sum_c Wd[c, i] dOk[t, c]
            g.A = s->Wd; g.lda_m = 1; g.lda_k = I; g.a_outer = C;
            g.B = s->dOk; g.ldb_n = C; g.ldb_k = 1; g.b_outer = s->cap_k;
            g.M = I; g.N = NB; g.n_from_nk = 1; g.K = C;
            if (s->tune[SKIPFFN_TUNE_GATHER]) { g.gather_src = dout; g.gather_rows = N; }
        } else {
            g.A = s->dOk; g.lda_m = C; g.lda_k = 1; g.a_outer = s->cap_k;
            g.B = s->Wd; g.ldb_n = 1; g.ldb_k = I; g.b_outer = C;
            g.M = NB; g.m_from_nk = 1; g.N = I; g.K = C;
        }
        g.in0 = s->G; g.in1 = s->U; g.out0 = s->dG; g.out1 = s->dU; g.ldo = I;
        if (run_gemm(s, SLOT_DH, EPI_DH, g, st) != cudaSuccess) return SKIPFFN_ECUDA;
    } else if (cudaMemsetAsync(s->status, 0, 4, st) != cudaSuccess) {
        return SKIPFFN_ECUDA;
    }

    // weight gradients: reductions over the kept-token axis (K = Nk, read on the device)
    //   dWd[c, i] = sum_r dOk[r, c] H[r, i];  dWg[i, c] = sum_r dG[r, i] Xk[r, c];  dWu likewise with dU
    const int32_t kmax = NB;
    GemmArgs dw[3];
    int dw_slot[3], n_dw = 0;
    void *dw_dst[3] = {dW_down, dW_gate, dW_up};
    for (int w = 0; w < 3; ++w) {
        if (!dw_dst[w]) continue;
        GemmArgs &q = dw[n_dw];
        q = base_args(s);
        if (w == 0) {
            q.A = s->dOk; q.lda_k = C; q.B = s->H; q.ldb_k = I; q.M = C; q.N = I; q.ldo = I;
        } else {
            q.A = w == 1 ? s->dG : s->dU; q.lda_k = I; q.B = prenorm ? s->Xn : s->Xk; q.ldb_k = C;
            q.M = I; q.N = C; q.ldo = C;
        }
        q.lda_m = 1; q.ldb_n = 1; q.a_outer = s->cap_k; q.b_outer = s->cap_k;
        q.K = kmax; q.k_from_nk = 1;
        q.out0 = dw_dst[w]; q.accumulate = s->cfg.accumulate_dw;
        q.out_fp32 = s->cfg.grad_dtype_fp32 || s->cfg.dtype == SKIPFFN_FP32;
        dw_slot[n_dw++] = SLOT_DW_DOWN + w;
    }
    if (use_umma(s) && n_dw > 1) {
        // one grouped launch: the problems are independent, and together their tiles fill the
        // persistent grid's waves better than one launch each; timed under the first one's slot
        if (++s->sk_epoch <= 0) s->sk_epoch = 1;
        for (int i = 0; i < n_dw; ++i) dw[i].sk_epoch = s->sk_epoch;
        if (timed_launch(s, dw_slot[0], st, [&] { return launch_umma_dw_group(dw, n_dw, st); }) != cudaSuccess)
            return SKIPFFN_ECUDA;
    } else {
        for (int i = 0; i < n_dw; ++i)
            if (run_gemm(s, dw_slot[i], EPI_DW, dw[i], st) != cudaSuccess) return SKIPFFN_ECUDA;
    }

    if (N > 0) {   // dx[idx[r]] = dOk[r] + dG Wg + dU Wu
        g = base_args(s);
        if (tc) {   // dx^T[c, t] = sum_i Wg[i, c] dG[t, i] + Wu[i, c] dU[t, i]
            g.A = s->Wg; g.A2 = s->Wu; g.lda_m = 1; g.lda_k = C; g.a_outer = I;
            g.B = s->dG; g.B2 = s->dU; g.ldb_n = I; g.ldb_k = 1; g.b_outer = s->cap_k;
            g.M = C; g.N = NB; g.n_from_nk = 1; g.K = I;
        } else {
            g.A = s->dG; g.A2 = s->dU; g.lda_m = I; g.lda_k = 1; g.a_outer = s->cap_k;
            g.B = s->Wg; g.B2 = s->Wu; g.ldb_n = 1; g.ldb_k = C; g.b_outer = I;
            g.M = NB; g.m_from_nk = 1; g.N = C; g.K = I;
        }
        if (prenorm) { g.in0 = nullptr; g.out0 = s->dY; g.out_fp32 = 1; }   // gradient w.r.t. the normalised rows
        else { g.in0 = s->dOk; g.out0 = dx; }
        g.ldo = C;
        if (run_gemm(s, SLOT_DX, EPI_DX, g, st) != cudaSuccess) return SKIPFFN_ECUDA;
    }
    if (prenorm) {   // through the normalisation: dx rows (scattered) and the gain's gradient
        const int gfp32 = s->cfg.grad_dtype_fp32 || s->cfg.dtype == SKIPFFN_FP32;
        if (N == 0 && dgamma && !s->cfg.accumulate_dw) {
            if (cudaMemsetAsync(dgamma, 0, (size_t)C * (gfp32 ? 4 : 2), st) != cudaSuccess) return SKIPFFN_ECUDA;
        } else if (N > 0) {
            if (timed_launch(s, SLOT_NORM_BWD, st, [&] {
                    return launch_norm_bwd(s->dY, s->Xk, s->dOk, s->rstd, s->gamma, dx, dgamma, s->dg_part, s->idx, s->status,
                                           N, C, s->esize, gfp32, s->cfg.accumulate_dw, st);
                }) != cudaSuccess)
                return SKIPFFN_ECUDA;
            if (dgamma) s->launches[1] += 2;   // the slot covers three kernels: rows, then the gain's gradient in two stages
        }
    }
    return SKIPFFN_OK;
}

skipffn_status skipffn_backward(const void *dout, skipffn_saved *s, void *dx, void *dW_gate,
                                void *dW_up, void *dW_down, void *stream)
{
    if (s && s->cfg.prenorm) return SKIPFFN_EINVAL;   // wrong entry point
    return backward_impl(dout, s, dx, nullptr, dW_gate, dW_up, dW_down, stream);
}

skipffn_status skipffn_backward_prenorm(const void *dout, skipffn_saved *s, void *dx, void *dgamma,
                                        void *dW_gate, void *dW_up, void *dW_down, void *stream)
{
    if (s && !s->cfg.prenorm) return SKIPFFN_EINVAL;
    return backward_impl(dout, s, dx, dgamma, dW_gate, dW_up, dW_down, stream);
}

skipffn_status skipffn_kv_compact(const skipffn_saved *s, const void *src, void *dst, int64_t planes,
                                  int64_t row_bytes, int64_t dst_rows, const int32_t *cu_seqlens,
                                  int32_t n_seq, int32_t *kept_cu_seqlens, void *stream)
{
    if (!s || s->planned_N < 0 || planes < 0 || row_bytes <= 0 || dst_rows < 0) return SKIPFFN_EINVAL;
    if (row_bytes % 16) return SKIPFFN_EUNSUPPORTED;
    const int64_t N = s->planned_N;
    cudaStream_t st = (cudaStream_t)stream;
    if (planes > 0 && N > 0 && dst_rows > 0) {
        if (!src || !dst || !aligned16(src) || !aligned16(dst)) return SKIPFFN_EINVAL;
        // the gather runs in parallel over rows, so the two caches must not overlap
        const char *a = (const char *)src, *b = (const char *)dst;
        const int64_t src_bytes = planes * N * row_bytes, dst_bytes = planes * dst_rows * row_bytes;
        if (a < b + dst_bytes && b < a + src_bytes) return SKIPFFN_EINVAL;
        if (launch_kv_compact(src, dst, s->idx, s->status, planes, N, dst_rows, row_bytes, st) != cudaSuccess)
            return SKIPFFN_ECUDA;
    }
    if (kept_cu_seqlens) {
        if (!cu_seqlens || n_seq < 0) return SKIPFFN_EINVAL;
        if (launch_kept_cu_seqlens(cu_seqlens, kept_cu_seqlens, n_seq + 1, s->idx, s->status, st) != cudaSuccess)
            return SKIPFFN_ECUDA;
    }
    return SKIPFFN_OK;
}

size_t skipffn_summary_scratch_bytes(int64_t n_rows, int32_t C)
{
    if (n_rows < 0 || C <= 0) return 0;
    return (size_t)(((n_rows + 63) / 64) * 64 + (int64_t)DG_CHUNKS * C) * sizeof(float);
}

static bool summary_args_ok(const void *X, const int32_t *off, int32_t n_seg, int64_t n_rows, int32_t C,
                            int32_t dtype, const void *w)
{
    return n_seg >= 0 && n_rows >= 0 && n_rows < ((int64_t)1 << 31) && C > 0 && C % 8 == 0 &&
           (dtype == SKIPFFN_BF16 || dtype == SKIPFFN_FP32) && w && (n_seg == 0 || off) && (n_rows == 0 || X) &&
           aligned16(X) && aligned16(w);
}

skipffn_status skipffn_summary_forward(const void *X, const int32_t *seg_offsets, int32_t n_seg, int64_t n_rows,
                                       int32_t C, int32_t dtype, const void *w, void *xs, float *probs,
                                       void *stream)
{
    if (!summary_args_ok(X, seg_offsets, n_seg, n_rows, C, dtype, w)) return SKIPFFN_EINVAL;
    if (n_seg > 0 && (!xs || (n_rows > 0 && !probs))) return SKIPFFN_EINVAL;
    if (!aligned16(xs)) return SKIPFFN_EINVAL;
    return launch_summary_forward(X, seg_offsets, n_seg, n_rows, C, dtype, w, xs, probs, (cudaStream_t)stream) ==
                   cudaSuccess ? SKIPFFN_OK : SKIPFFN_ECUDA;
}

skipffn_status skipffn_summary_backward(const void *X, const int32_t *seg_offsets, int32_t n_seg, int64_t n_rows,
                                        int32_t C, int32_t dtype, const void *w, const float *probs,
                                        const void *dxs, void *dX, void *dw, int32_t dw_fp32, void *scratch,
                                        size_t scratch_bytes, void *stream)
{
    if (!summary_args_ok(X, seg_offsets, n_seg, n_rows, C, dtype, w)) return SKIPFFN_EINVAL;
    if (n_seg > 0 && (!dxs || !scratch || (n_rows > 0 && !probs))) return SKIPFFN_EINVAL;
    if (!aligned16(dxs) || !aligned16(dX)) return SKIPFFN_EINVAL;
    if (scratch_bytes < skipffn_summary_scratch_bytes(n_rows, C)) return SKIPFFN_EWORKSPACE;
    if (((uintptr_t)scratch & 15u) != 0) return SKIPFFN_EINVAL;
    return launch_summary_backward(X, seg_offsets, n_seg, n_rows, C, dtype, w, probs, dxs, dX, dw, dw_fp32,
                                   (float *)scratch, (cudaStream_t)stream) == cudaSuccess ? SKIPFFN_OK : SKIPFFN_ECUDA;
}

size_t skipffn_token_merge_scratch_bytes(int64_t n, int32_t C, int32_t k, int32_t dtype)
{
    if (n <= 0 || C <= 0 || k <= 0 || k > n || (dtype != SKIPFFN_BF16 && dtype != SKIPFFN_FP32)) return 0;
    return merge_scratch_bytes(n, C, k, dtype);
}

skipffn_status skipffn_token_merge(const void *X, int64_t n, int32_t C, int32_t k, int32_t dtype,
                                   int32_t *kept, int32_t *assign, void *merged, void *scratch,
                                   size_t scratch_bytes, void *stream)
{
    if (!X || !kept || !assign || !merged || !scratch || n <= 0 || k <= 0 || k > n || C <= 0) return SKIPFFN_EINVAL;
    if (dtype != SKIPFFN_BF16 && dtype != SKIPFFN_FP32) return SKIPFFN_EINVAL;
    if (C % 8 || C > 16384 || k % 4 || n > 65536) return SKIPFFN_EUNSUPPORTED;
    if (!aligned16(X) || !aligned16(merged) || ((uintptr_t)scratch & 255u)) return SKIPFFN_EINVAL;
    if (scratch_bytes < merge_scratch_bytes(n, C, k, dtype)) return SKIPFFN_EWORKSPACE;
    return launch_token_merge(X, n, C, k, dtype, kept, assign, merged, scratch, (cudaStream_t)stream) == cudaSuccess
               ? SKIPFFN_OK : SKIPFFN_ECUDA;
}

skipffn_status skipffn_token_merge_poll(void *scratch, int64_t n, int32_t C, int32_t k, int32_t dtype, void *stream,
                                        int32_t *site_out)
{
    if (!scratch || n <= 0 || k <= 0 || k > n || C <= 0 || (dtype != SKIPFFN_BF16 && dtype != SKIPFFN_FP32))
        return SKIPFFN_EINVAL;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return SKIPFFN_ECUDA;
    int32_t w[3] = {0, 0, 0};
    if (cudaMemcpy(w, merge_status_ptr(scratch, n, C, k, dtype), sizeof(w), cudaMemcpyDeviceToHost) != cudaSuccess)
        return SKIPFFN_ECUDA;
    if (site_out) *site_out = w[ST_SITE];
    return (skipffn_status)w[ST_STATUS];
}

skipffn_status skipffn_get_kept(const skipffn_saved *s, const int32_t **idx_dev, const int32_t **nk_dev)
{
    if (!s || s->planned_N < 0) return SKIPFFN_EINVAL;
    if (idx_dev) *idx_dev = s->idx;
    if (nk_dev) *nk_dev = s->status + ST_NK;
    return SKIPFFN_OK;
}

skipffn_status skipffn_get_intermediate(const skipffn_saved *s, int32_t which, const void **ptr_dev)
{
    if (!s || !ptr_dev) return SKIPFFN_EINVAL;
    const void *t[8] = {s->G, s->U, s->H, s->dG, s->dU, s->Xk, s->dOk, s->Xn};
    if (which < 0 || which > 7 || (which == 7 && !s->cfg.prenorm)) return SKIPFFN_EINVAL;
    *ptr_dev = t[which];
    return SKIPFFN_OK;
}

skipffn_status skipffn_poll(skipffn_saved *s, void *stream, int32_t *site_out)
{
    if (!s) return SKIPFFN_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    if (s->cfg.debug && s->planned_N >= 0 && launch_check_guards(s->guards, s->status, st) != cudaSuccess) return SKIPFFN_ECUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SKIPFFN_ECUDA;
    int32_t w[3] = {0, 0, 0};
    if (cudaMemcpy(w, s->status, sizeof(w), cudaMemcpyDeviceToHost) != cudaSuccess) return SKIPFFN_ECUDA;
    if (site_out) *site_out = w[ST_SITE];
    if (w[ST_STATUS] != 0) {
        if (cudaMemset(s->status + ST_STATUS, 0, 8) != cudaSuccess) return SKIPFFN_ECUDA;
        return (skipffn_status)w[ST_STATUS];
    }
    return SKIPFFN_OK;
}

int32_t skipffn_last_launches(const skipffn_saved *s, int32_t which)
{
    return (s && (which == 0 || which == 1)) ? s->launches[which] : -1;
}

int32_t skipffn_schedule_segment(int32_t workers, int32_t tiles, int32_t k_blocks, int32_t split_k,
                                 int32_t worker, int32_t i, int32_t *seg)
{
    if (workers <= 0 || tiles < 0 || k_blocks < 0 || worker < 0 || worker >= workers) return -1;
    Sched sc;
    sc.init(worker, workers, tiles, k_blocks, split_k);
    const int n = sc.count();
    if (seg && i >= 0 && i < n) {
        const Seg g = sc.get(i);
        seg[0] = g.tile; seg[1] = g.kb0; seg[2] = g.kb1; seg[3] = g.partial; seg[4] = g.src_lo;
    }
    return n;
}

int32_t skipffn_schedule_plan_segment(int32_t workers, int32_t panels, int32_t token_tiles, int32_t k_blocks,
                                      int32_t min_saving, int32_t group_mode, int32_t worker, int32_t i, int32_t *seg)
{
    if (workers <= 0 || panels < 0 || token_tiles <= 0 || k_blocks < 0 || worker < 0 || worker >= workers ||
        (int64_t)panels * token_tiles > INT_MAX)
        return -1;
    Plan pl;
    pl.init(worker, workers, panels, token_tiles, k_blocks, min_saving, group_mode);
    const int n = pl.count();
    if (seg && i >= 0 && i < n) {
        const Seg g = pl.get(i);
        seg[0] = g.tile; seg[1] = g.kb0; seg[2] = g.kb1; seg[3] = g.partial;
        seg[4] = pl.slot_worker(g.src_lo);
        seg[5] = pl.gw;
    }
    return n;
}

double skipffn_flops(const skipffn_config *cfg, int64_t n_kept)
{
    if (!cfg) return 0.0;
    return 18.0 * (double)n_kept * (double)cfg->C * (double)cfg->I;
}

const char *skipffn_strerror(skipffn_status st)
{
    switch (st) {
    case SKIPFFN_OK: return "ok";
    case SKIPFFN_EINVAL: return "invalid argument";
    case SKIPFFN_EUNSUPPORTED: return "unsupported shape";
    case SKIPFFN_EWORKSPACE: return "workspace too small";
    case SKIPFFN_ECUDA: return "CUDA call failed";
    case SKIPFFN_ETIMEOUT: return "device-side wait timed out";
    case SKIPFFN_EDEBUG: return "debug check failed";
    }
    return "unknown status";
}

}  // extern "C"
