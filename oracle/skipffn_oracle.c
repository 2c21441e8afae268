/*
 * Skip-FFN reference oracle -- TEST INFRASTRUCTURE, not part of the product.
 * (Parity unpinned: the merge OPERATOR of skipffn_oracle_token_merge / skipffn_oracle_merge_given,
 * which the paper does not define; everything else below is pinned.)
 *
 * A plain, slow, obviously-correct CPU statement of what the Skip-FFN decoder
 * sublayer computes, forward and backward, in double precision.  It shares no
 * code, header, table or constant with the CUDA library; only tests, the smoke
 * check and the benchmark's cpu_baseline leg may call it.
 *
 * Definition followed (paper section 4.2, "Training speed-up: skip FFN"):
 *   retained tokens (Eq. 4):  h = h_attn + FFN(h_attn)
 *   skipped  tokens (Eq. 5):  h = h_attn
 * FFN body: the paper's backbones are LLaMA-3-8B / Vicuna, and its cost model
 * (section 6.2: 3*N*C*M multiply-adds; Table 1: 10.5*L*N*C^2 and 5.64 B FFN
 * parameters) fixes three C x M matrices, i.e. the bias-free SwiGLU
 *   FFN(x) = ( silu(x W_gate^T) * (x W_up^T) ) W_down^T ,  silu(z) = z / (1 + exp(-z)).
 * Backward is the exact derivative of that definition (the paper's claim is a
 * training speed-up, so the vjp is on the path).
 *
 * Layouts (all row-major, contiguous):
 *   x, dout, out, dx : [N, C]      skip_mask : [N] bytes, nonzero = skipped
 *   W_gate, W_up     : [I, C]      W_down    : [C, I]
 * Everything is evaluated one token at a time; no compaction, tiling, blocking
 * or reordering beyond the definition.  OpenMP only spreads independent
 * iterations (tokens, or intermediate indices i) over host cores.
 *
 * Pins (tests/test_oracle_pins.py): pure-Python per-token brute force on tiny
 * inputs, scalar closed form, W_gate = 0 / W_down = 0 identities, all-kept ==
 * dense FFN via a library matmul, all-skipped == input, central finite
 * differences for every gradient, linearity and homogeneity properties, and the
 * per-layer skip error of Eq. 8.  Skip KV-cache: library boolean indexing, a set-difference
 * restatement of Eq. 7 on tagged rows, and hand-written tiny cases.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ascending list of kept token indices (mask byte == 0); returns their count */
int64_t skipffn_oracle_compact(const uint8_t *skip_mask, int64_t N, int32_t *idx)
{
    int64_t nk = 0;
    for (int64_t t = 0; t < N; ++t)
        if (skip_mask[t] == 0)
            idx[nk++] = (int32_t)t;
    return nk;
}

static double sigmoid(double z) { return 1.0 / (1.0 + exp(-z)); }

/* g[i], u[i], h[i] of one token (the three SwiGLU intermediates) */
static void token_intermediates(const double *xt, const double *Wg, const double *Wu,
                                int64_t C, int64_t I, double *g, double *u, double *h)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < I; ++i) {
        double sg = 0.0, su = 0.0;
        for (int64_t c = 0; c < C; ++c) {
            sg += xt[c] * Wg[i * C + c];
            su += xt[c] * Wu[i * C + c];
        }
        g[i] = sg;
        u[i] = su;
        h[i] = sg * sigmoid(sg) * su;
    }
}

/* out[t,:] for every token: Eq. 5 for skipped rows, Eq. 4 for the others.
 * ffn_only != 0 returns FFN(x) alone on kept rows (and 0 on skipped rows). */
void skipffn_oracle_forward(const double *x, const uint8_t *skip_mask, const double *Wg,
                            const double *Wu, const double *Wd, int64_t N, int64_t C,
                            int64_t I, int ffn_only, double *out)
{
    double *g = (double *)malloc(sizeof(double) * (size_t)I * 3);
    double *u = g + I, *h = u + I;
    for (int64_t t = 0; t < N; ++t) {
        const double *xt = x + t * C;
        double *ot = out + t * C;
        if (skip_mask[t] != 0) {
            for (int64_t c = 0; c < C; ++c)
                ot[c] = ffn_only ? 0.0 : xt[c];
            continue;
        }
        token_intermediates(xt, Wg, Wu, C, I, g, u, h);
#pragma omp parallel for schedule(static)
        for (int64_t c = 0; c < C; ++c) {
            double y = 0.0;
            for (int64_t i = 0; i < I; ++i)
                y += h[i] * Wd[c * I + i];
            ot[c] = ffn_only ? y : xt[c] + y;
        }
    }
    free(g);
}

/* Gradients of L = sum(dout * out) w.r.t. x and the three matrices.
 * dWg, dWu, dWd may be NULL (then only dx is produced); when given they are
 * overwritten (zeroed first), never accumulated into. */
void skipffn_oracle_backward(const double *x, const uint8_t *skip_mask, const double *Wg,
                             const double *Wu, const double *Wd, const double *dout,
                             int64_t N, int64_t C, int64_t I, double *dx, double *dWg,
                             double *dWu, double *dWd)
{
    double *g = (double *)malloc(sizeof(double) * (size_t)I * 6);
    double *u = g + I, *h = u + I, *dh = h + I, *dg = dh + I, *du = dg + I;
    if (dWg) memset(dWg, 0, sizeof(double) * (size_t)I * (size_t)C);
    if (dWu) memset(dWu, 0, sizeof(double) * (size_t)I * (size_t)C);
    if (dWd) memset(dWd, 0, sizeof(double) * (size_t)I * (size_t)C);
    for (int64_t t = 0; t < N; ++t) {
        const double *xt = x + t * C, *dot = dout + t * C;
        double *dxt = dx + t * C;
        if (skip_mask[t] != 0) { /* derivative of the identity */
            for (int64_t c = 0; c < C; ++c)
                dxt[c] = dot[c];
            continue;
        }
        token_intermediates(xt, Wg, Wu, C, I, g, u, h);
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < I; ++i) {
            double s = 0.0;
            for (int64_t c = 0; c < C; ++c)
                s += dot[c] * Wd[c * I + i];
            dh[i] = s;
            double sg = sigmoid(g[i]);
            du[i] = s * (g[i] * sg);                                   /* d/du of silu(g)*u */
            dg[i] = s * u[i] * (sg * (1.0 + g[i] * (1.0 - sg)));       /* silu'(g)          */
            if (dWd)
                for (int64_t c = 0; c < C; ++c)
                    dWd[c * I + i] += dot[c] * h[i];
            if (dWg)
                for (int64_t c = 0; c < C; ++c)
                    dWg[i * C + c] += dg[i] * xt[c];
            if (dWu)
                for (int64_t c = 0; c < C; ++c)
                    dWu[i * C + c] += du[i] * xt[c];
        }
#pragma omp parallel for schedule(static)
        for (int64_t c = 0; c < C; ++c) {
            double s = 0.0;
            for (int64_t i = 0; i < I; ++i)
                s += dg[i] * Wg[i * C + c] + du[i] * Wu[i * C + c];
            dxt[c] = dot[c] + s;
        }
    }
    free(g);
}

/* Sampled mode, rows: out[t,:] and dx[t,:] for the listed tokens only (any order,
 * kept or skipped), written to out_rows / dx_rows [n_tokens, C].  Same per-element
 * arithmetic as the full functions; dout / dx_rows may be NULL for forward only. */
void skipffn_oracle_rows(const double *x, const uint8_t *skip_mask, const double *Wg,
                         const double *Wu, const double *Wd, const double *dout, int64_t C,
                         int64_t I, const int64_t *tokens, int64_t n_tokens, double *out_rows,
                         double *dx_rows)
{
    for (int64_t k = 0; k < n_tokens; ++k) {
        int64_t t = tokens[k];
        uint8_t one = skip_mask[t];
        skipffn_oracle_forward(x + t * C, &one, Wg, Wu, Wd, 1, C, I, 0, out_rows + k * C);
        if (dout && dx_rows)
            skipffn_oracle_backward(x + t * C, &one, Wg, Wu, Wd, dout + t * C, 1, C, I,
                                    dx_rows + k * C, NULL, NULL, NULL);
    }
}

/* Sampled mode, weight gradients: for each listed intermediate index i the exact
 *   dW_gate[i,:], dW_up[i,:]  (rows, [n_cols, C])  and  dW_down[:,i]  (column, [n_cols, C])
 * summed over every kept token.  Needs only g, u, dh at index i per token: O(N_kept * C) per i. */
void skipffn_oracle_dw_columns(const double *x, const uint8_t *skip_mask, const double *Wg,
                               const double *Wu, const double *Wd, const double *dout,
                               int64_t N, int64_t C, int64_t I, const int64_t *cols,
                               int64_t n_cols, double *dWg_rows, double *dWu_rows,
                               double *dWd_cols)
{
#pragma omp parallel for schedule(dynamic)
    for (int64_t k = 0; k < n_cols; ++k) {
        int64_t i = cols[k];
        double *rg = dWg_rows + k * C, *ru = dWu_rows + k * C, *rd = dWd_cols + k * C;
        for (int64_t c = 0; c < C; ++c)
            rg[c] = ru[c] = rd[c] = 0.0;
        for (int64_t t = 0; t < N; ++t) {
            if (skip_mask[t] != 0)
                continue;
            const double *xt = x + t * C, *dot = dout + t * C;
            double g = 0.0, u = 0.0, dh = 0.0;
            for (int64_t c = 0; c < C; ++c) {
                g += xt[c] * Wg[i * C + c];
                u += xt[c] * Wu[i * C + c];
                dh += dot[c] * Wd[c * I + i];
            }
            double sg = sigmoid(g);
            double h = g * sg * u;
            double du = dh * (g * sg);
            double dg = dh * u * (sg * (1.0 + g * (1.0 - sg)));
            for (int64_t c = 0; c < C; ++c) {
                rd[c] += dot[c] * h;
                rg[c] += dg * xt[c];
                ru[c] += du * xt[c];
            }
        }
    }
}

/* Skip KV-cache (section 4.3, Eq. 7): the cache after prefill is the set difference
 * K_cache \ K_skip (likewise V), i.e. the rows of the retained tokens in their original order.
 * src: [planes, N, row_bytes] bytes; dst: [planes, n_kept, row_bytes], written densely.
 * Returns n_kept.  Plain byte copies, one token at a time. */
int64_t skipffn_oracle_kv_compact(const uint8_t *src, const uint8_t *skip_mask, int64_t planes,
                                  int64_t N, int64_t row_bytes, uint8_t *dst)
{
    int64_t n_kept = 0;
    for (int64_t t = 0; t < N; ++t)
        if (skip_mask[t] == 0)
            ++n_kept;
    for (int64_t p = 0; p < planes; ++p) {
        int64_t r = 0;
        for (int64_t t = 0; t < N; ++t) {
            if (skip_mask[t] != 0)
                continue; /* a skipped token's key / value leaves the cache */
            memcpy(dst + (p * n_kept + r) * row_bytes, src + (p * N + t) * row_bytes, (size_t)row_bytes);
            ++r;
        }
    }
    return n_kept;
}

/* Sequence offsets of the pruned cache: kept_cu[s] = number of retained tokens before cu[s]. */
void skipffn_oracle_kept_cu_seqlens(const uint8_t *skip_mask, const int32_t *cu, int64_t n_entries,
                                    int32_t *kept_cu)
{
    for (int64_t s = 0; s < n_entries; ++s) {
        int32_t c = 0;
        for (int64_t t = 0; t < cu[s]; ++t)
            if (skip_mask[t] == 0)
                ++c;
        kept_cu[s] = c;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Pre-norm variant.  The paper writes FFN(h_attn) (Eq. 4) and does not mention a normalisation,
 * but the blocks of its LLaMA-3 / Vicuna backbones compute h + FFN(RMSNorm(h)).  This variant
 * applies the textbook RMSNorm to the FFN input of retained tokens only:
 *     rstd = 1 / sqrt(mean_c x[c]^2 + eps),   xn[c] = x[c] * rstd * gamma[c],
 *     out  = x + FFN(xn)                      (skipped tokens: out = x, Eq. 5, unchanged).
 * Backward is the exact derivative; with xh = x * rstd, gy = gamma * dxn:
 *     dgamma[c] = sum over retained tokens of dxn[c] * xh[c]
 *     dx[c]     = dout[c] + rstd * (gy[c] - xh[c] * mean_c(gy * xh)).
 * Pins: rows of unit RMS with gamma = 1, eps = 0 reproduce the plain functions above exactly;
 * scale invariance in x (eps = 0); fp64 autograd of a library restatement; finite differences.
 */
static double row_rstd(const double *xt, int64_t C, double eps)
{
    double ss = 0.0;
    for (int64_t c = 0; c < C; ++c)
        ss += xt[c] * xt[c];
    return 1.0 / sqrt(ss / (double)C + eps);
}

void skipffn_oracle_forward_prenorm(const double *x, const uint8_t *skip_mask, const double *gamma,
                                    double eps, const double *Wg, const double *Wu, const double *Wd,
                                    int64_t N, int64_t C, int64_t I, double *out)
{
    double *xn = (double *)malloc(sizeof(double) * (size_t)C);
    uint8_t keep = 0;
    for (int64_t t = 0; t < N; ++t) {
        const double *xt = x + t * C;
        double *ot = out + t * C;
        if (skip_mask[t] != 0) {
            for (int64_t c = 0; c < C; ++c)
                ot[c] = xt[c];
            continue;
        }
        double rstd = row_rstd(xt, C, eps);
        for (int64_t c = 0; c < C; ++c)
            xn[c] = xt[c] * rstd * gamma[c];
        /* FFN(xn) alone, then the residual of the un-normalised row */
        skipffn_oracle_forward(xn, &keep, Wg, Wu, Wd, 1, C, I, 1, ot);
        for (int64_t c = 0; c < C; ++c)
            ot[c] += xt[c];
    }
    free(xn);
}

void skipffn_oracle_backward_prenorm(const double *x, const uint8_t *skip_mask, const double *gamma,
                                     double eps, const double *Wg, const double *Wu, const double *Wd,
                                     const double *dout, int64_t N, int64_t C, int64_t I, double *dx,
                                     double *dgamma, double *dWg, double *dWu, double *dWd)
{
    double *xn = (double *)malloc(sizeof(double) * (size_t)C * 2);
    double *dxn = xn + C;
    double *tg = NULL, *tu = NULL, *td = NULL;
    uint8_t keep = 0;
    for (int64_t c = 0; c < C; ++c)
        dgamma[c] = 0.0;
    if (dWg) { memset(dWg, 0, sizeof(double) * (size_t)I * (size_t)C); tg = (double *)malloc(sizeof(double) * (size_t)I * (size_t)C); }
    if (dWu) { memset(dWu, 0, sizeof(double) * (size_t)I * (size_t)C); tu = (double *)malloc(sizeof(double) * (size_t)I * (size_t)C); }
    if (dWd) { memset(dWd, 0, sizeof(double) * (size_t)I * (size_t)C); td = (double *)malloc(sizeof(double) * (size_t)I * (size_t)C); }
    for (int64_t t = 0; t < N; ++t) {
        const double *xt = x + t * C, *dot = dout + t * C;
        double *dxt = dx + t * C;
        if (skip_mask[t] != 0) {
            for (int64_t c = 0; c < C; ++c)
                dxt[c] = dot[c];
            continue;
        }
        double rstd = row_rstd(xt, C, eps);
        for (int64_t c = 0; c < C; ++c)
            xn[c] = xt[c] * rstd * gamma[c];
        /* gradient of the FFN branch w.r.t. its input xn: the plain backward gives dout + that */
        skipffn_oracle_backward(xn, &keep, Wg, Wu, Wd, dot, 1, C, I, dxn, tg, tu, td);
        for (int64_t c = 0; c < C; ++c)
            dxn[c] -= dot[c];
        int64_t nW = I * C;
        if (dWg) for (int64_t k = 0; k < nW; ++k) dWg[k] += tg[k];
        if (dWu) for (int64_t k = 0; k < nW; ++k) dWu[k] += tu[k];
        if (dWd) for (int64_t k = 0; k < nW; ++k) dWd[k] += td[k];
        double m = 0.0;
        for (int64_t c = 0; c < C; ++c) {
            double xh = xt[c] * rstd;
            dgamma[c] += dxn[c] * xh;
            m += gamma[c] * dxn[c] * xh;
        }
        m /= (double)C;
        for (int64_t c = 0; c < C; ++c) {
            double xh = xt[c] * rstd;
            dxt[c] = dot[c] + rstd * (gamma[c] * dxn[c] - xh * m);
        }
    }
    free(xn);
    free(tg); free(tu); free(td);
}

/* ---------------------------------------------------------------------------------------------
 * Adaptive summary token (section 4.2, Eq. 6):  x_s = softmax(X w^T)^T X, with X [n, C] the retained
 * or skipped visual tokens of one sample and w [C] the layer's only weight.  Segments of a packed
 * X are processed independently: rows off[s] .. off[s+1]-1 give xs[s].  An empty segment gives 0.
 * Backward for L = sum(dxs * xs): with p = softmax(X w), a_i = dxs . X_i, t = sum_j p_j a_j,
 * ds_i = p_i (a_i - t):   dX_i = p_i dxs + ds_i w,   dw = sum_i ds_i X_i.
 * Pins: w = 0 gives the mean of the rows; a one-row segment returns the row; a large score gap
 * selects one row; the softmax weights are a library softmax; fp64 autograd; finite differences.
 */
void skipffn_oracle_summary_forward(const double *X, const int32_t *off, int64_t n_seg, int64_t C,
                                    const double *w, double *xs, double *probs)
{
    for (int64_t s = 0; s < n_seg; ++s) {
        int64_t lo = off[s], hi = off[s + 1];
        double *y = xs + s * C;
        for (int64_t c = 0; c < C; ++c)
            y[c] = 0.0;
        if (hi <= lo)
            continue;
        double mx = -INFINITY;
        for (int64_t i = lo; i < hi; ++i) {
            double sc = 0.0;
            for (int64_t c = 0; c < C; ++c)
                sc += X[i * C + c] * w[c];
            probs[i] = sc;
            if (sc > mx)
                mx = sc;
        }
        double den = 0.0;
        for (int64_t i = lo; i < hi; ++i) {
            probs[i] = exp(probs[i] - mx);
            den += probs[i];
        }
        for (int64_t i = lo; i < hi; ++i) {
            probs[i] /= den;
            for (int64_t c = 0; c < C; ++c)
                y[c] += probs[i] * X[i * C + c];
        }
    }
}

void skipffn_oracle_summary_backward(const double *X, const int32_t *off, int64_t n_seg, int64_t C,
                                     const double *w, const double *dxs, double *dX, double *dw)
{
    int64_t total = off[n_seg];
    double *probs = (double *)malloc(sizeof(double) * (size_t)(total > 0 ? total : 1));
    double *xs = (double *)malloc(sizeof(double) * (size_t)(n_seg > 0 ? n_seg : 1) * (size_t)C);
    skipffn_oracle_summary_forward(X, off, n_seg, C, w, xs, probs);
    for (int64_t c = 0; c < C; ++c)
        dw[c] = 0.0;
    for (int64_t s = 0; s < n_seg; ++s) {
        const double *g = dxs + s * C;
        double t = 0.0;
        for (int64_t i = off[s]; i < off[s + 1]; ++i) {
            double a = 0.0;
            for (int64_t c = 0; c < C; ++c)
                a += g[c] * X[i * C + c];
            t += probs[i] * a;
        }
        for (int64_t i = off[s]; i < off[s + 1]; ++i) {
            double a = 0.0;
            for (int64_t c = 0; c < C; ++c)
                a += g[c] * X[i * C + c];
            double ds = probs[i] * (a - t);
            for (int64_t c = 0; c < C; ++c) {
                dX[i * C + c] = probs[i] * g[c] + ds * w[c];
                dw[c] += ds * X[i * C + c];
            }
        }
    }
    free(probs);
    free(xs);
}

/* ---------------------------------------------------------------------------------------------
 * Token merge of the skipped tokens (section 4.1, three steps):
 *   1. cosine similarity between every pair of tokens; an average similarity per token;
 *   2. keep the k tokens with the LOWEST average similarity (the most distinctive ones);
 *   3. merge each of the other n-k tokens into the most similar kept token.
 * Readings where the paper is silent: the average runs over all n tokens including the token
 * itself (leaving it out is a monotone change, so the order is the same); ties in step 2 go to
 * the lower token index; the kept tokens are listed in ascending token order; ties in step 3 go
 * to the first kept token in that list; the merge operator is NOT stated in the paper -- this
 * oracle takes the mean of the kept token and everything merged into it ("parity unpinned" for
 * that operator; steps 1-3 are pinned by brute force and closed forms).
 * Outputs: avg[n]; kept[k] ascending token indices; assign[n] = position in `kept` of the token's
 * target (a kept token maps to itself); merged[k, C].  A zero row has similarity 0 with everything.
 */
void skipffn_oracle_token_merge(const double *X, int64_t n, int64_t C, int64_t k, double *avg,
                                int32_t *kept, int32_t *assign, double *merged)
{
    double *rn = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    for (int64_t i = 0; i < n; ++i) {
        double ss = 0.0;
        for (int64_t c = 0; c < C; ++c)
            ss += X[i * C + c] * X[i * C + c];
        rn[i] = ss > 0.0 ? 1.0 / sqrt(ss) : 0.0;
    }
    for (int64_t i = 0; i < n; ++i) {
        double s = 0.0;
        for (int64_t j = 0; j < n; ++j) {
            double d = 0.0;
            for (int64_t c = 0; c < C; ++c)
                d += X[i * C + c] * X[j * C + c];
            s += d * rn[i] * rn[j];
        }
        avg[i] = s / (double)n;
    }
    /* rank by (avg, index); keep ranks 0..k-1, listed by ascending index */
    int64_t nk = 0;
    for (int64_t i = 0; i < n; ++i) {
        int64_t rank = 0;
        for (int64_t j = 0; j < n; ++j)
            if (avg[j] < avg[i] || (avg[j] == avg[i] && j < i))
                ++rank;
        if (rank < k)
            kept[nk++] = (int32_t)i;
    }
    double *cnt = (double *)malloc(sizeof(double) * (size_t)(k > 0 ? k : 1));
    for (int64_t j = 0; j < k; ++j) {
        cnt[j] = 1.0;
        assign[kept[j]] = (int32_t)j;
        for (int64_t c = 0; c < C; ++c)
            merged[j * C + c] = X[(int64_t)kept[j] * C + c];
    }
    for (int64_t i = 0, q = 0; i < n; ++i) {
        if (q < k && kept[q] == i) { ++q; continue; } /* a kept token */
        int64_t best = 0;
        double best_s = -INFINITY;
        for (int64_t j = 0; j < k; ++j) {
            double d = 0.0;
            for (int64_t c = 0; c < C; ++c)
                d += X[i * C + c] * X[(int64_t)kept[j] * C + c];
            d *= rn[i] * rn[kept[j]];
            if (d > best_s) { best_s = d; best = j; }
        }
        assign[i] = (int32_t)best;
        cnt[best] += 1.0;
        for (int64_t c = 0; c < C; ++c)
            merged[best * C + c] += X[i * C + c];
    }
    for (int64_t j = 0; j < k; ++j)
        for (int64_t c = 0; c < C; ++c)
            merged[j * C + c] /= cnt[j];
    free(rn);
    free(cnt);
}

/* The merge operator alone, for a given assignment (used to compare merged rows when the
 * assignment itself was decided elsewhere): mean over {t : assign[t] == j}. */
void skipffn_oracle_merge_given(const double *X, int64_t n, int64_t C, int64_t k, const int32_t *assign,
                                double *merged)
{
    double *cnt = (double *)calloc((size_t)(k > 0 ? k : 1), sizeof(double));
    for (int64_t j = 0; j < k * C; ++j)
        merged[j] = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        cnt[assign[i]] += 1.0;
        for (int64_t c = 0; c < C; ++c)
            merged[(int64_t)assign[i] * C + c] += X[i * C + c];
    }
    for (int64_t j = 0; j < k; ++j)
        for (int64_t c = 0; c < C; ++c)
            merged[j * C + c] /= (cnt[j] > 0.0 ? cnt[j] : 1.0);
    free(cnt);
}
