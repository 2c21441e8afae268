"""Pins for the fp64 CPU oracle: it is checked against things other than itself --
pure-Python brute force, closed forms, identities the paper fixes (Eq. 4 / Eq. 5 / Eq. 8),
library routines (numpy matmul, torch autograd in fp64) and central finite differences."""
import math
import os

import numpy as np
import pytest

import oracle
import workloads as wl

RNG = np.random.default_rng(1234)


def _rand_case(N, C, I, p_skip=0.5, seed=0):
    r = np.random.default_rng(seed)
    x = r.normal(size=(N, C))
    wg = r.normal(size=(I, C)) * 0.7
    wu = r.normal(size=(I, C)) * 0.7
    wd = r.normal(size=(C, I)) * 0.7
    dout = r.normal(size=(N, C))
    mask = (r.random(N) < p_skip).astype(np.uint8)
    return x, mask, wg, wu, wd, dout


# ------------------------------------------------------------------ index list
def test_compact_bruteforce_and_invariants():
    for seed in range(5):
        r = np.random.default_rng(seed)
        for N in (0, 1, 2, 31, 32, 33, 1000):
            m = (r.random(N) < 0.6).astype(np.uint8) * r.integers(1, 255, size=N).astype(np.uint8)
            idx = oracle.compact(m)
            assert idx.dtype == np.int32
            assert idx.tolist() == [t for t in range(N) if m[t] == 0]
            assert idx.size == N - np.count_nonzero(m)
            assert np.all(np.diff(idx) > 0)


def test_compact_structured_highres_closed_form():
    w = wl.config3(C=8, I=8)          # mask layout does not depend on C, I
    idx = oracle.compact(w.skip_mask)
    S = 20 + 48 * 48 + 20
    assert idx.size == 4 * (12 * 24 + 40) == 1312
    first = idx[idx < S]
    vis = first[(first >= 20) & (first < 20 + 2304)] - 20
    assert vis.size == 288
    assert np.all((vis // 48) % 4 == 0) and np.all((vis % 48) % 2 == 0)


# ------------------------------------------------------------------ forward values
def _py_token(xt, wg, wu, wd):
    """Pure-Python SwiGLU FFN of one token, written from the definition."""
    C, I = len(xt), len(wg)
    h = []
    for i in range(I):
        g = sum(xt[c] * wg[i][c] for c in range(C))
        u = sum(xt[c] * wu[i][c] for c in range(C))
        h.append(g / (1.0 + math.exp(-g)) * u)
    return [sum(h[i] * wd[c][i] for i in range(I)) for c in range(C)]


@pytest.mark.parametrize("N,C,I", [(5, 4, 6), (7, 3, 2), (4, 8, 12)])
def test_forward_bruteforce_tiny(N, C, I):
    x, mask, wg, wu, wd, _ = _rand_case(N, C, I, seed=N + C)
    mask[0], mask[-1] = 0, 1
    out = oracle.forward(x, mask, wg, wu, wd)
    for t in range(N):
        if mask[t]:
            assert out[t].tolist() == x[t].tolist()
        else:
            y = _py_token(x[t].tolist(), wg.tolist(), wu.tolist(), wd.tolist())
            np.testing.assert_allclose(out[t], x[t] + np.array(y), rtol=1e-13, atol=1e-13)


def test_forward_scalar_closed_form():
    # C = I = 1: out = x + silu(x*wg) * (x*wu) * wd
    for xv, g, u, d in [(0.5, 2.0, -3.0, 0.25), (-1.5, 0.3, 0.7, -2.0), (2.0, -1.0, 1.0, 1.0)]:
        out = oracle.forward([[xv]], [0], [[g]], [[u]], [[d]])
        z = xv * g
        want = xv + z / (1 + math.exp(-z)) * (xv * u) * d
        assert abs(out[0, 0] - want) < 1e-15
    # a hand-computed value: x=1, wg=0 -> silu(0)=0 -> out = x exactly
    assert oracle.forward([[1.0]], [0], [[0.0]], [[5.0]], [[7.0]])[0, 0] == 1.0
    # x=1, wg=ln(3): sigmoid(ln 3) = 3/4 -> silu = 0.75*ln3 ; wu=2, wd=4 -> out = 1 + 6*ln3
    out = oracle.forward([[1.0]], [0], [[math.log(3.0)]], [[2.0]], [[4.0]])
    assert abs(out[0, 0] - (1 + 6 * math.log(3.0))) < 1e-14


def test_zero_gate_or_zero_down_is_identity():
    x, mask, wg, wu, wd, _ = _rand_case(6, 5, 7, p_skip=0.3)
    assert np.array_equal(oracle.forward(x, mask, np.zeros_like(wg), wu, wd), x)
    assert np.array_equal(oracle.forward(x, mask, wg, wu, np.zeros_like(wd)), x)


def test_all_skipped_is_input_bitwise_and_zero_dw():
    x, _, wg, wu, wd, dout = _rand_case(9, 6, 10)
    x[2, 3] = np.nan
    x[4, 0] = -0.0
    x[5, 1] = np.inf
    mask = np.full(9, 7, dtype=np.uint8)
    out = oracle.forward(x, mask, wg, wu, wd)
    assert out.tobytes() == x.tobytes()
    dx, dwg, dwu, dwd = oracle.backward(x, mask, wg, wu, wd, dout)
    assert dx.tobytes() == dout.tobytes()
    assert not dwg.any() and not dwu.any() and not dwd.any()


def test_all_kept_equals_dense_ffn_library_matmul():
    from scipy.special import expit
    x, _, wg, wu, wd, _ = _rand_case(33, 24, 40, seed=3)
    mask = np.zeros(33, dtype=np.uint8)
    g = x @ wg.T
    dense = x + (g * expit(g) * (x @ wu.T)) @ wd.T
    np.testing.assert_allclose(oracle.forward(x, mask, wg, wu, wd), dense, rtol=1e-12, atol=1e-12)


def test_masked_dense_restatement_and_skip_error_eq8():
    """out = x + keep * FFN_dense(x); on a skipped row the dense output differs from the skip
    output by FFN(x) of that row, whose 2-norm is the per-layer skip error of Eq. 8."""
    from scipy.special import expit
    x, mask, wg, wu, wd, _ = _rand_case(21, 16, 28, seed=5)
    g = x @ wg.T
    ffn = (g * expit(g) * (x @ wu.T)) @ wd.T
    keep = (mask == 0)[:, None]
    out_skip = oracle.forward(x, mask, wg, wu, wd)
    np.testing.assert_allclose(out_skip, x + keep * ffn, rtol=1e-12, atol=1e-12)
    out_dense = oracle.forward(x, np.zeros_like(mask), wg, wu, wd)
    sk = mask != 0
    np.testing.assert_allclose((out_dense - out_skip)[sk], ffn[sk], rtol=1e-11, atol=1e-12)
    eps = np.linalg.norm((out_dense - out_skip)[sk], axis=1)
    np.testing.assert_allclose(eps, np.linalg.norm(ffn[sk], axis=1), rtol=1e-11)
    # ffn_only mode
    np.testing.assert_allclose(oracle.forward(x, mask, wg, wu, wd, ffn_only=True), keep * ffn,
                               rtol=1e-12, atol=1e-12)


def test_token_permutation_equivariance_and_homogeneity():
    x, mask, wg, wu, wd, _ = _rand_case(13, 8, 12, seed=8)
    perm = np.random.default_rng(0).permutation(13)
    a = oracle.forward(x, mask, wg, wu, wd)
    b = oracle.forward(x[perm], mask[perm], wg, wu, wd)
    np.testing.assert_allclose(b, a[perm], rtol=0, atol=0)
    c = oracle.forward(x, mask, wg, wu, -2.5 * wd)
    np.testing.assert_allclose(c - x, -2.5 * (a - x), rtol=1e-12, atol=1e-13)


def test_poisoned_skipped_rows_do_not_leak():
    x, mask, wg, wu, wd, dout = _rand_case(12, 6, 9, seed=11)
    xp, dp = x.copy(), dout.copy()
    xp[mask != 0] = np.nan
    dp[mask != 0] = np.inf
    a = oracle.forward(x, mask, wg, wu, wd)
    b = oracle.forward(xp, mask, wg, wu, wd)
    kept = mask == 0
    assert np.array_equal(a[kept], b[kept])
    ga = oracle.backward(x, mask, wg, wu, wd, dout)
    gb = oracle.backward(xp, mask, wg, wu, wd, dp)
    assert np.array_equal(ga[0][kept], gb[0][kept])
    for u, v in zip(ga[1:], gb[1:]):
        assert np.array_equal(u, v)


# ------------------------------------------------------------------ backward values
def _loss(x, mask, wg, wu, wd, dout):
    return float(np.sum(dout * oracle.forward(x, mask, wg, wu, wd)))


def test_backward_central_finite_differences():
    N, C, I = 5, 4, 6
    x, mask, wg, wu, wd, dout = _rand_case(N, C, I, seed=21)
    mask[:] = [0, 1, 0, 0, 1]
    dx, dwg, dwu, dwd = oracle.backward(x, mask, wg, wu, wd, dout)
    eps = 1e-6
    args = [x, wg, wu, wd]
    grads = [dx, dwg, dwu, dwd]
    for k, (a, g) in enumerate(zip(args, grads)):
        num = np.zeros_like(a)
        for j in np.ndindex(a.shape):
            ap, am = a.copy(), a.copy()
            ap[j] += eps
            am[j] -= eps
            cur_p = list(args); cur_p[k] = ap
            cur_m = list(args); cur_m[k] = am
            num[j] = (_loss(cur_p[0], mask, *cur_p[1:], dout) - _loss(cur_m[0], mask, *cur_m[1:], dout)) / (2 * eps)
        np.testing.assert_allclose(g, num, rtol=2e-7, atol=2e-8)


def test_backward_matches_fp64_autograd():
    import torch
    x, mask, wg, wu, wd, dout = _rand_case(17, 12, 20, seed=31)
    tx, twg, twu, twd = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (x, wg, wu, wd))
    keep = torch.tensor((mask == 0).astype(np.float64))[:, None]
    out = tx + keep * ((torch.nn.functional.silu(tx @ twg.T) * (tx @ twu.T)) @ twd.T)
    (out * torch.tensor(dout)).sum().backward()
    dx, dwg, dwu, dwd = oracle.backward(x, mask, wg, wu, wd, dout)
    for got, want in [(dx, tx.grad), (dwg, twg.grad), (dwu, twu.grad), (dwd, twd.grad)]:
        np.testing.assert_allclose(got, want.numpy(), rtol=1e-11, atol=1e-12)


def test_silu_derivative_via_scalar_case():
    # C = I = 1, wu = wd = 1, x = 1: out = 1 + silu(wg) ; d out / d wg = silu'(wg)
    for z in (-3.0, -0.5, 0.0, 0.7, 4.0):
        _, dwg, _, _ = oracle.backward([[1.0]], [0], [[z]], [[1.0]], [[1.0]], [[1.0]])
        s = 1 / (1 + math.exp(-z))
        assert abs(dwg[0, 0] - (s + z * s * (1 - s))) < 1e-15
        h = 1e-5
        silu = lambda t: t / (1 + math.exp(-t))
        assert abs(dwg[0, 0] - (silu(z + h) - silu(z - h)) / (2 * h)) < 1e-9


def test_backward_linearity_in_dout_and_skipped_rows():
    x, mask, wg, wu, wd, d1 = _rand_case(10, 6, 8, seed=41)
    d2 = np.random.default_rng(5).normal(size=d1.shape)
    a = oracle.backward(x, mask, wg, wu, wd, d1)
    b = oracle.backward(x, mask, wg, wu, wd, d2)
    c = oracle.backward(x, mask, wg, wu, wd, 2 * d1 - 3 * d2)
    for u, v, w in zip(a, b, c):
        np.testing.assert_allclose(w, 2 * u - 3 * v, rtol=1e-11, atol=1e-12)
    sk = mask != 0
    assert a[0][sk].tobytes() == d1[sk].tobytes()
    # weight gradients ignore dout on skipped rows entirely
    d3 = d1.copy()
    d3[sk] = 123.0
    e = oracle.backward(x, mask, wg, wu, wd, d3)
    for u, v in zip(a[1:], e[1:]):
        assert np.array_equal(u, v)


def test_dw_equals_dense_backward_with_masked_ffn_branch():
    x, mask, wg, wu, wd, dout = _rand_case(14, 6, 10, seed=51)
    keep = (mask == 0)
    # dense backward over only the kept rows == skip backward weight grads
    a = oracle.backward(x, mask, wg, wu, wd, dout)
    b = oracle.backward(x[keep], np.zeros(keep.sum(), np.uint8), wg, wu, wd, dout[keep])
    for u, v in zip(a[1:], b[1:]):
        np.testing.assert_allclose(u, v, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(a[0][keep], b[0], rtol=0, atol=0)


# ------------------------------------------------------------------ sampled mode
def test_sampled_modes_match_full():
    w = wl.small_case(3, "bf16", 64, 96, 2, 8, 48, 0.75)
    out = oracle.forward(w.x, w.skip_mask, w.W_gate, w.W_up, w.W_down)
    dx, dwg, dwu, dwd = oracle.backward(w.x, w.skip_mask, w.W_gate, w.W_up, w.W_down, w.dout)
    tok = [0, 5, 17, 33, w.N - 1, 20, 21]
    o_r, dx_r = oracle.rows(w.x, w.skip_mask, w.W_gate, w.W_up, w.W_down, w.dout, tok)
    assert np.array_equal(o_r, out[tok]) and np.array_equal(dx_r, dx[tok])
    cols = [0, 1, 50, 95]
    a, b, c = oracle.dw_columns(w.x, w.skip_mask, w.W_gate, w.W_up, w.W_down, w.dout, cols)
    np.testing.assert_allclose(a, dwg[cols], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(b, dwu[cols], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(c, dwd[:, cols].T, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------ whole-matrix statement
def _dense():
    from oracle import dense
    return dense


@pytest.mark.parametrize("p_skip", [0.0, 0.5, 1.0])
def test_dense_statement_equals_the_per_token_loops(p_skip):
    # two statements of the same definition, written independently (C loops over tokens; numpy
    # matmuls over the retained rows): they must agree to rounding on every result
    x, mask, wg, wu, wd, dout = _rand_case(23, 10, 14, p_skip=p_skip, seed=61)
    d = _dense().forward_backward(x, mask, wg, wu, wd, dout)
    out = oracle.forward(x, mask, wg, wu, wd)
    dx, dwg, dwu, dwd = oracle.backward(x, mask, wg, wu, wd, dout)
    for got, want in ((d["out"], out), (d["dx"], dx), (d["dW_gate"], dwg), (d["dW_up"], dwu), (d["dW_down"], dwd)):
        np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-12)
    sk = mask != 0
    assert d["out"][sk].tobytes() == x[sk].tobytes() and d["dx"][sk].tobytes() == dout[sk].tobytes()
    if p_skip == 1.0:
        assert not d["dW_gate"].any() and not d["dW_up"].any() and not d["dW_down"].any()


def test_dense_statement_scalar_closed_form_and_finite_differences():
    # C = I = 1: out = x + silu(x wg) (x wu) wd
    r = _dense().forward_backward([[0.5]], [0], [[2.0]], [[-3.0]], [[0.25]])
    z = 0.5 * 2.0
    assert abs(r["out"][0, 0] - (0.5 + z / (1 + math.exp(-z)) * (0.5 * -3.0) * 0.25)) < 1e-15
    # central differences of its own forward for the loss sum(dout * out)
    x, mask, wg, wu, wd, dout = _rand_case(6, 4, 5, seed=71)
    mask[0], mask[1] = 0, 1
    d = _dense().forward_backward(x, mask, wg, wu, wd, dout)
    loss = lambda *a: float(np.sum(dout * _dense().forward_backward(a[0], mask, a[1], a[2], a[3])["out"]))
    args = [x, wg, wu, wd]
    for k, name in enumerate(("dx", "dW_gate", "dW_up", "dW_down")):
        num = np.zeros_like(args[k])
        for pos in np.ndindex(*args[k].shape):
            hi = [a.copy() for a in args]
            lo = [a.copy() for a in args]
            hi[k][pos] += 1e-6
            lo[k][pos] -= 1e-6
            num[pos] = (loss(*hi) - loss(*lo)) / 2e-6
        np.testing.assert_allclose(d[name], num, rtol=1e-6, atol=1e-7)


def test_dense_statement_prenorm_equals_the_per_token_loops():
    x, mask, wg, wu, wd, dout = _rand_case(17, 12, 9, seed=81)
    gamma = 1.0 + 0.2 * np.random.default_rng(3).normal(size=12)
    d = _dense().forward_backward(x, mask, wg, wu, wd, dout, gamma=gamma, eps=1e-3)
    out = oracle.forward_prenorm(x, mask, gamma, 1e-3, wg, wu, wd)
    dx, dg, dwg, dwu, dwd = oracle.backward_prenorm(x, mask, gamma, 1e-3, wg, wu, wd, dout)
    for got, want in ((d["out"], out), (d["dx"], dx), (d["dgamma"], dg), (d["dW_gate"], dwg), (d["dW_up"], dwu),
                      (d["dW_down"], dwd)):
        np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-12)
    # a 3-4-0-0 row has mean square 6.25: with eps = 0 its normalised row is (1.2, 1.6, 0, 0)
    one = _dense().forward_backward([[3.0, 4.0, 0.0, 0.0]], [0], np.eye(4), np.eye(4), np.eye(4), gamma=np.ones(4))
    silu = lambda t: t / (1 + math.exp(-t))
    np.testing.assert_allclose(one["out"][0], [3 + silu(1.2) * 1.2, 4 + silu(1.6) * 1.6, 0, 0], rtol=1e-14)


# ------------------------------------------------------------------ paper closed forms
def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "llama3_8b_ffn_shape.txt")
    vals = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            vals[k.strip()] = float(v)
    return vals


def test_paper_table1_fixes_swiglu_shape():
    g = _golden()
    C, I, L = wl.SWEEP_SHAPES["llama3-8b"] + (32,)
    assert round(L * 3 * C * I / 1e9, 2) == g["ffn_params_billion"]          # three C x I matrices
    assert 3 * I / C == g["ffn_complexity_coeff"]                              # 3 * (M / C) = 10.5
    assert round(L * (2 * C * C + 2 * C * 1024) / 1e9, 2) == g["attention_params_billion"]
    w = wl.config2(C=8, I=8)
    per_seq = w.N // w.B
    assert per_seq == g["visual_tokens"] + g["text_tokens"]
    # the oracle's weight shapes are exactly those three matrices
    x, mask, wg, wu, wd, _ = _rand_case(2, 4, 14)
    assert wg.size + wu.size + wd.size == g["ffn_macs_per_token_coeff"] * 4 * 14
    oracle.forward(x, mask, wg, wu, wd)


# ------------------------------------------------------------------ skip KV-cache (Eq. 7)
def test_kv_compact_is_the_set_difference_in_order():
    r = np.random.default_rng(7)
    planes, N, heads, d = 3, 41, 2, 4
    mask = (r.random(N) < 0.6).astype(np.uint8) * r.integers(1, 200, size=N).astype(np.uint8)
    # tag every row with (plane, token) so that rows are distinguishable set elements
    cache = np.zeros((planes, N, heads, d), dtype=np.float32)
    cache[..., 0, 0] = np.arange(planes)[:, None]
    cache[..., 0, 1] = np.arange(N)[None, :]
    cache[..., 1, :] = r.normal(size=(planes, N, d))
    out = oracle.kv_compact(cache, mask)
    # library routine: boolean indexing
    assert np.array_equal(out, cache[:, mask == 0])
    # Eq. 7 as a set difference: the tokens present afterwards are exactly those not skipped
    for p in range(planes):
        present = [int(t) for t in out[p, :, 0, 1]]
        assert set(present) == set(range(N)) - set(np.flatnonzero(mask).tolist())
        assert present == sorted(present)                       # original order
        assert np.all(out[p, :, 0, 0] == p)                     # no mixing across planes
    # NaN payloads and negative zero survive a byte copy
    cache[0, int(np.flatnonzero(mask == 0)[0]), 1, 0] = np.nan
    cache[0, int(np.flatnonzero(mask == 0)[0]), 1, 1] = -0.0
    out = oracle.kv_compact(cache, mask)
    assert out.tobytes() == cache[:, mask == 0].tobytes()


def test_kv_compact_hand_cases_and_offsets():
    cache = np.arange(2 * 5 * 2, dtype=np.int16).reshape(2, 5, 2)
    out = oracle.kv_compact(cache, [0, 1, 1, 0, 0])
    assert out.tolist() == [[[0, 1], [6, 7], [8, 9]], [[10, 11], [16, 17], [18, 19]]]
    assert oracle.kv_compact(cache, [1] * 5).shape == (2, 0, 2)
    assert np.array_equal(oracle.kv_compact(cache, [0] * 5), cache)
    # offsets: sequences [0,2) [2,5): one kept in the first, two in the second
    assert oracle.kept_cu_seqlens([0, 1, 1, 0, 0], [0, 2, 5]).tolist() == [0, 1, 3]
    w = wl.config4(seed=1, C=8, I=8, n_seq=5)
    got = oracle.kept_cu_seqlens(w.skip_mask, w.cu_seqlens)
    want = [int((w.skip_mask[:c] == 0).sum()) for c in w.cu_seqlens]
    assert got.tolist() == want and got[-1] == w.n_kept


# ------------------------------------------------------------------ pre-norm variant
def test_prenorm_unit_rms_rows_reduce_to_plain_skipffn():
    x, mask, wg, wu, wd, dout = _rand_case(11, 8, 12, seed=61)
    x /= np.sqrt(np.mean(x * x, axis=1, keepdims=True))          # every row has RMS exactly 1
    ones = np.ones(8)
    a = oracle.forward_prenorm(x, mask, ones, 0.0, wg, wu, wd)
    b = oracle.forward(x, mask, wg, wu, wd)
    np.testing.assert_allclose(a, b, rtol=1e-13, atol=1e-13)
    # weight gradients see the same FFN input, so they agree too (dx does not: the norm has a Jacobian)
    ga = oracle.backward_prenorm(x, mask, ones, 0.0, wg, wu, wd, dout)
    gb = oracle.backward(x, mask, wg, wu, wd, dout)
    for u, v in zip(ga[2:], gb[1:]):
        np.testing.assert_allclose(u, v, rtol=1e-12, atol=1e-13)
    sk = mask != 0
    assert ga[0][sk].tobytes() == dout[sk].tobytes() and a[sk].tobytes() == x[sk].tobytes()


def test_prenorm_closed_forms_and_scale_invariance():
    # a constant row c: rstd = 1/|c| for eps = 0, so xn = sign(c) * gamma
    C, I = 4, 3
    r = np.random.default_rng(3)
    wg, wu, wd = r.normal(size=(I, C)), r.normal(size=(I, C)), r.normal(size=(C, I))
    gamma = r.normal(size=C)
    x = np.full((1, C), -2.5)
    out = oracle.forward_prenorm(x, [0], gamma, 0.0, wg, wu, wd)
    want = x + oracle.forward(-gamma[None, :], [0], wg, wu, wd, ffn_only=True)
    np.testing.assert_allclose(out, want, rtol=1e-13)
    # eps: x = (3, 4, 0, 0), eps = 0.75 -> mean square 6.25, rstd = 1/sqrt(7) exactly as written
    x = np.array([[3.0, 4.0, 0.0, 0.0]])
    out = oracle.forward_prenorm(x, [0], gamma, 0.75, wg, wu, wd)
    xn = x / math.sqrt(7.0) * gamma
    np.testing.assert_allclose(out, x + oracle.forward(xn, [0], wg, wu, wd, ffn_only=True), rtol=1e-13)
    # eps = 0: the FFN branch does not depend on the scale of x
    x = r.normal(size=(5, C))
    m = np.zeros(5, np.uint8)
    a = oracle.forward_prenorm(x, m, gamma, 0.0, wg, wu, wd) - x
    b = oracle.forward_prenorm(7.0 * x, m, gamma, 0.0, wg, wu, wd) - 7.0 * x
    np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)


def test_prenorm_backward_matches_fp64_autograd_and_finite_differences():
    import torch
    x, mask, wg, wu, wd, dout = _rand_case(9, 6, 10, seed=71)
    gamma = np.random.default_rng(2).normal(size=6) + 1.0
    eps = 1e-2
    tx, tg, twg, twu, twd = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (x, gamma, wg, wu, wd))
    keep = torch.tensor((mask == 0).astype(np.float64))[:, None]
    xn = tx * torch.rsqrt((tx * tx).mean(dim=1, keepdim=True) + eps) * tg
    out = tx + keep * ((torch.nn.functional.silu(xn @ twg.T) * (xn @ twu.T)) @ twd.T)
    np.testing.assert_allclose(oracle.forward_prenorm(x, mask, gamma, eps, wg, wu, wd), out.detach().numpy(),
                               rtol=1e-12, atol=1e-13)
    (out * torch.tensor(dout)).sum().backward()
    got = oracle.backward_prenorm(x, mask, gamma, eps, wg, wu, wd, dout)
    for g, w in zip(got, (tx.grad, tg.grad, twg.grad, twu.grad, twd.grad)):
        np.testing.assert_allclose(g, w.numpy(), rtol=1e-10, atol=1e-12)
    # central differences on gamma and on one row of x
    h = 1e-6
    loss = lambda xx, gg: float(np.sum(dout * oracle.forward_prenorm(xx, mask, gg, eps, wg, wu, wd)))
    for c in range(6):
        gp, gm = gamma.copy(), gamma.copy()
        gp[c] += h; gm[c] -= h
        assert abs((loss(x, gp) - loss(x, gm)) / (2 * h) - got[1][c]) < 1e-6
    t = int(np.flatnonzero(mask == 0)[0])
    for c in range(6):
        xp, xm = x.copy(), x.copy()
        xp[t, c] += h; xm[t, c] -= h
        assert abs((loss(xp, gamma) - loss(xm, gamma)) / (2 * h) - got[0][t, c]) < 1e-6


# ------------------------------------------------------------------ adaptive summary token (Eq. 6)
def test_summary_token_special_cases():
    r = np.random.default_rng(5)
    X = r.normal(size=(9, 6))
    off = [0, 4, 4, 5, 9]                     # sizes 4, 0, 1, 4
    # w = 0: uniform weights, the summary token is the mean of the rows
    xs, p = oracle.summary_forward(X, off, np.zeros(6))
    np.testing.assert_allclose(xs[0], X[0:4].mean(0), rtol=1e-14)
    assert not xs[1].any()                    # empty segment
    assert xs[2].tolist() == X[4].tolist()    # one row: itself
    np.testing.assert_allclose(p, [0.25] * 4 + [1.0] + [0.25] * 4)
    # library softmax
    from scipy.special import softmax
    w = r.normal(size=6)
    xs, p = oracle.summary_forward(X, off, w)
    for lo, hi, s in [(0, 4, 0), (5, 9, 3)]:
        q = softmax(X[lo:hi] @ w)
        np.testing.assert_allclose(p[lo:hi], q, rtol=1e-13)
        np.testing.assert_allclose(xs[s], q @ X[lo:hi], rtol=1e-13)
    # a huge score gap selects one row (and the shifted exponent does not overflow)
    X2 = np.eye(4, 6)
    xs, p = oracle.summary_forward(X2, [0, 4], np.array([0.0, 0.0, 2000.0, 0.0, 0.0, 0.0]))
    assert p.tolist() == [0.0, 0.0, 1.0, 0.0] and xs[0].tolist() == X2[2].tolist()
    # two-row closed form: weights sigmoid(+-d) with d the score difference
    X3 = np.array([[1.0, 0.0], [0.0, 1.0]])
    xs, p = oracle.summary_forward(X3, [0, 2], np.array([math.log(3.0), 0.0]))
    np.testing.assert_allclose(p, [0.75, 0.25], rtol=1e-15)
    np.testing.assert_allclose(xs[0], [0.75, 0.25], rtol=1e-15)


def test_summary_token_backward_autograd_and_finite_differences():
    import torch
    r = np.random.default_rng(6)
    X, w = r.normal(size=(7, 5)), r.normal(size=5)
    off = [0, 3, 7]
    dxs = r.normal(size=(2, 5))
    tX = torch.tensor(X, requires_grad=True)
    tw = torch.tensor(w, requires_grad=True)
    ys = [torch.softmax(tX[lo:hi] @ tw, 0) @ tX[lo:hi] for lo, hi in [(0, 3), (3, 7)]]
    (torch.stack(ys) * torch.tensor(dxs)).sum().backward()
    dX, dw = oracle.summary_backward(X, off, w, dxs)
    np.testing.assert_allclose(dX, tX.grad.numpy(), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dw, tw.grad.numpy(), rtol=1e-11, atol=1e-13)
    loss = lambda XX, ww: float(np.sum(dxs * oracle.summary_forward(XX, off, ww)[0]))
    h = 1e-6
    for c in range(5):
        wp, wm = w.copy(), w.copy()
        wp[c] += h; wm[c] -= h
        assert abs((loss(X, wp) - loss(X, wm)) / (2 * h) - dw[c]) < 1e-7
    Xp, Xm = X.copy(), X.copy()
    Xp[4, 2] += h; Xm[4, 2] -= h
    assert abs((loss(Xp, w) - loss(Xm, w)) / (2 * h) - dX[4, 2]) < 1e-7


# ------------------------------------------------------------------ token merge (section 4.1)
def test_token_merge_bruteforce_and_hand_case():
    r = np.random.default_rng(8)
    X = r.normal(size=(13, 6))
    k = 4
    avg, kept, assign, merged = oracle.token_merge(X, k)
    Xh = X / np.linalg.norm(X, axis=1, keepdims=True)
    S = Xh @ Xh.T                                            # library routine
    np.testing.assert_allclose(avg, S.mean(1), rtol=1e-12)
    want_kept = sorted(np.argsort(S.mean(1), kind="stable")[:k].tolist())
    assert kept.tolist() == want_kept
    for i in range(13):
        if i in want_kept:
            assert kept[assign[i]] == i
        else:
            assert assign[i] == int(np.argmax(S[i, want_kept]))
    for j in range(k):
        members = [i for i in range(13) if assign[i] == j]
        np.testing.assert_allclose(merged[j], X[members].mean(0), rtol=1e-12)
    np.testing.assert_allclose(oracle.merge_given(X, k, assign), merged, rtol=1e-13)
    # hand case in the plane: e1, e1 (duplicate), e2, -e1.  S rows sum to (1, 1, 1, -1): the
    # most distinctive token is -e1 (average -1/4); next, by index, token 0.
    X = np.array([[1.0, 0.0], [2.0, 0.0], [0.0, 3.0], [-1.0, 0.0]])
    avg, kept, assign, merged = oracle.token_merge(X, 2)
    assert avg.tolist() == [0.25, 0.25, 0.25, -0.25]
    assert kept.tolist() == [0, 3]
    assert assign.tolist() == [0, 0, 0, 1]                   # e2 is orthogonal to both: tie -> first
    assert merged.tolist() == [[1.0, 1.0], [-1.0, 0.0]]
    # k = n keeps everything unchanged
    avg, kept, assign, merged = oracle.token_merge(X, 4)
    assert kept.tolist() == [0, 1, 2, 3] and assign.tolist() == [0, 1, 2, 3] and np.array_equal(merged, X)
    # average similarity without the full matrix: dot with the mean unit vector (used as a closed form)
    Y = r.normal(size=(40, 9))
    Yh = Y / np.linalg.norm(Y, axis=1, keepdims=True)
    np.testing.assert_allclose(oracle.token_merge(Y, 5)[0], Yh @ Yh.mean(0), rtol=1e-12)
