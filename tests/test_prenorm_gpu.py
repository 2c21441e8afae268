"""Pre-norm variant on the GPU (skipffn_forward_prenorm / skipffn_backward_prenorm through the C
ABI) against the fp64 oracle: identity rows bit-exact, floating point within the stated tolerances."""
import numpy as np
import pytest

import oracle
import workloads as wl
from gpu_util import DeviceWorkload, bits, to_dev, to_host
from parity import check

pytestmark = pytest.mark.gpu
EPS = 1e-5


def _gamma(w, seed=0):
    g = 1.0 + 0.1 * wl.normal(seed, 9, w.C)
    return wl.round_to(g, w.dtype)


def _run(w, gamma, path=0, inplace=False, grad_fp32=False, accumulate=False, init=None):
    import paper_2503_21817_b200 as sk
    dev = DeviceWorkload(w)
    dt = sk.BF16 if w.dtype == "bf16" else sk.FP32
    ctx = sk.SkipFFN(w.C, w.I, max(w.N, 1), dtype=dt, path=path, prenorm=True, grad_fp32=grad_fp32,
                     accumulate_dw=accumulate)
    g = to_dev(gamma, w.dtype)
    x, dout = dev.x.clone(), dev.dout.clone()
    out = ctx.forward(x, dev.mask, dev.W_gate, dev.W_up, dev.W_down, out=x if inplace else None, gamma=g, eps=EPS)
    kw = {}
    if init is not None:
        kw = dict(dW_gate=init[0], dW_up=init[1], dW_down=init[2], dgamma=init[3])
    dx, dwg, dwu, dwd, dg = ctx.backward(dout, dx=dout if inplace else None, **kw)
    ctx.poll()
    return dict(out=out, dx=dx, dW_gate=dwg, dW_up=dwu, dW_down=dwd, dgamma=dg, ctx=ctx, dev=dev)


def _ref(w, gamma):
    out = oracle.forward_prenorm(w.x, w.skip_mask, gamma, EPS, w.W_gate, w.W_up, w.W_down)
    dx, dg, dwg, dwu, dwd = oracle.backward_prenorm(w.x, w.skip_mask, gamma, EPS, w.W_gate, w.W_up, w.W_down, w.dout)
    return dict(out=out, dx=dx, dgamma=dg, dW_gate=dwg, dW_up=dwu, dW_down=dwd)


def _compare(w, r, ref):
    N, C = w.N, w.C
    kept = w.skip_mask == 0
    out, dx = r["out"].reshape(N, C), r["dx"].reshape(N, C)
    assert np.array_equal(bits(out)[~kept], bits(r["dev"].x.reshape(N, C))[~kept])
    assert np.array_equal(bits(dx)[~kept], bits(r["dev"].dout.reshape(N, C))[~kept])
    check(to_host(out), ref["out"], w.dtype, "out")
    check(to_host(dx), ref["dx"], w.dtype, "dx")
    if kept.any():
        for k in ("dW_gate", "dW_up", "dW_down"):
            check(to_host(r[k]), ref[k], w.dtype, k)
        check(to_host(r["dgamma"])[None, :], ref["dgamma"][None, :], w.dtype, "dgamma")
        # the FFN branch alone
        x64 = w.x.astype(np.float64)
        eps_out = 2.0 ** -9 if w.dtype == "bf16" else 2.0 ** -24
        tol = (5e-3 if w.dtype == "bf16" else 1e-5) * np.linalg.norm((ref["out"] - x64)[kept]) + \
            eps_out * np.linalg.norm(ref["out"][kept])
        assert np.linalg.norm((to_host(out) - ref["out"])[kept]) <= tol
    else:
        for k in ("dW_gate", "dW_up", "dW_down", "dgamma"):
            assert not to_host(r[k]).any()


@pytest.mark.parametrize("dtype,path", [("bf16", 0), ("fp32", 0), ("bf16", 1)])
def test_prenorm_tiny_and_ragged(dtype, path):
    for w in (wl.config1(dtype=dtype), wl.small_case(31, dtype, 576, 1000, 3, 20, 200, 0.6)):
        g = _gamma(w)
        _compare(w, _run(w, g, path=path), _ref(w, g))


def test_prenorm_medium_full_oracle():
    # several 256-row tiles, K-split on the down / dX launches, Nk = 620
    w = wl.small_case(33, "bf16", 1024, 2048, 4, 24, 524, 0.75)
    assert w.n_kept == 4 * (24 + 131)
    g = _gamma(w, 1)
    _compare(w, _run(w, g), _ref(w, g))


def test_prenorm_degenerate_masks_inplace_and_rescaled_rows():
    w0 = wl.uniform_batch(35, "bf16", 128, 256, 1, 0, 200, 0, n_skip=200)      # nothing kept
    g = _gamma(w0)
    r = _run(w0, g)
    _compare(w0, r, _ref(w0, g))
    assert np.array_equal(bits(r["out"]), bits(r["dev"].x))
    w = wl.small_case(37, "bf16", 256, 512, 2, 16, 120, 0.7)
    g = _gamma(w)
    a, b = _run(w, g), _run(w, g, inplace=True)
    for k in ("out", "dx", "dW_gate", "dW_up", "dW_down", "dgamma"):
        assert np.array_equal(bits(a[k]), bits(b[k])), k
    # rows scaled by a power of two: the normalised rows that feed the FFN must not change
    # (eps is negligible here; rstd absorbs the scale up to fp32 rounding, i.e. at most one bf16 ulp)
    ws = wl.small_case(37, "bf16", 256, 512, 2, 16, 120, 0.7)
    ws.x[:] = ws.x * 4.0
    c = _run(ws, g)
    nk = w.n_kept
    xa, xc = to_host(a["ctx"].intermediate(7, nk)), to_host(c["ctx"].intermediate(7, nk))
    assert np.max(np.abs(xa - xc)) <= 2.0 ** -7 * np.max(np.abs(xa))
    assert np.mean(xa != xc) < 0.02
    # and they are RMSNorm(x) * gamma: unit RMS per row up to gamma's spread and bf16 rounding
    want = w.x[w.skip_mask == 0].astype(np.float64)
    want = want / np.sqrt(np.mean(want * want, axis=1, keepdims=True) + EPS) * g.astype(np.float64)
    assert np.max(np.abs(xa - want)) <= 2.0 ** -8 * np.max(np.abs(want))


def test_prenorm_fp32_grads_accumulate_and_entry_point_checks():
    import torch
    import paper_2503_21817_b200 as sk
    w = wl.small_case(39, "bf16", 256, 512, 2, 16, 120, 0.7)
    g = _gamma(w)
    ref = _ref(w, g)
    r = _run(w, g, grad_fp32=True)
    assert r["dgamma"].dtype == torch.float32
    _compare(w, r, ref)
    init = [torch.full((w.I, w.C), 0.5, device="cuda"), torch.full((w.I, w.C), -0.25, device="cuda"),
            torch.full((w.C, w.I), 1.0, device="cuda"), torch.full((w.C,), 2.0, device="cuda")]
    r2 = _run(w, g, grad_fp32=True, accumulate=True, init=[t.clone() for t in init])
    for k, t in zip(("dW_gate", "dW_up", "dW_down", "dgamma"), init):
        assert torch.equal(r2[k], r[k] + t), k
    # the plain entry points reject a pre-norm handle and vice versa
    dev = DeviceWorkload(w)
    plain = sk.SkipFFN(w.C, w.I, w.N)
    with pytest.raises(ValueError):
        plain.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down, gamma=to_dev(g, "bf16"))
    lib = sk.load_library()
    import ctypes
    pn = sk.SkipFFN(w.C, w.I, w.N, prenorm=True)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    out = torch.empty_like(dev.x)
    assert lib.skipffn_forward(pn._saved, p(dev.x), p(dev.mask), 1, w.N, None, 0, p(dev.W_gate), p(dev.W_up),
                               p(dev.W_down), p(out), None) == 1
    assert lib.skipffn_forward_prenorm(plain._saved, p(dev.x), p(dev.mask), 1, w.N, None, 0, p(dev.W_gate),
                                       ctypes.c_float(1e-5), p(dev.W_gate), p(dev.W_up), p(dev.W_down), p(out),
                                       None) == 1


def test_prenorm_config2_full_size():
    # benchmark configuration (8B shape).  The per-token loops evaluate stratified sampled rows of
    # out / dx; the whole-matrix float64 statement gives every element of out, dx, the three weight
    # gradients and dgamma.
    from oracle import dense as oracle_dense
    from gpu_util import stratified_tokens
    w = wl.config2()
    g = _gamma(w, 2)
    r = _run(w, g)
    N, C = w.N, w.C
    kept = w.skip_mask == 0
    assert np.array_equal(bits(r["out"].reshape(N, C))[~kept], bits(r["dev"].x.reshape(N, C))[~kept])
    assert np.array_equal(bits(r["dx"].reshape(N, C))[~kept], bits(r["dev"].dout.reshape(N, C))[~kept])
    tok = stratified_tokens(w.skip_mask, np.random.default_rng(1))
    x64, do64, m = w.x[tok].astype(np.float64), w.dout[tok].astype(np.float64), w.skip_mask[tok]
    ref_out = oracle.forward_prenorm(x64, m, g, EPS, w.W_gate, w.W_up, w.W_down)
    ref_dx = oracle.backward_prenorm(x64, m, g, EPS, w.W_gate, w.W_up, w.W_down, do64, need_dw=False)[0]
    check(to_host(r["out"].reshape(N, C)[tok]), ref_out, "bf16", "out rows")
    check(to_host(r["dx"].reshape(N, C)[tok]), ref_dx, "bf16", "dx rows")
    ref = oracle_dense.forward_backward(w.x, w.skip_mask, w.W_gate, w.W_up, w.W_down, w.dout, gamma=g, eps=EPS)
    check(to_host(r["out"]).reshape(N, C), ref["out"], "bf16", "out (all elements)")
    check(to_host(r["dx"]).reshape(N, C), ref["dx"], "bf16", "dx (all elements)")
    for k in ("dW_gate", "dW_up", "dW_down"):
        check(to_host(r[k]), ref[k], "bf16", k + " (all elements)")
    check(to_host(r["dgamma"])[None, :], ref["dgamma"][None, :], "bf16", "dgamma")
