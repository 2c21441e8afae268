"""Adaptive summary token (Eq. 6) on the GPU against the fp64 oracle."""
import numpy as np
import pytest

import oracle
import workloads as wl
from gpu_util import to_dev, to_host
from parity import check

pytestmark = pytest.mark.gpu


def _case(seed, sizes, C, dtype):
    n = int(sum(sizes))
    X = wl.round_to(wl.normal(seed, wl.TID_X, n * C), dtype).reshape(n, C)
    w = wl.round_to(wl.normal(seed, wl.TID_WGATE, C, 0.05), dtype)
    dxs = wl.round_to(wl.normal(seed, wl.TID_DOUT, len(sizes) * C), dtype).reshape(len(sizes), C)
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    return X, w, dxs, off


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("sizes,C", [((144, 432) * 4, 512), ((1, 0, 5, 33, 300), 264), ((7,), 8)])
def test_summary_token_forward_backward(dtype, sizes, C):
    import torch
    import paper_2503_21817_b200 as sk
    X, w, dxs, off = _case(len(sizes), sizes, C, dtype)
    dX_, dw_, dxs_d = None, None, to_dev(dxs, dtype)
    Xd, wd, offd = to_dev(X, dtype), to_dev(w, dtype), torch.from_numpy(off).cuda()
    xs, probs = sk.summary_forward(Xd, offd, wd)
    dX_, dw_ = sk.summary_backward(Xd, offd, wd, probs, dxs_d, dw_fp32=True)
    torch.cuda.synchronize()
    ref_xs, ref_p = oracle.summary_forward(X, off, w)
    ref_dX, ref_dw = oracle.summary_backward(X, off, w, dxs)
    assert np.allclose(to_host(probs), ref_p, rtol=1e-4, atol=1e-7)          # fp32 softmax weights
    nonempty = np.diff(off) > 0
    check(to_host(xs)[nonempty], ref_xs[nonempty], dtype, "xs")
    assert not to_host(xs)[~nonempty].any()
    check(to_host(dX_), ref_dX, dtype, "dX")
    check(to_host(dw_)[None, :], ref_dw[None, :], dtype, "dw")
    # run twice: bit-identical (fixed summation order)
    xs2, probs2 = sk.summary_forward(Xd, offd, wd)
    dX2, dw2 = sk.summary_backward(Xd, offd, wd, probs2, dxs_d, dw_fp32=True)
    assert torch.equal(xs, xs2) and torch.equal(dX_, dX2) and torch.equal(dw_, dw2)


def test_summary_token_zero_weight_is_the_mean_and_argument_checks():
    import ctypes
    import torch
    import paper_2503_21817_b200 as sk
    X, w, dxs, off = _case(3, (64, 17), 128, "fp32")
    Xd, offd = to_dev(X, "fp32"), torch.from_numpy(off).cuda()
    xs, probs = sk.summary_forward(Xd, offd, torch.zeros(128, device="cuda"))
    torch.cuda.synchronize()
    assert np.allclose(to_host(xs)[0], X[:64].mean(0), rtol=1e-5, atol=1e-6)
    assert np.allclose(to_host(probs)[64:], 1 / 17, rtol=1e-6)
    lib = sk.load_library()
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    assert lib.skipffn_summary_scratch_bytes(81, 128) == (128 + 32 * 128) * 4
    # scratch too small -> EWORKSPACE; null weight -> EINVAL
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    assert lib.skipffn_summary_backward(p(Xd), p(offd), 2, 81, 128, 1, p(Xd), p(probs), p(xs), None, None, 1,
                                        p(small), 16, None) == 3
    assert lib.skipffn_summary_forward(p(Xd), p(offd), 2, 81, 128, 1, None, p(xs), p(probs), None) == 1
