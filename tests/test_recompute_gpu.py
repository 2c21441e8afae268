"""Memory modes of a handle on the GPU: the recomputing backward (no G, U, H kept between forward and
backward), compacted arrays sized by a kept-token bound, and one scratch buffer shared by the
layers of a model.  Results must be the bits of the default mode and match the fp64 oracle."""
import numpy as np
import pytest

import oracle
import workloads as wl
from gpu_util import DeviceWorkload, bits, run, to_dev, to_host
from parity import check

pytestmark = pytest.mark.gpu
KEYS = ("out", "dx", "dW_gate", "dW_up", "dW_down")


def _sk():
    import paper_2503_21817_b200 as sk
    return sk


@pytest.mark.parametrize("dtype,path", [("bf16", 0), ("fp32", 0), ("bf16", 1)])
def test_recompute_gives_the_same_bits_and_matches_the_oracle(dtype, path):
    w = wl.small_case(51, dtype, 576, 1000, 3, 20, 200, 0.6)
    a = run(w, path=path)
    b = run(w, path=path, recompute=True)
    for k in KEYS:
        assert np.array_equal(bits(a[k]), bits(b[k])), k
    assert b["ctx"].launches() == (a["ctx"].launches()[0], a["ctx"].launches()[1] + 1)   # gate/up runs again
    assert b["ctx"].saved_bytes < a["ctx"].saved_bytes
    ref_out = oracle.forward(w.x, w.skip_mask, w.W_gate, w.W_up, w.W_down)
    ref = oracle.backward(w.x, w.skip_mask, w.W_gate, w.W_up, w.W_down, w.dout)
    check(to_host(b["out"]), ref_out, dtype, "out")
    for k, r in zip(KEYS[1:], ref):
        check(to_host(b[k]), r, dtype, k)


def test_recompute_full_size_config2_same_bits():
    w = wl.config2()
    a = run(w)
    b = run(w, recompute=True, max_kept=w.n_kept, dev=a["dev"])
    for k in KEYS:
        assert np.array_equal(bits(a[k]), bits(b[k])), k
    sk = _sk()
    full = sk.SkipFFN(w.C, w.I, w.N)
    # kept-sized and recomputing: what a layer holds between forward and backward shrinks from the
    # token-sized G, U, H, Xk to the kept rows of x alone
    assert b["ctx"].saved_bytes < 0.05 * full.saved_bytes
    assert b["ctx"].saved_bytes + b["ctx"].scratch_bytes < 0.4 * (full.saved_bytes + full.scratch_bytes)


def test_kept_bound_exact_fit_and_overflow_is_reported():
    sk = _sk()
    w = wl.small_case(53, "bf16", 256, 512, 2, 16, 120, 0.7)
    ok = run(w, max_kept=w.n_kept)                       # exactly as many rows as the mask keeps
    ref = run(w)
    for k in KEYS:
        assert np.array_equal(bits(ok[k]), bits(ref[k])), k
    # a bound below the kept count: no out-of-bounds access, the problem is reported by poll
    dev = ok["dev"]
    ctx = sk.SkipFFN(w.C, w.I, w.N, max_kept=w.n_kept - 7)
    ctx.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down)
    with pytest.raises(sk.SkipFFNError) as e:
        ctx.poll()
    assert e.value.status == 3 and "site 8" in str(e.value)
    idx, nk = ctx.kept()
    assert nk == w.n_kept - 7 and np.array_equal(idx.cpu().numpy(), oracle.compact(w.skip_mask)[:nk])
    # the handle stays usable: a mask within the bound gives correct results afterwards
    few = w.skip_mask.copy()
    few[np.flatnonzero(few == 0)[-20:]] = 1
    import torch
    out = ctx.forward(dev.x, torch.from_numpy(few).cuda(), dev.W_gate, dev.W_up, dev.W_down)
    ctx.poll()
    check(to_host(out), oracle.forward(w.x, few, w.W_gate, w.W_up, w.W_down), "bf16", "out within the bound")
    with pytest.raises(sk.SkipFFNError):
        sk.SkipFFN(w.C, w.I, w.N, max_kept=w.N + 1)      # bound above max_tokens


def test_two_layers_share_one_scratch_buffer():
    # layer 1 forward, layer 2 forward, layer 2 backward, layer 1 backward, as autograd would run a
    # two-layer stack; both handles recompute and share one scratch buffer
    sk = _sk()
    w = wl.small_case(55, "bf16", 256, 512, 2, 16, 120, 0.7)
    dev = DeviceWorkload(w)
    l1 = sk.SkipFFN(w.C, w.I, w.N, recompute=True, max_kept=w.n_kept)
    l2 = sk.SkipFFN(w.C, w.I, w.N, recompute=True, max_kept=w.n_kept, scratch_from=l1)
    assert l2.scratch.data_ptr() == l1.scratch.data_ptr()
    h1 = l1.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down)
    h2 = l2.forward(h1, dev.mask, dev.W_up, dev.W_gate, dev.W_down)
    d1, g2g, g2u, g2d = l2.backward(dev.dout)
    d0, g1g, g1u, g1d = l1.backward(d1)
    l1.poll()
    # the same stack on two independent default-mode handles
    a1, a2 = sk.SkipFFN(w.C, w.I, w.N), sk.SkipFFN(w.C, w.I, w.N)
    r1 = a1.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down)
    r2 = a2.forward(r1, dev.mask, dev.W_up, dev.W_gate, dev.W_down)
    e1, f2g, f2u, f2d = a2.backward(dev.dout)
    e0, f1g, f1u, f1d = a1.backward(e1)
    a1.poll()
    for got, want in ((h2, r2), (d0, e0), (g1g, f1g), (g1u, f1u), (g1d, f1d), (g2g, f2g), (g2u, f2u), (g2d, f2d)):
        assert np.array_equal(bits(got), bits(want))
    # and against the oracle, layer by layer (layer 2 starts from the oracle's own rounded layer-1 output)
    o1 = oracle.forward(w.x, w.skip_mask, w.W_gate, w.W_up, w.W_down)
    o2 = oracle.forward(wl.round_to(o1, "bf16"), w.skip_mask, w.W_up, w.W_gate, w.W_down)
    check(to_host(h2), o2, "bf16", "two-layer output")


def test_recompute_prenorm_same_bits():
    sk = _sk()
    w = wl.small_case(57, "bf16", 256, 512, 2, 16, 120, 0.7)
    dev = DeviceWorkload(w)
    g = to_dev(wl.round_to(1.0 + 0.1 * wl.normal(0, 9, w.C), "bf16"), "bf16")
    res = []
    for rec in (False, True):
        ctx = sk.SkipFFN(w.C, w.I, w.N, prenorm=True, recompute=rec, max_kept=w.n_kept if rec else None)
        out = ctx.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down, gamma=g, eps=1e-5)
        res.append((out,) + tuple(ctx.backward(dev.dout)))
        ctx.poll()
    for a, b in zip(*res):
        assert np.array_equal(bits(a), bits(b))
