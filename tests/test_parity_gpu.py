"""GPU parity tests: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the
same seeded inputs.  Index lists and identity rows bit-exact; floating point within the stated
tolerances (tests/parity.py)."""
import ctypes

import numpy as np
import pytest

import oracle
import workloads as wl
from gpu_util import DeviceWorkload, bits, run, stratified_cols, stratified_tokens, to_dev, to_host
from parity import check, few_term_dw_bounds, rel_fro

pytestmark = pytest.mark.gpu


def _sk():
    import paper_2503_21817_b200 as sk
    return sk


def _oracle_all(w, mask=None):
    m = w.skip_mask if mask is None else mask
    out = oracle.forward(w.x, m, w.W_gate, w.W_up, w.W_down)
    dx, dwg, dwu, dwd = oracle.backward(w.x, m, w.W_gate, w.W_up, w.W_down, w.dout)
    return dict(out=out, dx=dx, dW_gate=dwg, dW_up=dwu, dW_down=dwd)


def _compare(w, r, ref, mask=None):
    m = w.skip_mask if mask is None else mask
    N, C = w.N, w.C
    out = r["out"].reshape(N, C)
    dx = r["dx"].reshape(N, C)
    kept = m == 0
    # integer / byte work: index list and identity rows are bit-exact
    idx, nk = r["ctx"].kept()
    assert nk == int(kept.sum())
    assert np.array_equal(idx.cpu().numpy(), oracle.compact(m))
    xb, db = bits(r["dev"].x.reshape(N, C)), bits(r["dev"].dout.reshape(N, C))
    assert np.array_equal(bits(out)[~kept], xb[~kept])
    assert np.array_equal(bits(dx)[~kept], db[~kept])
    # floating point
    check(to_host(out), ref["out"], w.dtype, "out")
    check(to_host(dx), ref["dx"], w.dtype, "dx")
    # weight gradients summed over fewer than 8 kept tokens (bf16): the elementwise forward-error
    # bound of the arithmetic replaces the per-row criterion (parity.few_term_dw_bounds)
    few = None
    if w.dtype == "bf16" and 0 < int(kept.sum()) < 8:
        few = few_term_dw_bounds(w.x[kept], w.dout[kept], w.W_gate, w.W_up, w.W_down)
    for k in ("dW_gate", "dW_up", "dW_down"):
        if kept.any():
            check(to_host(r[k]), ref[k], w.dtype, k, elem_bound=None if few is None else few[k])
        else:
            assert not to_host(r[k]).any()
    # the FFN branch alone (out - x on kept rows), so that the O(1) residual cannot hide an FFN
    # error: its error budget is the tolerance on FFN(x) plus the rounding of `out` itself
    if kept.any():
        x64 = w.x.astype(np.float64)
        ffn_ref = (ref["out"] - x64)[kept]
        ffn_got = (to_host(out) - x64)[kept]
        eps_out = 2.0 ** -9 if w.dtype == "bf16" else 2.0 ** -24
        tol = (5e-3 if w.dtype == "bf16" else 1e-5) * np.linalg.norm(ffn_ref) + \
            eps_out * np.linalg.norm(ref["out"][kept])
        assert np.linalg.norm(ffn_got - ffn_ref) <= tol


# ------------------------------------------------------------------ a1: compaction
@pytest.mark.parametrize("N", [1, 15, 16, 17, 31, 32, 33, 1000, 4095, 4096, 4097, 4928, 16384, 16385, 50001, 300000])
def test_compaction_bit_exact(N):
    import torch
    sk = _sk()
    r = np.random.default_rng(N)
    m = ((r.random(N) < 0.7) * r.integers(1, 256, size=N)).astype(np.uint8)
    for mask in (m, np.zeros(N, np.uint8), np.full(N, 255, np.uint8)):
        ctx = sk.SkipFFN(64, 64, N)
        ctx.plan(torch.from_numpy(mask).cuda())
        idx, nk = ctx.kept()
        ref = oracle.compact(mask)
        assert nk == ref.size == N - np.count_nonzero(mask)
        assert np.array_equal(idx.cpu().numpy(), ref)
    dense = sk.SkipFFN(64, 64, N, dense=True)
    dense.plan(torch.from_numpy(m).cuda())
    idx, nk = dense.kept()
    assert nk == N and np.array_equal(idx.cpu().numpy(), np.arange(N))


# ------------------------------------------------------------------ configs[0]
@pytest.mark.parametrize("dtype,path", [("fp32", 0), ("bf16", 0), ("bf16", 1)])
def test_config1_tiny(dtype, path):
    w = wl.config1(dtype=dtype)
    _compare(w, run(w, path=path), _oracle_all(w))


# ------------------------------------------------------------------ several tiles + ragged tails
@pytest.mark.parametrize("dtype,path", [("bf16", 0), ("fp32", 0), ("bf16", 1)])
def test_multi_tile_ragged(dtype, path):
    # C = 576 (2.25 N-tiles of 256, 9 K-blocks), I = 1000 (ragged N and K), Nk = 300 (2.3 M-tiles)
    w = wl.small_case(1, dtype, 576, 1000, 3, 20, 200, 0.6)
    assert w.n_kept == 300
    _compare(w, run(w, path=path), _oracle_all(w))


@pytest.mark.parametrize("tile_n", [32, 48, 96, 128, 160, 192, 224, 256])
def test_every_tile_width(tile_n):
    # tiles are 256 accumulator columns wide by default; narrower widths are forced in turn (token
    # problems take any multiple of 16, the weight-gradient tiles multiples of 32)
    w = wl.small_case(21, "bf16", 576, 1000, 3, 20, 200, 0.6)
    _compare(w, run(w, tune=dict(tile_n=tile_n)), _oracle_all(w))


@pytest.mark.parametrize("nk", [1, 15, 16, 17, 63, 64, 65, 255, 256, 257, 300, 511, 513])
def test_kept_counts_around_tile_and_mma_granularity(nk):
    # the kept count decides the width of the last token tile (a multiple of 16) and the length
    # of the last K-block of the weight-gradient reductions: every boundary case of both
    base = wl.uniform_batch(45, "bf16", 192, 320, 1, 0, 600, 0, n_skip=600 - nk)
    assert base.n_kept == nk
    _compare(base, run(base), _oracle_all(base))


@pytest.mark.parametrize("min_saving", [0, 1])
@pytest.mark.parametrize("case", ["tiny", "ragged", "wide"])
def test_k_split_schedule_forced_on_and_off(min_saving, case):
    # the STREAMK knob = least K-blocks per worker that cutting the last waves along K must save:
    # 1 cuts whenever the tile count is not a multiple of the worker count (several hand-overs per
    # tile on these small shapes), 0 never cuts.  Both must match the oracle.
    if case == "tiny":
        w = wl.config1(dtype="bf16")
    elif case == "ragged":
        w = wl.small_case(23, "bf16", 576, 1000, 3, 20, 200, 0.6)
    else:   # long reductions: I = 4096 gives 64 K-blocks for the down projection, 128 for dX
        w = wl.small_case(25, "bf16", 256, 4096, 2, 16, 200, 0.5)
    _compare(w, run(w, tune=dict(streamk=min_saving)), _oracle_all(w))


@pytest.mark.parametrize("mode", [0, 2])
@pytest.mark.parametrize("case", ["ragged", "long_k", "one_token_tile", "many_panels"])
def test_down_and_dx_schedules_by_weight_panel_or_by_worker(case, mode):
    # down and dX either give every worker its own run of K-blocks (0) or let groups of workers, one
    # per token tile, walk a weight panel's K-blocks side by side (2 = always, also where the
    # library would not choose it).  The partial sums are cut at different K-blocks, so the two agree
    # with the oracle, not bit for bit with each other.
    if case == "ragged":            # 3-4 token tiles, C not a multiple of the panel height
        w = wl.small_case(31, "bf16", 576, 1000, 4, 30, 400, 0.55)
    elif case == "long_k":          # 64 / 128 K-blocks, two panels, groups share them along K
        w = wl.small_case(32, "bf16", 512, 4096, 2, 16, 300, 0.4)
    elif case == "one_token_tile":  # fewer kept tokens than one tile: groups of one
        w = wl.small_case(33, "bf16", 1024, 2048, 2, 16, 100, 0.7)
    else:                           # more panels than groups: whole panels first, the rest cut along K
        w = wl.small_case(34, "bf16", 8192, 256, 3, 16, 260, 0.3)
    _compare(w, run(w, tune=dict(panel_sync=mode)), _oracle_all(w))


@pytest.mark.parametrize("knob", ["one_box", "tma_stores", "gather"])
@pytest.mark.parametrize("grad_fp32", [False, True])
def test_alternative_load_and_store_paths_give_the_same_bits(knob, grad_fp32):
    # operand tiles fetched with one 3-D box or one 2-D box per piece; weight-gradient tiles written
    # by TMA tile stores or per-lane stores; token rows of gate/up and dH gathered from x / dout by
    # tile::gather4 loads or read from the compacted copy.  Shapes: multiples of 64 (where the one-box loads
    # apply) and ragged ones (where the tile stores clip at the matrix edges).
    for w in (wl.small_case(27, "bf16", 512, 1024, 3, 20, 300, 0.5), wl.small_case(28, "bf16", 576, 1000, 3, 20, 200, 0.6)):
        ref = _oracle_all(w)
        a = run(w, grad_fp32=grad_fp32, tune={knob: 1})
        b = run(w, grad_fp32=grad_fp32, tune={knob: 0})
        _compare(w, a, ref)
        for k in ("out", "dx", "dW_gate", "dW_up", "dW_down"):
            assert np.array_equal(bits(a[k]), bits(b[k])), k


@pytest.mark.parametrize("C,I", [(8, 8), (8, 24), (24, 40), (72, 136), (200, 328)])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_tiny_and_odd_layer_widths(C, I, dtype):
    # widths far below one tile and one K-block, multiples of 8 only: every box reaches past the
    # arrays' ends (zero fill on loads, clipping on tile stores)
    w = wl.uniform_batch(61, dtype, C, I, 2, 3, 70, 2, skip_ratio=0.6)
    _compare(w, run(w), _oracle_all(w))
    if dtype == "bf16":
        _compare(w, run(w, grad_fp32=True), _oracle_all(w))


def test_contiguous_span_layout():
    # the paper's layout: one contiguous skipped span per sequence
    w = wl.uniform_batch(2, "bf16", 256, 512, 4, 10, 150, 10, skip_ratio=0.8, contiguous_span=True)
    _compare(w, run(w), _oracle_all(w))


def test_packed_variable_length_small():
    w = wl.config4(seed=3, C=128, I=256, n_seq=3)
    _compare(w, run(w), _oracle_all(w))
    # bad offsets are rejected on the host
    sk = _sk()
    dev = DeviceWorkload(w)
    ctx = sk.SkipFFN(w.C, w.I, w.N)
    bad = w.cu_seqlens.copy()
    bad[-1] -= 1
    with pytest.raises(sk.SkipFFNError):
        ctx.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down, cu_seqlens=bad)


# ------------------------------------------------------------------ degenerate kept counts
@pytest.mark.parametrize("nk", [0, 1, 2, 7, 8, 127, 128, 129, 257])
def test_kept_count_edges(nk):
    base = wl.uniform_batch(5, "bf16", 128, 256, 1, 0, 300, 0, n_skip=300 - nk)
    assert base.n_kept == nk
    r = run(base)
    _compare(base, r, _oracle_all(base))
    if nk == 0:   # all skipped: out == x, dx == dout bitwise, zero weight gradients
        assert np.array_equal(bits(r["out"]), bits(r["dev"].x))
        assert np.array_equal(bits(r["dx"]), bits(r["dev"].dout))


def test_empty_batch():
    import torch
    sk = _sk()
    ctx = sk.SkipFFN(128, 256, 16)
    w = wl.uniform_batch(0, "bf16", 128, 256, 1, 0, 4, 0, n_skip=0)
    dev = DeviceWorkload(w)
    x = torch.empty(0, 128, dtype=torch.bfloat16, device="cuda")
    out = ctx.forward(x, torch.empty(0, dtype=torch.uint8, device="cuda"), dev.W_gate, dev.W_up, dev.W_down)
    dx, dwg, dwu, dwd = ctx.backward(torch.empty_like(x))
    ctx.poll()
    assert out.numel() == 0 and dx.numel() == 0
    assert not dwg.float().any() and not dwu.float().any() and not dwd.float().any()


# ------------------------------------------------------------------ all kept == dense comparator
def test_all_kept_equals_dense_and_eq8_skip_error():
    w = wl.small_case(7, "bf16", 256, 512, 2, 16, 120, 0.5)
    zeros = np.zeros_like(w.skip_mask)
    ref_dense = _oracle_all(w, zeros)
    w_all = wl.small_case(7, "bf16", 256, 512, 2, 16, 120, 0.0)
    assert np.array_equal(w_all.x, w.x) and not w_all.skip_mask.any()
    r_all = run(w_all)
    r_dense = run(w, dense=True)          # mask present but ignored
    for k in ("out", "dx", "dW_gate", "dW_up", "dW_down"):
        assert np.array_equal(bits(r_all[k]), bits(r_dense[k])), k
    _compare(w, r_dense, ref_dense, zeros)
    # Eq. 8: on a skipped row the dense output differs from the skip output by FFN(x)
    r_skip = run(w)
    sk_rows = w.skip_mask != 0
    diff = (to_host(r_dense["out"]) - to_host(r_skip["out"])).reshape(w.N, w.C)[sk_rows]
    ffn = oracle.forward(w.x, zeros, w.W_gate, w.W_up, w.W_down, ffn_only=True)[sk_rows]
    x_norm = np.linalg.norm(w.x[sk_rows])
    assert np.linalg.norm(diff - ffn) <= 5e-3 * np.linalg.norm(ffn) + 2.0 ** -9 * x_norm


# ------------------------------------------------------------------ aliasing, poisoning, options
def test_inplace_aliasing_matches_out_of_place():
    w = wl.small_case(9, "bf16", 256, 512, 2, 16, 120, 0.7)
    a = run(w)
    b = run(w, inplace=True)
    for k in ("out", "dx", "dW_gate", "dW_up", "dW_down"):
        assert np.array_equal(bits(a[k]), bits(b[k])), k


def test_poisoned_skipped_rows_do_not_leak():
    import torch
    w = wl.small_case(11, "bf16", 256, 512, 2, 16, 120, 0.7)
    clean = run(w)
    dev = DeviceWorkload(w)
    sk_rows = torch.from_numpy(w.skip_mask != 0).cuda()
    dev.x[sk_rows] = float("nan")
    dev.dout[sk_rows] = float("inf")
    dirty = run(w, dev=dev)
    kept = w.skip_mask == 0
    N, C = w.N, w.C
    assert np.array_equal(bits(clean["out"].reshape(N, C))[kept], bits(dirty["out"].reshape(N, C))[kept])
    assert np.array_equal(bits(clean["dx"].reshape(N, C))[kept], bits(dirty["dx"].reshape(N, C))[kept])
    for k in ("dW_gate", "dW_up", "dW_down"):
        assert np.array_equal(bits(clean[k]), bits(dirty[k])), k
    # the poisoned rows themselves pass through bit-exactly (NaN payloads included)
    assert np.array_equal(bits(dirty["out"].reshape(N, C))[~kept], bits(dev.x.reshape(N, C))[~kept])


@pytest.mark.parametrize("path", [0, 1])
def test_fp32_gradients_and_accumulation(path):
    import torch
    w = wl.small_case(13, "bf16", 256, 512, 2, 16, 120, 0.7)
    ref = _oracle_all(w)
    r = run(w, grad_fp32=True, path=path)
    assert r["dW_gate"].dtype == torch.float32
    _compare(w, r, ref)
    # fp32 gradients carry no output rounding: tighter than the bf16 bound
    assert rel_fro(to_host(r["dW_down"]), ref["dW_down"]) < 4e-3
    init = [torch.full((w.I, w.C), 0.5, device="cuda"), torch.full((w.I, w.C), -0.25, device="cuda"),
            torch.full((w.C, w.I), 1.0, device="cuda")]
    r2 = run(w, grad_fp32=True, accumulate_dw=True, dw_init=[t.clone() for t in init], path=path)
    for k, t in zip(("dW_gate", "dW_up", "dW_down"), init):
        assert torch.equal(r2[k], r[k] + t), k


def test_plan_once_reuse_for_next_layer():
    sk = _sk()
    w = wl.small_case(15, "bf16", 256, 512, 2, 16, 120, 0.7)
    dev = DeviceWorkload(w)
    ctx = sk.SkipFFN(w.C, w.I, w.N)
    ctx.plan(dev.mask)
    out1 = ctx.forward(dev.x, None, dev.W_gate, dev.W_up, dev.W_down)       # reuses the list
    out2 = ctx.forward(out1, None, dev.W_up, dev.W_gate, dev.W_down)        # "next layer"
    ctx.poll()
    ref1 = oracle.forward(w.x, w.skip_mask, w.W_gate, w.W_up, w.W_down)
    check(to_host(out1), ref1, "bf16", "layer 1")
    # the oracle's second layer starts from the oracle's own first-layer output (rounded to the run
    # dtype as the layer boundary does), never from anything the GPU produced
    ref2 = oracle.forward(wl.round_to(ref1, "bf16"), w.skip_mask, w.W_up, w.W_gate, w.W_down)
    check(to_host(out2), ref2, "bf16", "layer 2")
    # without a list to reuse the call is rejected
    fresh = sk.SkipFFN(w.C, w.I, w.N)
    with pytest.raises(sk.SkipFFNError):
        fresh.forward(dev.x, None, dev.W_gate, dev.W_up, dev.W_down)


@pytest.mark.parametrize("tune", [None, dict(panel_sync=2), dict(streamk=1, panel_sync=0)])
def test_run_twice_bit_identical(tune):
    # every reduction has a fixed order (no atomics): also with the worker groups of down / dX
    # forced on, and with every launch cut along K
    w = wl.small_case(17, "bf16", 576, 1000, 3, 20, 200, 0.6)
    a, b = run(w, tune=tune), run(w, tune=tune)
    for k in ("out", "dx", "dW_gate", "dW_up", "dW_down"):
        assert np.array_equal(bits(a[k]), bits(b[k])), k


@pytest.mark.parametrize("tune", [None, dict(streamk=1, panel_sync=2)])
def test_step_captured_in_a_cuda_graph_replays_the_same_bits(tune):
    # the library never synchronises, allocates or reads back inside a call, so one forward +
    # backward can be captured into a CUDA graph; every replay repeats the launches with the kernel
    # arguments of the capture (the same hand-over flag values too) and must give the eager bits
    import torch
    sk = _sk()
    w = wl.small_case(19, "bf16", 576, 2048, 3, 20, 200, 0.6)
    d = DeviceWorkload(w)
    ctx = sk.SkipFFN(w.C, w.I, w.N)
    if tune:
        ctx.tune(**tune)
    out, dx = torch.empty_like(d.x), torch.empty_like(d.x)
    dW = [torch.empty_like(t) for t in (d.W_gate, d.W_up, d.W_down)]

    def step():
        ctx.forward(d.x, d.mask, d.W_gate, d.W_up, d.W_down, out=out)
        ctx.backward(d.dout, dx=dx, dW_gate=dW[0], dW_up=dW[1], dW_down=dW[2])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):       # warm-up on the side stream: first-use work happens outside the capture
        step()
        step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    eager = [bits(t).copy() for t in (out, dx, *dW)]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for _ in range(3):
        for t in (out, dx, *dW):
            t.fill_(7.0)
        g.replay()
        torch.cuda.synchronize()
        for a, t in zip(eager, (out, dx, *dW)):
            assert np.array_equal(a, bits(t))
    ctx.poll()


def test_unsupported_and_invalid_arguments():
    import torch
    sk = _sk()
    with pytest.raises(sk.SkipFFNError):
        sk.SkipFFN(100, 256, 16)                       # C % 8 != 0
    ctx = sk.SkipFFN(128, 256, 16)
    w = wl.uniform_batch(0, "bf16", 128, 256, 1, 0, 32, 0, n_skip=8)
    dev = DeviceWorkload(w)
    with pytest.raises(sk.SkipFFNError):
        ctx.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down)   # 32 tokens > max_tokens 16
    with pytest.raises(sk.SkipFFNError):
        ctx.backward(dev.dout)                                               # no forward yet


# ------------------------------------------------------------------ full size
def _full_size(w, dense=False, rows_from_loops=True):
    """Full-size run in the benchmark's launch configuration, checked two ways.
    (1) The per-token C loops evaluate sampled output rows and sampled weight-gradient rows /
        columns one by one; the samples are stratified over the kernels' tiles (gpu_util).
    (2) The whole-matrix float64 statement of the same definition (oracle.dense) gives EVERY
        element of out, dx and the three weight gradients, compared with the stated tolerances."""
    import torch
    from oracle import dense as oracle_dense
    r = run(w, dense=dense)
    m = np.zeros_like(w.skip_mask) if dense else w.skip_mask
    N, C = w.N, w.C
    rng = np.random.default_rng(0)
    x64, wg, wu, wd, do = (a.astype(np.float64) for a in (w.x, w.W_gate, w.W_up, w.W_down, w.dout))
    # properties that hold at any size: exact index list, identity rows
    idx, nk = r["ctx"].kept()
    assert np.array_equal(idx.cpu().numpy(), oracle.compact(m))
    kept = m == 0
    assert np.array_equal(bits(r["out"].reshape(N, C))[~kept], bits(r["dev"].x.reshape(N, C))[~kept])
    assert np.array_equal(bits(r["dx"].reshape(N, C))[~kept], bits(r["dev"].dout.reshape(N, C))[~kept])
    got = {k: to_host(r[k]).reshape(N, C) if k in ("out", "dx") else to_host(r[k])
           for k in ("out", "dx", "dW_gate", "dW_up", "dW_down")}
    # (1) sampled, per-token loops
    if rows_from_loops:
        tok = stratified_tokens(m, rng)
        out_r, dx_r = oracle.rows(x64, m, wg, wu, wd, do, tok)
        check(got["out"][tok], out_r, "bf16", "out rows")
        check(got["dx"][tok], dx_r, "bf16", "dx rows")
    cols = stratified_cols(w.I, rng)
    a, b, c = oracle.dw_columns(x64, m, wg, wu, wd, do, cols)
    check(got["dW_gate"][cols], a, "bf16", "dW_gate rows")
    check(got["dW_up"][cols], b, "bf16", "dW_up rows")
    check(got["dW_down"][:, cols].T, c, "bf16", "dW_down cols")
    # (2) every element, whole-matrix statement
    ref = oracle_dense.forward_backward(x64, m, wg, wu, wd, do)
    for k in ("out", "dx", "dW_gate", "dW_up", "dW_down"):
        check(got[k], ref[k], "bf16", k + " (all elements)")
    # the FFN branch alone on kept rows (the O(1) residual must not hide an FFN error)
    ffn_ref, ffn_got = (ref["out"] - x64)[kept], (got["out"] - x64)[kept]
    assert np.linalg.norm(ffn_got - ffn_ref) <= 5e-3 * np.linalg.norm(ffn_ref) + 2.0 ** -9 * np.linalg.norm(ref["out"][kept])
    return r


def test_config2_llama3_8b_full_size():
    w = wl.config2()
    assert (w.N, w.n_kept, w.C, w.I) == (4928, 1472, 4096, 14336)
    _full_size(w)


def test_config3_highres_full_size():
    w = wl.config3()
    assert (w.N, w.n_kept) == (9376, 1312)
    _full_size(w)


def test_config4_packed_full_size():
    # 16 packed sequences, about 32 k tokens of which about 11 k are kept
    w = wl.config4()
    assert w.cu_seqlens.shape == (17,) and 25000 < w.N < 40000 and w.n_kept > 8000
    _full_size(w)


@pytest.mark.parametrize("shape,ratio", [("llama3-8b", 0.0), ("llama3-8b", 0.25), ("llama3-8b", 0.5),
                                         ("llama3-8b", 0.9), ("llama3-8b", 1.0),
                                         ("vicuna-13b", 0.0), ("vicuna-13b", 0.9), ("vicuna-13b", 1.0)])
def test_skip_ratio_sweep_points_full_size(shape, ratio):
    # the points of the skip-ratio sweep the benchmark times (ratio 0.75 at the 8B shape is
    # config 2 above): 4928, 3776, 2624, 784 and 320 kept rows of 4928 tokens
    C, I = wl.SWEEP_SHAPES[shape]
    w = wl.config2(skip_ratio=ratio, C=C, I=I)
    assert w.n_kept == {0.0: 4928, 0.25: 3776, 0.5: 2624, 0.9: 784, 1.0: 320}[ratio]
    r = _full_size(w, rows_from_loops=ratio >= 0.5)
    if ratio == 0.0:
        idx, nk = r["ctx"].kept()
        assert nk == w.N and np.array_equal(idx.cpu().numpy(), np.arange(w.N))


def test_dense_comparator_full_size():
    # the in-library dense comparator on config 2's inputs: the mask is ignored, every row takes the FFN
    _full_size(wl.config2(), dense=True, rows_from_loops=False)


def test_lost_hand_over_is_reported_and_the_context_stays_usable():
    # Failure path without a fault: on a debug handle the LOSE_HANDOVER knob makes the units that
    # finish a K-split tile wait for a hand-over that never comes.  The wait is bounded (about
    # 1 s): the kernel must return, skipffn_poll must report SKIPFFN_ETIMEOUT with the hand-over
    # site, and the same handle must then produce correct results again.
    import time
    sk = _sk()
    w = wl.small_case(25, "bf16", 256, 4096, 2, 16, 200, 0.5)
    dev = DeviceWorkload(w)
    plain = sk.SkipFFN(w.C, w.I, w.N)
    with pytest.raises(sk.SkipFFNError):
        plain.tune(lose_handover=1)                        # the hook exists on debug handles only
    ctx = sk.SkipFFN(w.C, w.I, w.N, debug=True)
    ctx.tune(streamk=1, lose_handover=1)                   # cut along K whenever tiles do not fill a wave
    t0 = time.time()
    ctx.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down)
    with pytest.raises(sk.SkipFFNError) as e:
        ctx.poll()
    assert e.value.status == 5 and "site 6" in str(e.value)
    assert time.time() - t0 < 30
    ctx.tune(lose_handover=0)
    out = ctx.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down)
    ctx.poll()                                              # status word was cleared by the failed poll
    check(to_host(out), oracle.forward(w.x, w.skip_mask, w.W_gate, w.W_up, w.W_down), "bf16", "out after recovery")


def test_debug_handle_checks_kept_list_and_guard_bands():
    # A debug handle verifies the kept-row list on the device after every compaction and keeps a
    # guard band behind every workspace slab, which skipffn_poll checks.  A normal run raises
    # nothing and gives the same bits as a plain handle; a byte changed inside a guard band (done
    # here from the host, as an overrunning kernel would) is reported as SKIPFFN_EDEBUG.
    import torch
    sk = _sk()
    w = wl.small_case(29, "bf16", 256, 512, 2, 16, 120, 0.7)
    dev = DeviceWorkload(w)
    plain = sk.SkipFFN(w.C, w.I, w.N)
    ctx = sk.SkipFFN(w.C, w.I, w.N, debug=True)
    assert ctx.saved_bytes > plain.saved_bytes
    out = ctx.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down)
    res = ctx.backward(dev.dout)
    ctx.poll()
    ref_out = plain.forward(dev.x, dev.mask, dev.W_gate, dev.W_up, dev.W_down)
    ref = plain.backward(dev.dout)
    plain.poll()
    for a, b in zip((out,) + tuple(res), (ref_out,) + tuple(ref)):
        assert np.array_equal(bits(a), bits(b))
    # find a guard band (1 KiB of the fill byte) in the saved region and damage it
    ws = ctx.workspace
    is_fill = (ws == 0xA5).to(torch.int32)
    runs = torch.nn.functional.avg_pool1d(is_fill.float()[None, None], 1024, stride=1)[0, 0]
    start = int(torch.nonzero(runs == 1.0)[0, 0])
    ws[start + 100] = 0
    with pytest.raises(sk.SkipFFNError) as e:
        ctx.poll()
    assert e.value.status == 6
    ws[start + 100] = 0xA5
    ctx.poll()                                                        # repaired: clean again


def test_single_cta_launch_shape_in_a_fresh_process():
    # The one-CTA-per-tile shape (used when SM pairs cannot be co-scheduled) is chosen once per
    # process, so it is exercised in a child process: the tiny, ragged, K-split and grouped cases.
    import os
    import subprocess
    import sys
    env = dict(os.environ, SKIPFFN_SINGLE_CTA="1")
    here = os.path.abspath(__file__)
    p = subprocess.run([sys.executable, "-m", "pytest", here, "-m", "gpu", "-x", "-q", "-k",
                        "config1_tiny or multi_tile_ragged or k_split_schedule or kept_count_edges or fp32_gradients"],
                       env=env, capture_output=True, text=True, timeout=900)
    assert p.returncode == 0, p.stdout[-3000:] + p.stderr[-2000:]
    assert " passed" in p.stdout


def test_bf16_gradient_accumulation():
    # dW += ... with bf16 gradients: the fp32 tile is added to the stored value and rounded once
    import torch
    w = wl.small_case(41, "bf16", 256, 512, 2, 16, 120, 0.7)
    ref = _oracle_all(w)
    init = [torch.full((w.I, w.C), 0.5, device="cuda", dtype=torch.bfloat16),
            torch.full((w.I, w.C), -0.25, device="cuda", dtype=torch.bfloat16),
            torch.full((w.C, w.I), 1.0, device="cuda", dtype=torch.bfloat16)]
    r = run(w, accumulate_dw=True, dw_init=[t.clone() for t in init])
    for k, t in zip(("dW_gate", "dW_up", "dW_down"), init):
        want = ref[k] + float(t[0, 0])
        got = to_host(r[k])
        # one bf16 rounding of a value near |init|: absolute error below half an ulp of the sum
        assert np.max(np.abs(got - want)) <= 2.0 ** -8 * np.max(np.abs(want)) + 3e-2 * np.sqrt(np.mean(ref[k] ** 2))
        assert abs(np.mean(got - want)) < 1e-3


def test_many_tokens_small_hidden():
    # 40 000 tokens in 10 sequences (grids far beyond one wave of CTAs), narrow layer: full oracle
    w = wl.uniform_batch(43, "bf16", 64, 128, 10, 100, 3800, 100, skip_ratio=0.9)
    assert w.N == 40000 and w.n_kept == 10 * (200 + 380)
    _compare(w, run(w), _oracle_all(w))
