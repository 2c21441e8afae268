"""Helpers for the GPU parity tests: move a workload to the device, run the library, fetch results."""
import numpy as np

import workloads as wl


def to_dev(a, dtype):
    import torch
    if dtype == "bf16":
        bits = wl.to_bf16_bits(a).view(np.int16)
        return torch.from_numpy(bits).cuda().view(torch.bfloat16).reshape(a.shape)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def to_host(t):
    import torch
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def bits(t):
    """Raw bytes of a tensor as a numpy array (for bit-exact comparisons)."""
    import torch
    return t.detach().contiguous().view(torch.uint8).cpu().numpy()


class DeviceWorkload:
    def __init__(self, w):
        import torch
        self.w = w
        d = w.dtype
        self.x = to_dev(w.x, d)
        self.dout = to_dev(w.dout, d)
        self.W_gate = to_dev(w.W_gate, d)
        self.W_up = to_dev(w.W_up, d)
        self.W_down = to_dev(w.W_down, d)
        self.mask = torch.from_numpy(w.skip_mask).cuda()


def run(w, dense=False, path=0, grad_fp32=False, accumulate_dw=False, inplace=False, dev=None,
        dw_init=None, tune=None, recompute=False, max_kept=None):
    """Forward + backward through the C ABI; returns a dict of device tensors and the context."""
    import torch
    import paper_2503_21817_b200 as sk
    dev = dev or DeviceWorkload(w)
    dt = sk.BF16 if w.dtype == "bf16" else sk.FP32
    ctx = sk.SkipFFN(w.C, w.I, max(w.N, 1), dtype=dt, dense=dense, path=path, grad_fp32=grad_fp32,
                     accumulate_dw=accumulate_dw, recompute=recompute, max_kept=max_kept)
    if tune:
        ctx.tune(**tune)
    x = dev.x.clone()
    dout = dev.dout.clone()
    out = ctx.forward(x, dev.mask, dev.W_gate, dev.W_up, dev.W_down, out=x if inplace else None,
                      cu_seqlens=w.cu_seqlens)
    kw = {}
    if dw_init is not None:
        kw = dict(dW_gate=dw_init[0], dW_up=dw_init[1], dW_down=dw_init[2])
    dx, dwg, dwu, dwd = ctx.backward(dout, dx=dout if inplace else None, **kw)
    ctx.poll()
    return dict(out=out, dx=dx, dW_gate=dwg, dW_up=dwu, dW_down=dwd, ctx=ctx, dev=dev)


def stratified_tokens(mask, rng, n_skipped=3):
    """Token indices for sampled full-size checks, chosen so that the compacted row axis is covered
    tile by tile: one kept token in every 256-row tile of the kept-row list, one in every 32-row
    slab of its first and of its last tile (the rows one epilogue warp owns), the first and the last
    kept token, and a few skipped tokens."""
    kept_tok = np.flatnonzero(mask == 0)
    skip_tok = np.flatnonzero(mask != 0)
    nk = kept_tok.size
    ranks = set()
    if nk:
        ranks |= {0, nk - 1}
        for t0 in range(0, nk, 256):
            ranks.add(min(nk - 1, t0 + int(rng.integers(256))))
        for base in (0, (nk - 1) // 256 * 256):
            for s0 in range(base, min(base + 256, nk), 32):
                ranks.add(min(nk - 1, s0 + int(rng.integers(32))))
    tok = [kept_tok[r] for r in sorted(ranks)]
    if skip_tok.size:
        tok += list(rng.choice(skip_tok, min(n_skipped, skip_tok.size), replace=False))
    return np.asarray(tok, dtype=np.int64)


def stratified_cols(I, rng):
    """Intermediate indices for sampled weight-gradient checks: one in every 256-wide tile of the
    intermediate axis, walking through the eight 32-row slabs of a tile from tile to tile, plus the
    indices on both sides of the first and the last tile seam and the ends.  Index i selects row i
    of dW_gate / dW_up and column i of dW_down, so every output tile of the three weight-gradient
    problems (and both ends of each problem in the grouped launch's tile list) is touched."""
    cols = {0, 255 if I > 255 else I - 1, min(256, I - 1), I - 1, max(0, (I - 1) // 256 * 256 - 1), (I - 1) // 256 * 256}
    for t, i0 in enumerate(range(0, I, 256)):
        cols.add(min(I - 1, i0 + 32 * (t % 8) + int(rng.integers(32))))
    return np.asarray(sorted(cols), dtype=np.int64)
