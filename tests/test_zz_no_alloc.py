"""skipffn_compact_static: the kept-row list for callers that cannot allocate device memory.

The entry point keeps the compaction kernel's scratch in a fixed array inside the library instead
of a caller-allocated workspace, so it serves code that must not (or cannot) call cudaMalloc: a
process whose framework already owns all device memory, a loop that cannot take cudaMalloc's
device-wide synchronisation, a host that forbids allocation from extensions.  Here it is called
through the C ABI twice in a row on different masks and compared bit for bit with the list the
regular handle-based entry point (skipffn_plan + skipffn_get_kept) produces.  The second mask is
shorter and keeps other tokens, so a kept count or a rank left over from the first call (both live
in the shared array) would give a wrong length or wrong entries.  Collected last on purpose."""
import ctypes

import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu


def _regular(sk, mask_dev):
    ctx = sk.SkipFFN(64, 64, max(mask_dev.numel(), 1))
    ctx.plan(mask_dev)
    idx, nk = ctx.kept()
    return idx.cpu().numpy(), nk


def test_static_compaction_matches_regular_entry_point_twice_in_a_row():
    import torch
    import paper_2503_21817_b200 as sk
    w1 = wl.config2(C=8, I=8)                                    # 4928 tokens, 1472 kept
    w2 = wl.uniform_batch(3, "bf16", 8, 8, 2, 7, 300, 6, skip_ratio=0.9)   # 626 tokens
    # the caller's buffers, allocated once up front and reused by both calls
    idx = torch.full((w1.N,), -7, dtype=torch.int32, device="cuda")
    nk = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    for w in (w1, w2):
        mask = torch.from_numpy(w.skip_mask).cuda()
        sk.skipffn_compact_static(mask, idx, nk)
        torch.cuda.synchronize()
        got_nk = int(nk.item())
        want_idx, want_nk = _regular(sk, mask)
        assert got_nk == want_nk == w.n_kept
        assert np.array_equal(idx[:got_nk].cpu().numpy(), want_idx)


def test_static_compaction_edges_and_limit():
    import torch
    import paper_2503_21817_b200 as sk
    idx = torch.empty(sk.STATIC_MAX_TOKENS, dtype=torch.int32, device="cuda")
    nk = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    # all skipped, all kept, the largest size the fixed scratch admits
    r = np.random.default_rng(0)
    full = (r.random(sk.STATIC_MAX_TOKENS) < 0.5).astype(np.uint8)
    for m in (np.full(100, 1, np.uint8), np.zeros(100, np.uint8), full):
        mask = torch.from_numpy(m).cuda()
        sk.skipffn_compact_static(mask, idx, nk)
        torch.cuda.synchronize()
        want = np.flatnonzero(m == 0).astype(np.int32)
        assert int(nk.item()) == want.size
        assert np.array_equal(idx[:want.size].cpu().numpy(), want)
    # empty input: Nk = 0, nothing else touched
    sk.skipffn_compact_static(torch.empty(0, dtype=torch.uint8, device="cuda"), idx, nk)
    torch.cuda.synchronize()
    assert int(nk.item()) == 0
    # one token too many: refused with a status, nothing launched
    lib = sk.load_library()
    big = torch.zeros(sk.STATIC_MAX_TOKENS + 1, dtype=torch.uint8, device="cuda")
    big_idx = torch.empty(sk.STATIC_MAX_TOKENS + 1, dtype=torch.int32, device="cuda")
    st = lib.skipffn_compact_static(ctypes.c_void_p(big.data_ptr()), big.numel(),
                                    ctypes.c_void_p(big_idx.data_ptr()), ctypes.c_void_p(nk.data_ptr()), None)
    assert st == 2
    with pytest.raises(sk.SkipFFNError, match="exceeds the fixed scratch"):
        sk.skipffn_compact_static(big, big_idx, nk)
    assert lib.skipffn_compact_static(None, 5, None, None, None) == 1
