"""Skip KV-cache (Eq. 7) on the GPU against the CPU oracle: byte-exact row selection."""
import numpy as np
import pytest

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu


def _cache(planes, N, heads, d, seed, dtype=np.float32):
    v = wl.normal(seed, wl.TID_X, planes * N * heads * d).astype(dtype)
    return v.reshape(planes, N, heads, d)


@pytest.mark.parametrize("case", ["cfg2-mask", "packed", "all-kept", "all-skipped", "one-row"])
def test_kv_compact_matches_oracle_bytes(case):
    import torch
    import paper_2503_21817_b200 as sk
    cu = None
    if case == "cfg2-mask":
        mask = wl.config2(C=8, I=8).skip_mask                       # 4928 tokens, 1472 kept
    elif case == "packed":
        w = wl.config4(seed=2, C=8, I=8, n_seq=4)
        mask, cu = w.skip_mask, w.cu_seqlens
    elif case == "all-kept":
        mask = np.zeros(300, np.uint8)
    elif case == "all-skipped":
        mask = np.ones(300, np.uint8)
    else:
        mask = np.ones(257, np.uint8)
        mask[200] = 0
    N = mask.size
    planes, heads, d = 6, 2, 24                                      # 6 planes of rows of 96 bytes (bf16)
    host = wl.to_bf16_bits(_cache(planes, N, heads, d, seed=N)).reshape(planes, N, heads, d)
    src = torch.from_numpy(host.view(np.int16)).cuda().view(torch.bfloat16)
    ctx = sk.SkipFFN(64, 64, N)
    ctx.plan(torch.from_numpy(mask).cuda())
    sentinel = torch.full_like(src, -7.0)
    dst, new_cu = ctx.kv_compact(src, dst=sentinel.clone(), cu_seqlens=cu)
    ctx.poll()
    ref = oracle.kv_compact(host, mask)
    nk = ref.shape[1]
    got = dst.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got[:, :nk], ref)
    # rows past Nk are not written
    assert np.array_equal(got[:, nk:], sentinel.view(torch.int16).cpu().numpy().view(np.uint16)[:, nk:])
    if cu is not None:
        assert np.array_equal(new_cu.cpu().numpy(), oracle.kept_cu_seqlens(mask, cu))


def test_kv_compact_3d_fp32_and_argument_checks():
    import torch
    import paper_2503_21817_b200 as sk
    mask = wl.uniform_batch(4, "bf16", 8, 8, 2, 5, 90, 5, skip_ratio=0.7).skip_mask
    N = mask.size
    host = _cache(3, N, 1, 20, seed=5).reshape(3, N, 20)             # [planes, N, row]: 80-byte rows
    src = torch.from_numpy(host).cuda()
    ctx = sk.SkipFFN(64, 64, N)
    with pytest.raises(sk.SkipFFNError):
        ctx.kv_compact(src)                                          # nothing planned yet
    ctx.plan(torch.from_numpy(mask).cuda())
    dst, _ = ctx.kv_compact(src)
    ref = oracle.kv_compact(host, mask)
    assert dst[:, :ref.shape[1]].cpu().numpy().tobytes() == ref.tobytes()
    with pytest.raises(sk.SkipFFNError):
        ctx.kv_compact(src, dst=src)                                 # overlapping caches
    with pytest.raises(sk.SkipFFNError):
        ctx.kv_compact(torch.zeros(2, N, 6, device="cuda"))          # 24-byte rows: not a multiple of 16
