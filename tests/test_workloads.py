"""The seeded input generators: determinism, shapes and mask structure of each configuration."""
import numpy as np

import workloads as wl


def test_counter_based_generator_is_order_independent():
    a = wl.normal(3, wl.TID_X, 5000)
    b = wl.normal(3, wl.TID_X, 100, start=1234)
    assert np.array_equal(a[1234:1334], b)
    assert not np.array_equal(a[:100], wl.normal(4, wl.TID_X, 100))
    assert not np.array_equal(a[:100], wl.normal(3, wl.TID_DOUT, 100))
    big = wl.normal(0, wl.TID_X, 1 << 21)
    assert abs(big.mean()) < 5e-3 and abs(big.std() - 1) < 5e-3


def test_bf16_rounding_is_rne_and_lossless_roundtrip():
    import torch
    f = np.concatenate([np.random.default_rng(0).normal(size=4096).astype(np.float32),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, -1e-40], np.float32)])
    bits = wl.to_bf16_bits(f)
    want = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    again = wl.to_bf16_bits(wl.bf16_bits_to_f32(bits))
    assert np.array_equal(bits, again)


def test_config_token_counts():
    c1 = wl.config1()
    assert (c1.N, c1.n_kept, c1.C, c1.I) == (80, 32, 256, 688)
    assert not c1.skip_mask[:8].any() and not c1.skip_mask[72:].any()
    c2 = wl.config2(C=8, I=16)
    assert (c2.N, c2.n_kept) == (4928, 1472)
    m = c2.skip_mask.reshape(8, 616)
    assert (m.sum(1) == 432).all() and not m[:, :20].any() and not m[:, 596:].any()
    assert not np.array_equal(m[0], m[1])
    c3 = wl.config3(C=8, I=16)
    assert (c3.N, c3.n_kept) == (9376, 1312)
    c4 = wl.config4(C=8, I=16)
    cu = c4.cu_seqlens
    assert cu.shape == (17,) and cu[-1] == c4.N
    for s in range(16):
        seg_vis = c4.is_visual[cu[s]:cu[s + 1]]
        V = int(seg_vis.sum())
        assert V % 144 == 0 and 576 <= V <= 2880
        assert 20 <= (cu[s + 1] - cu[s]) - V <= 200
        r = c4.skip_mask[cu[s]:cu[s + 1]].sum() / V
        assert 0.49 <= r <= 0.91
    assert not c4.skip_mask[c4.is_visual == 0].any()


def test_sweep_ratios_and_span_layout():
    kept = [wl.config2(C=8, I=8, skip_ratio=r).n_kept for r in wl.SWEEP_RATIOS]
    assert kept == [4928, 3776, 2624, 1472, 784, 320]
    w = wl.uniform_batch(0, "bf16", 8, 8, 2, 20, 576, 20, skip_ratio=0.75, contiguous_span=True)
    m = w.skip_mask.reshape(2, 616)
    for b in range(2):
        pos = np.flatnonzero(m[b])
        assert pos.size == 432 and np.all(np.diff(pos) == 1)
        assert m[b, 20 + 575] == 0            # the final visual token passes the FFN
    d = wl.config1(dtype="bf16")
    assert np.array_equal(wl.round_to(d.x, "bf16"), d.x)
