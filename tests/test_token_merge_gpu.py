"""Token merge (section 4.1) on the GPU against the fp64 oracle.  Floating point decides integers
here (which tokens are kept, where each token goes), so what is unique is compared exactly and the
rest is checked for validity within the arithmetic's tolerance; every merged row is checked against
the mean of its own (validated) group, and against the oracle's row for every group whose
membership the two sides agree on (the oracle is never fed anything the GPU produced)."""
import numpy as np
import pytest

import oracle
import workloads as wl
from gpu_util import to_dev, to_host
from parity import check

pytestmark = pytest.mark.gpu


def _tokens(seed, n, C, dtype, clusters=24, noise=0.35):
    centers = wl.normal(seed, wl.TID_WGATE, clusters * C).reshape(clusters, C)
    which = (wl.raw_u64(seed, wl.TID_LAYOUT, 0, n) % np.uint64(clusters)).astype(np.int64)
    X = centers[which] + noise * wl.normal(seed, wl.TID_X, n * C).reshape(n, C)
    return wl.round_to(X, dtype)


def _validate(X, k, kept, assign, merged, dtype):
    n, C = X.shape
    X64 = X.astype(np.float64)
    avg, o_kept, o_assign, o_merged = oracle.token_merge(X64, k)
    tol_avg = 1e-5 if dtype == "fp32" else 1e-4
    tol_sim = 1e-4 if dtype == "fp32" else 2e-2
    # (2) the kept set: k distinct tokens in ascending order; everything clearly below the k-th
    # smallest average is in, everything clearly above is out
    assert kept.shape == (k,) and np.all(np.diff(kept) > 0) and kept.min() >= 0 and kept.max() < n
    thr = np.sort(avg)[k - 1]
    in_set = np.zeros(n, bool)
    in_set[kept] = True
    assert in_set[avg < thr - tol_avg].all() and not in_set[avg > thr + tol_avg].any()
    if np.min(np.abs(np.delete(np.sort(avg), k - 1) - thr)) > 10 * tol_avg:
        assert np.array_equal(kept, o_kept)                         # no near-tie at the boundary: unique
    # (3) assignment: kept tokens to themselves, the others to a kept token whose cosine similarity
    # is the maximum within the tolerance of the arithmetic
    assert np.array_equal(assign[kept], np.arange(k))
    Xh = X64 / np.maximum(np.linalg.norm(X64, axis=1, keepdims=True), 1e-300)
    S = Xh @ Xh[kept].T
    rest = np.flatnonzero(~in_set)
    assert np.all((assign >= 0) & (assign < k))
    chosen = S[rest, assign[rest]]
    assert np.all(chosen >= S[rest].max(1) - tol_sim)
    gap = np.sort(S[rest], axis=1)
    clear = (gap[:, -1] - gap[:, -2]) > 4 * tol_sim if k > 1 else np.ones(rest.size, bool)
    assert np.array_equal(assign[rest][clear], np.argmax(S[rest], axis=1)[clear])
    assert clear.any()                                             # some decisions are unambiguous
    # merged rows.  The integer assignment above is valid (several are, within the arithmetic's
    # tolerance), so EVERY merged row is checked against the mean of the rows of its own group,
    # written out here from the definition of the operator (a validity check: no oracle call takes
    # anything the GPU produced).  Groups on whose members the oracle agrees are also compared
    # with the oracle's rows.
    groups = np.zeros((k, C))
    count = np.zeros(k)
    np.add.at(groups, assign, X64)
    np.add.at(count, assign, 1.0)
    assert count.min() >= 1                                        # a kept token is in its own group
    check(merged, groups / count[:, None], dtype, "merged rows vs mean of own group")
    if np.array_equal(kept, o_kept):
        same = np.array([np.array_equal(np.flatnonzero(assign == j), np.flatnonzero(o_assign == j)) for j in range(k)])
        assert same.mean() >= 0.3
        check(merged[same], o_merged[same], dtype, "merged")
    return bool(np.array_equal(kept, o_kept))


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("n,C,k", [(576, 512, 144), (300, 264, 20), (2304, 1024, 288)])
def test_token_merge_against_oracle(dtype, n, C, k):
    import torch
    import paper_2503_21817_b200 as sk
    X = _tokens(n + k, n, C, dtype)
    Xd = to_dev(X, dtype)
    kept, assign, merged = sk.token_merge(Xd, k, poll=True)      # poll: no device-side wait timed out
    same_kept = _validate(X, k, kept.cpu().numpy(), assign.cpu().numpy(), to_host(merged), dtype)
    if dtype == "fp32":
        assert same_kept                      # fp32 reproduces the oracle's kept set on this data
    k2, a2, m2 = sk.token_merge(Xd, k)                              # run twice: bit-identical
    assert torch.equal(kept, k2) and torch.equal(assign, a2) and torch.equal(merged, m2)


def test_token_merge_keep_all_and_argument_checks():
    import torch
    import paper_2503_21817_b200 as sk
    X = _tokens(3, 64, 128, "bf16")
    Xd = to_dev(X, "bf16")
    kept, assign, merged = sk.token_merge(Xd, 64)                    # k = n: nothing to merge
    torch.cuda.synchronize()
    assert np.array_equal(kept.cpu().numpy(), np.arange(64)) and np.array_equal(assign.cpu().numpy(), np.arange(64))
    assert torch.equal(merged, Xd)
    with pytest.raises(sk.SkipFFNError):
        sk.token_merge(Xd, 30)                                       # k not a multiple of 4
    with pytest.raises(sk.SkipFFNError):
        sk.token_merge(Xd, 68)                                       # k > n
