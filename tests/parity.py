"""Parity criteria shared by the GPU tests (element-by-element comparison with the fp64 oracle).

bf16 storage / fp32 accumulate: relative Frobenius error <= 5e-3 and, per row, max abs error
<= 3e-2 x RMS of the oracle row.  fp32 mode: relative Frobenius error <= 1e-5.
"""
import numpy as np

BF16_REL_FRO = 5e-3
BF16_ROW_MAXABS = 3e-2
FP32_REL_FRO = 1e-5


def rel_fro(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref)
    num = np.linalg.norm(got - ref)
    return num / den if den > 0 else num


def row_maxabs_ratio(got, ref, floor_matrix_rms=False):
    """max over rows of (max abs error of the row / RMS of the oracle row).  With
    `floor_matrix_rms` a row's RMS is floored by the RMS of the whole matrix."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if ref.size == 0:
        return 0.0
    rms = np.sqrt(np.mean(ref * ref, axis=-1))
    if floor_matrix_rms:
        rms = np.maximum(rms, np.sqrt(np.mean(ref * ref)))
    err = np.max(np.abs(got - ref), axis=-1)
    ok = rms > 0
    ratio = np.zeros_like(err)
    ratio[ok] = err[ok] / rms[ok]
    ratio[~ok] = np.where(err[~ok] == 0, 0.0, np.inf)
    return float(ratio.max())


def check(got, ref, dtype, what, few_terms=False):
    """Assert the stated tolerance for `dtype` ('bf16' or 'fp32').

    `few_terms`: the rows are sums over fewer than 8 kept tokens (weight gradients of a nearly
    empty batch).  A row of dW_gate is then dg[i] * x[t] for a single token, and its relative
    error is that of the one bf16 scalar dg[i], which is unbounded where silu'(g) crosses zero
    because G is saved in bf16.  Those rows are tiny, so the per-row bound is taken against
    max(row RMS, matrix RMS); the Frobenius bound is unchanged."""
    assert np.all(np.isfinite(np.asarray(got, dtype=np.float64))), f"{what}: non-finite values"
    rf = rel_fro(got, ref)
    if dtype == "fp32":
        assert rf <= FP32_REL_FRO, f"{what}: rel Frobenius {rf:.3e} > {FP32_REL_FRO}"
    else:
        assert rf <= BF16_REL_FRO, f"{what}: rel Frobenius {rf:.3e} > {BF16_REL_FRO}"
        rm = row_maxabs_ratio(got, ref, floor_matrix_rms=few_terms)
        assert rm <= BF16_ROW_MAXABS, f"{what}: max abs / row RMS {rm:.3e} > {BF16_ROW_MAXABS}"
    return rf
