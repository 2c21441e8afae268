"""Skip-FFN fp64 oracle, second statement (TEST INFRASTRUCTURE -- never imported by the product path).

The same definition as ``skipffn_oracle.c`` (paper section 4.2, Eq. 4 / Eq. 5, SwiGLU body fixed by
the section 6.2 cost model and Table 1), written with whole matrices instead of one token at a
time: the retained rows are selected by boolean indexing and every contraction is one float64
library matmul.  Nothing is tiled, fused or reordered; each line is one term of the definition or
of its derivative.  Because a float64 BLAS matmul is about a thousand times faster than the plain
C loops, this statement can produce EVERY element of out, dx, dW_gate, dW_up, dW_down (and dgamma
of the pre-norm variant) at the full benchmark sizes in seconds, where the C loops can only afford
sampled rows and columns.

Pins (tests/test_oracle_pins.py): equality with the per-token C loops to rounding on random cases
with every mask kind, central finite differences of its own forward, the scalar closed form, and
the identities of Eq. 5 (skipped rows bit-equal to the input, all-skipped gives zero gradients).
"""
from __future__ import annotations

import numpy as np


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _sigmoid(z: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-z))


def _rstd(xk: np.ndarray, eps: float) -> np.ndarray:
    return 1.0 / np.sqrt(np.mean(xk * xk, axis=1, keepdims=True) + eps)


def forward_backward(x, skip_mask, W_gate, W_up, W_down, dout=None, gamma=None, eps: float = 0.0):
    """All results of one forward (+ backward when ``dout`` is given) as a dict of float64 arrays:
    ``out`` and, with ``dout``, ``dx, dW_gate, dW_up, dW_down`` (+ ``dgamma`` with ``gamma``).

    ``gamma`` selects the pre-norm variant: the FFN input of a retained token is
    ``x / sqrt(mean(x^2) + eps) * gamma`` while the residual stays ``x``; skipped tokens are the
    identity either way."""
    x, wg, wu, wd = _f64(x), _f64(W_gate), _f64(W_up), _f64(W_down)
    keep = np.ascontiguousarray(skip_mask, dtype=np.uint8).reshape(-1) == 0
    N, C = x.shape
    I = wg.shape[0]
    assert wg.shape == (I, C) and wu.shape == (I, C) and wd.shape == (C, I) and keep.size == N
    xk = x[keep]                                   # retained rows, original order
    if gamma is not None:
        gam = _f64(gamma)
        rstd = _rstd(xk, eps)
        xh = xk * rstd                             # unit-RMS rows
        a = xh * gam                               # the FFN input
    else:
        a = xk
    G = a @ wg.T                                   # gate projection
    U = a @ wu.T                                   # up projection
    S = _sigmoid(G)
    H = G * S * U                                  # silu(G) * U
    out = x.copy()                                 # Eq. 5: skipped rows are the input
    out[keep] = xk + H @ wd.T                      # Eq. 4: residual + FFN
    res = {"out": out, "n_kept": int(keep.sum())}
    if dout is None:
        return res
    do = _f64(dout)
    assert do.shape == (N, C)
    dok = do[keep]
    dH = dok @ wd                                  # through the down projection
    dU = dH * (G * S)                              # d/dU of silu(G) * U
    dG = dH * U * (S * (1.0 + G * (1.0 - S)))      # silu'(G)
    res["dW_down"] = dok.T @ H
    res["dW_gate"] = dG.T @ a
    res["dW_up"] = dU.T @ a
    da = dG @ wg + dU @ wu                         # gradient w.r.t. the FFN input
    dx = do.copy()                                 # derivative of the identity / of the residual
    if gamma is not None:
        res["dgamma"] = np.sum(da * xh, axis=0)
        gy = da * gam
        dx[keep] = dok + rstd * (gy - xh * np.mean(gy * xh, axis=1, keepdims=True))
    else:
        dx[keep] = dok + da
    res["dx"] = dx
    return res
