"""Skip-FFN fp64 CPU oracle (TEST INFRASTRUCTURE -- never imported by the product path).

Thin ctypes wrapper around ``skipffn_oracle.c``: argument marshalling only, every number is
produced by the plain C loops.  Inputs may be any float arrays; they are widened to float64
(lossless for values already rounded to bf16 / fp32) before the call.

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s cpu_baseline / reference arm may
import this package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "skipffn_oracle.c")
_LIB = os.path.join(_HERE, "libskipffn_oracle.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (``-O2 -fopenmp``) next to its source; returns the path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-std=c11", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp, bp, i64 = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64
        lib.skipffn_oracle_compact.restype = i64
        lib.skipffn_oracle_compact.argtypes = [bp, i64, ctypes.c_void_p]
        lib.skipffn_oracle_forward.restype = None
        lib.skipffn_oracle_forward.argtypes = [dp, bp, dp, dp, dp, i64, i64, i64, ctypes.c_int, dp]
        lib.skipffn_oracle_backward.restype = None
        lib.skipffn_oracle_backward.argtypes = [dp, bp, dp, dp, dp, dp, i64, i64, i64, dp, dp, dp, dp]
        lib.skipffn_oracle_rows.restype = None
        lib.skipffn_oracle_rows.argtypes = [dp, bp, dp, dp, dp, dp, i64, i64, dp, i64, dp, dp]
        lib.skipffn_oracle_dw_columns.restype = None
        lib.skipffn_oracle_dw_columns.argtypes = [dp, bp, dp, dp, dp, dp, i64, i64, i64, dp, i64,
                                                  dp, dp, dp]
        lib.skipffn_oracle_forward_prenorm.restype = None
        lib.skipffn_oracle_forward_prenorm.argtypes = [dp, bp, dp, ctypes.c_double, dp, dp, dp, i64, i64, i64, dp]
        lib.skipffn_oracle_backward_prenorm.restype = None
        lib.skipffn_oracle_backward_prenorm.argtypes = [dp, bp, dp, ctypes.c_double, dp, dp, dp, dp, i64, i64, i64,
                                                        dp, dp, dp, dp, dp]
        lib.skipffn_oracle_summary_forward.restype = None
        lib.skipffn_oracle_summary_forward.argtypes = [dp, ctypes.c_void_p, i64, i64, dp, dp, dp]
        lib.skipffn_oracle_summary_backward.restype = None
        lib.skipffn_oracle_summary_backward.argtypes = [dp, ctypes.c_void_p, i64, i64, dp, dp, dp, dp]
        lib.skipffn_oracle_token_merge.restype = None
        lib.skipffn_oracle_token_merge.argtypes = [dp, i64, i64, i64, dp, ctypes.c_void_p, ctypes.c_void_p, dp]
        lib.skipffn_oracle_merge_given.restype = None
        lib.skipffn_oracle_merge_given.argtypes = [dp, i64, i64, i64, ctypes.c_void_p, dp]
        lib.skipffn_oracle_kv_compact.restype = i64
        lib.skipffn_oracle_kv_compact.argtypes = [bp, bp, i64, i64, i64, bp]
        lib.skipffn_oracle_kept_cu_seqlens.restype = None
        lib.skipffn_oracle_kept_cu_seqlens.argtypes = [bp, ctypes.c_void_p, i64, ctypes.c_void_p]
        _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _u8(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.uint8).reshape(-1)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def n_threads() -> int:
    """Host threads the OpenMP loops will use (OMP_NUM_THREADS, else all cores)."""
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else (os.cpu_count() or 1)


def compact(skip_mask) -> np.ndarray:
    """Ascending int32 indices of kept tokens (mask byte == 0)."""
    m = _u8(skip_mask)
    idx = np.empty(max(m.size, 1), dtype=np.int32)
    nk = _load().skipffn_oracle_compact(_p(m), m.size, _p(idx))
    return idx[:nk].copy()


def forward(x, skip_mask, W_gate, W_up, W_down, ffn_only: bool = False) -> np.ndarray:
    """``out[N, C]`` in float64: x + FFN(x) on kept rows, x on skipped rows (Eq. 4 / Eq. 5)."""
    x, wg, wu, wd, m = _f64(x), _f64(W_gate), _f64(W_up), _f64(W_down), _u8(skip_mask)
    N, C = x.shape
    I = wg.shape[0]
    assert wg.shape == (I, C) and wu.shape == (I, C) and wd.shape == (C, I) and m.size == N
    out = np.empty((N, C), dtype=np.float64)
    _load().skipffn_oracle_forward(_p(x), _p(m), _p(wg), _p(wu), _p(wd), N, C, I,
                                   1 if ffn_only else 0, _p(out))
    return out


def backward(x, skip_mask, W_gate, W_up, W_down, dout, need_dw: bool = True):
    """``(dx, dW_gate, dW_up, dW_down)`` in float64 for the loss ``sum(dout * out)``."""
    x, wg, wu, wd, m, do = _f64(x), _f64(W_gate), _f64(W_up), _f64(W_down), _u8(skip_mask), _f64(dout)
    N, C = x.shape
    I = wg.shape[0]
    assert wg.shape == (I, C) and wu.shape == (I, C) and wd.shape == (C, I)
    assert do.shape == (N, C) and m.size == N
    dx = np.empty((N, C), dtype=np.float64)
    dwg = np.empty((I, C), dtype=np.float64) if need_dw else None
    dwu = np.empty((I, C), dtype=np.float64) if need_dw else None
    dwd = np.empty((C, I), dtype=np.float64) if need_dw else None
    _load().skipffn_oracle_backward(_p(x), _p(m), _p(wg), _p(wu), _p(wd), _p(do), N, C, I,
                                    _p(dx), _p(dwg), _p(dwu), _p(dwd))
    return dx, dwg, dwu, dwd


def rows(x, skip_mask, W_gate, W_up, W_down, dout, tokens: Sequence[int]):
    """Sampled mode: ``(out_rows, dx_rows)`` ``[len(tokens), C]`` for the listed tokens only.
    ``dout=None`` gives ``(out_rows, None)``."""
    x, wg, wu, wd, m = _f64(x), _f64(W_gate), _f64(W_up), _f64(W_down), _u8(skip_mask)
    do = None if dout is None else _f64(dout)
    tok = np.ascontiguousarray(tokens, dtype=np.int64)
    N, C = x.shape
    I = wg.shape[0]
    assert tok.size == 0 or (tok.min() >= 0 and tok.max() < N)
    out_rows = np.empty((tok.size, C), dtype=np.float64)
    dx_rows = None if do is None else np.empty((tok.size, C), dtype=np.float64)
    _load().skipffn_oracle_rows(_p(x), _p(m), _p(wg), _p(wu), _p(wd), _p(do), C, I, _p(tok),
                                tok.size, _p(out_rows), _p(dx_rows))
    return out_rows, dx_rows


def dw_columns(x, skip_mask, W_gate, W_up, W_down, dout, cols: Sequence[int]):
    """Sampled mode: exact ``dW_gate[cols, :]``, ``dW_up[cols, :]`` and ``dW_down[:, cols].T``
    (each ``[len(cols), C]``) summed over every kept token."""
    x, wg, wu, wd, m, do = _f64(x), _f64(W_gate), _f64(W_up), _f64(W_down), _u8(skip_mask), _f64(dout)
    cc = np.ascontiguousarray(cols, dtype=np.int64)
    N, C = x.shape
    I = wg.shape[0]
    assert cc.size == 0 or (cc.min() >= 0 and cc.max() < I)
    a = np.empty((cc.size, C), dtype=np.float64)
    b = np.empty((cc.size, C), dtype=np.float64)
    c = np.empty((cc.size, C), dtype=np.float64)
    _load().skipffn_oracle_dw_columns(_p(x), _p(m), _p(wg), _p(wu), _p(wd), _p(do), N, C, I,
                                      _p(cc), cc.size, _p(a), _p(b), _p(c))
    return a, b, c


def kv_compact(cache, skip_mask) -> np.ndarray:
    """Skip KV-cache (Eq. 7): ``cache`` ``[planes, N, ...]`` (any dtype) without the rows of the
    skipped tokens, ``[planes, n_kept, ...]``, original order, byte for byte."""
    c = np.ascontiguousarray(cache)
    m = _u8(skip_mask)
    planes, N = c.shape[0], c.shape[1]
    assert m.size == N
    row_bytes = int(np.prod(c.shape[2:], dtype=np.int64)) * c.itemsize
    nk = int(N - np.count_nonzero(m))
    out = np.empty((planes, nk) + c.shape[2:], dtype=c.dtype)
    got = _load().skipffn_oracle_kv_compact(_p(c.view(np.uint8).reshape(-1)), _p(m), planes, N, row_bytes,
                                            _p(out.view(np.uint8).reshape(-1)))
    assert got == nk
    return out


def kept_cu_seqlens(skip_mask, cu_seqlens) -> np.ndarray:
    """Sequence offsets of the pruned cache: number of retained tokens before each offset."""
    m = _u8(skip_mask)
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    out = np.empty_like(cu)
    _load().skipffn_oracle_kept_cu_seqlens(_p(m), _p(cu), cu.size, _p(out))
    return out


def forward_prenorm(x, skip_mask, gamma, eps, W_gate, W_up, W_down) -> np.ndarray:
    """Pre-norm variant: ``x + FFN(RMSNorm(x) * gamma)`` on kept rows, ``x`` on skipped rows."""
    x, g, wg, wu, wd, m = _f64(x), _f64(gamma), _f64(W_gate), _f64(W_up), _f64(W_down), _u8(skip_mask)
    N, C = x.shape
    I = wg.shape[0]
    assert g.shape == (C,) and wg.shape == (I, C) and wu.shape == (I, C) and wd.shape == (C, I) and m.size == N
    out = np.empty((N, C), dtype=np.float64)
    _load().skipffn_oracle_forward_prenorm(_p(x), _p(m), _p(g), float(eps), _p(wg), _p(wu), _p(wd), N, C, I, _p(out))
    return out


def backward_prenorm(x, skip_mask, gamma, eps, W_gate, W_up, W_down, dout, need_dw: bool = True):
    """``(dx, dgamma, dW_gate, dW_up, dW_down)`` of the pre-norm variant for the loss ``sum(dout * out)``."""
    x, g, wg, wu, wd, m, do = (_f64(x), _f64(gamma), _f64(W_gate), _f64(W_up), _f64(W_down), _u8(skip_mask),
                               _f64(dout))
    N, C = x.shape
    I = wg.shape[0]
    dx = np.empty((N, C), dtype=np.float64)
    dg = np.empty(C, dtype=np.float64)
    dwg = np.empty((I, C), dtype=np.float64) if need_dw else None
    dwu = np.empty((I, C), dtype=np.float64) if need_dw else None
    dwd = np.empty((C, I), dtype=np.float64) if need_dw else None
    _load().skipffn_oracle_backward_prenorm(_p(x), _p(m), _p(g), float(eps), _p(wg), _p(wu), _p(wd), _p(do), N, C, I,
                                            _p(dx), _p(dg), _p(dwg), _p(dwu), _p(dwd))
    return dx, dg, dwg, dwu, dwd


def summary_forward(X, offsets, w):
    """Adaptive summary tokens (Eq. 6): ``(xs [n_seg, C], probs [n])`` for packed ``X [n, C]`` whose
    segment s is rows ``offsets[s] .. offsets[s+1]-1``."""
    X, w = _f64(X), _f64(w)
    off = np.ascontiguousarray(offsets, dtype=np.int32)
    n, C = X.shape
    assert w.shape == (C,) and off[0] == 0 and off[-1] == n and np.all(np.diff(off) >= 0)
    xs = np.empty((off.size - 1, C), dtype=np.float64)
    probs = np.zeros(max(n, 1), dtype=np.float64)
    _load().skipffn_oracle_summary_forward(_p(X), _p(off), off.size - 1, C, _p(w), _p(xs), _p(probs))
    return xs, probs[:n]


def summary_backward(X, offsets, w, dxs):
    """``(dX [n, C], dw [C])`` of the adaptive summary layer for the loss ``sum(dxs * xs)``."""
    X, w, dxs = _f64(X), _f64(w), _f64(dxs)
    off = np.ascontiguousarray(offsets, dtype=np.int32)
    n, C = X.shape
    dX = np.zeros((n, C), dtype=np.float64)
    dw = np.empty(C, dtype=np.float64)
    _load().skipffn_oracle_summary_backward(_p(X), _p(off), off.size - 1, C, _p(w), _p(dxs), _p(dX), _p(dw))
    return dX, dw


def token_merge(X, k):
    """Token merge of section 4.1: ``(avg [n], kept [k], assign [n], merged [k, C])``."""
    X = _f64(X)
    n, C = X.shape
    assert 0 < k <= n
    avg = np.empty(n, dtype=np.float64)
    kept = np.empty(k, dtype=np.int32)
    assign = np.empty(n, dtype=np.int32)
    merged = np.empty((k, C), dtype=np.float64)
    _load().skipffn_oracle_token_merge(_p(X), n, C, k, _p(avg), _p(kept), _p(assign), _p(merged))
    return avg, kept, assign, merged


def merge_given(X, k, assign):
    """Mean of the rows assigned to each of the k groups."""
    X = _f64(X)
    a = np.ascontiguousarray(assign, dtype=np.int32)
    n, C = X.shape
    merged = np.empty((k, C), dtype=np.float64)
    _load().skipffn_oracle_merge_given(_p(X), n, C, k, _p(a), _p(merged))
    return merged
