"""Seeded synthetic Skip-FFN workloads.

This module only manufactures *data*: Gaussian tensors, skip masks and the
token layouts of the benchmark configurations.  It contains none of the
method's arithmetic (no FFN, no compaction, no gradients) so that both the
CPU oracle and the CUDA path can be fed byte-identical inputs without sharing
any code that could hide a common mistake.

Random numbers are counter based: element ``e`` of tensor ``tensor_id`` under
``seed`` is a pure function of ``(seed, tensor_id, e)`` (SplitMix64 finaliser
-> two uniforms -> Box-Muller), so any slice of any tensor can be regenerated
independently and results do not depend on generation order.

Shapes follow the paper's workloads: 576 visual + 40 text tokens per sample
(24x24 CLIP-336 grid), higher-resolution 48x48 grids, packed variable-length
batches with 576..2880 visual tokens, LLaMA3-8B (C=4096, I=14336) and
Vicuna-13B (C=5120, I=13824) feed-forward shapes.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

_U64 = np.uint64
_GOLD = _U64(0x9E3779B97F4A7C15)

# tensor ids (streams) of the counter-based generator
TID_X, TID_WGATE, TID_WUP, TID_WDOWN, TID_DOUT, TID_MASK, TID_LAYOUT = 1, 2, 3, 4, 5, 6, 7


def _mix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function on a uint64 array (wraps modulo 2**64)."""
    z = z.astype(_U64, copy=True)
    z ^= z >> _U64(30)
    z *= _U64(0xBF58476D1CE4E5B9)
    z ^= z >> _U64(27)
    z *= _U64(0x94D049BB133111EB)
    z ^= z >> _U64(31)
    return z


def _key(seed: int, tensor_id: int) -> np.uint64:
    k = _mix64(np.array([(seed * 0x100000001B3 + tensor_id) & 0xFFFFFFFFFFFFFFFF], dtype=_U64))
    return k[0]


def raw_u64(seed: int, tensor_id: int, start: int, count: int, lane: int = 0) -> np.ndarray:
    """``count`` 64-bit words for elements ``start .. start+count-1``."""
    with np.errstate(over="ignore"):
        ctr = (np.arange(start, start + count, dtype=_U64) * _U64(2) + _U64(lane)) * _GOLD
        return _mix64(ctr + _key(seed, tensor_id))


def uniform01(seed: int, tensor_id: int, start: int, count: int, lane: int = 0) -> np.ndarray:
    """Uniform doubles in the open interval (0, 1)."""
    w = raw_u64(seed, tensor_id, start, count, lane)
    return ((w >> _U64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _normal_chunk(seed, tensor_id, start, n, std, out):
    u1 = uniform01(seed, tensor_id, start, n, 0)
    u2 = uniform01(seed, tensor_id, start, n, 1)
    np.log(u1, out=u1)
    u1 *= -2.0
    np.sqrt(u1, out=u1)
    u2 *= 2.0 * np.pi
    np.cos(u2, out=u2)
    u1 *= u2
    u1 *= std
    out[:] = u1


def normal(seed: int, tensor_id: int, count: int, std: float = 1.0, start: int = 0,
           chunk: int = 1 << 20) -> np.ndarray:
    """``count`` samples of N(0, std^2) as float64 (Box-Muller, cosine branch).  Chunks are
    generated on a thread pool; the values do not depend on the chunking."""
    out = np.empty(count, dtype=np.float64)
    jobs = [(lo, min(chunk, count - lo)) for lo in range(0, count, chunk)]
    if len(jobs) <= 1:
        for lo, n in jobs:
            _normal_chunk(seed, tensor_id, start + lo, n, std, out[lo:lo + n])
        return out
    from concurrent.futures import ThreadPoolExecutor
    import os
    with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 1)) as ex:
        list(ex.map(lambda j: _normal_chunk(seed, tensor_id, start + j[0], j[1], std,
                                            out[j[0]:j[0] + j[1]]), jobs))
    return out


# --------------------------------------------------------------------------- dtypes
def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32/64 values to bfloat16 (round-to-nearest-even); returns uint16 bit patterns."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    b = f.view(np.uint32)
    nan = np.isnan(f)
    bias = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    with np.errstate(over="ignore"):
        r = ((b + bias) >> np.uint32(16)).astype(np.uint16)
    if nan.any():
        r = np.where(nan, ((b >> np.uint32(16)) | np.uint32(0x40)).astype(np.uint16), r)
    return r


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float32 exactly."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round once to the run dtype and return float32 holding exactly those values."""
    if dtype == "bf16":
        return bf16_bits_to_f32(to_bf16_bits(a))
    if dtype == "fp32":
        return np.ascontiguousarray(a, dtype=np.float32)
    raise ValueError(f"unknown dtype {dtype!r}")


# --------------------------------------------------------------------------- masks
def random_subset(seed: int, stream: int, population: int, k: int) -> np.ndarray:
    """Sorted uniformly random k-subset of range(population): positions of the k smallest keys."""
    if k <= 0:
        return np.empty(0, dtype=np.int64)
    keys = raw_u64(seed, TID_MASK, stream * (1 << 20), population)
    order = np.argsort(keys, kind="stable")
    return np.sort(order[:k]).astype(np.int64)


def n_skipped(ratio: float, n_visual: int) -> int:
    return int(np.floor(ratio * n_visual + 0.5))


@dataclass
class Workload:
    """One Skip-FFN problem instance.  Float arrays are float32 holding values that are
    exactly representable in ``dtype`` (so widening them to float64 is lossless)."""
    name: str
    dtype: str
    B: int
    S: int
    C: int
    I: int
    x: np.ndarray            # [N, C]
    skip_mask: np.ndarray    # [N] uint8, nonzero = skipped
    W_gate: np.ndarray       # [I, C]
    W_up: np.ndarray         # [I, C]
    W_down: np.ndarray       # [C, I]
    dout: np.ndarray         # [N, C]
    cu_seqlens: Optional[np.ndarray] = None   # int32 [n_seq + 1] for packed batches
    is_visual: Optional[np.ndarray] = None    # [N] uint8
    meta: dict = field(default_factory=dict)

    @property
    def N(self) -> int:
        return int(self.skip_mask.shape[0])

    @property
    def n_kept(self) -> int:
        return int(self.N - np.count_nonzero(self.skip_mask))


def gaussian_tensors(seed: int, N: int, C: int, I: int, dtype: str, with_weights: bool = True):
    x = round_to(normal(seed, TID_X, N * C, 1.0), dtype).reshape(N, C)
    dout = round_to(normal(seed, TID_DOUT, N * C, 1.0), dtype).reshape(N, C)
    if not with_weights:
        return x, dout, None, None, None
    wg = round_to(normal(seed, TID_WGATE, I * C, 0.02), dtype).reshape(I, C)
    wu = round_to(normal(seed, TID_WUP, I * C, 0.02), dtype).reshape(I, C)
    wd = round_to(normal(seed, TID_WDOWN, C * I, 0.02), dtype).reshape(C, I)
    return x, dout, wg, wu, wd


def _finish(name, dtype, B, S, C, I, mask, seed, cu=None, is_visual=None, meta=None, weights=None):
    N = mask.shape[0]
    if weights is None:
        x, dout, wg, wu, wd = gaussian_tensors(seed, N, C, I, dtype)
    else:
        x, dout, _, _, _ = gaussian_tensors(seed, N, C, I, dtype, with_weights=False)
        wg, wu, wd = weights
    return Workload(name, dtype, B, S, C, I, x, mask.astype(np.uint8), wg, wu, wd, dout,
                    cu, is_visual, meta or {})


def uniform_batch(seed: int, dtype: str, C: int, I: int, B: int, text_before: int, n_visual: int,
                  text_after: int, skip_ratio: Optional[float] = None, n_skip: Optional[int] = None,
                  contiguous_span: bool = False, name: str = "uniform", weights=None) -> Workload:
    """B sequences ``[text_before | n_visual | text_after]``; per sequence an independent random
    subset of visual positions is skipped (or one contiguous span when ``contiguous_span``)."""
    S = text_before + n_visual + text_after
    k = n_skip if n_skip is not None else n_skipped(skip_ratio, n_visual)
    mask = np.zeros((B, S), dtype=np.uint8)
    vis = np.zeros((B, S), dtype=np.uint8)
    vis[:, text_before:text_before + n_visual] = 1
    for b in range(B):
        if contiguous_span:
            # paper layout: retained tokens first, then one skipped span up to the last visual token
            # but one (the final visual token must pass the FFN)
            lo = text_before + n_visual - 1 - k
            mask[b, max(lo, text_before):max(lo, text_before) + min(k, n_visual)] = 1
        else:
            mask[b, text_before + random_subset(seed, b, n_visual, k)] = 1
    return _finish(name, dtype, B, S, C, I, mask.reshape(-1), seed, is_visual=vis.reshape(-1),
                   meta={"n_visual": n_visual, "n_skip_per_seq": k}, weights=weights)


def config1(seed: int = 0, dtype: str = "fp32") -> Workload:
    """Tiny case: C=256, I=688, 8 text + 64 visual + 8 text, 48 visual skipped (Nk=32)."""
    return uniform_batch(seed, dtype, 256, 688, 1, 8, 64, 8, n_skip=48, name="cfg1-tiny")


def config2(seed: int = 0, dtype: str = "bf16", skip_ratio: float = 0.75, C: int = 4096,
            I: int = 14336, B: int = 8, weights=None) -> Workload:
    """LLaMA3-8B-shaped layer: 8 x (20 text + 576 visual + 20 text); 75 % of visual skipped."""
    return uniform_batch(seed, dtype, C, I, B, 20, 576, 20, skip_ratio=skip_ratio,
                         name=f"cfg2-llama3-8b-r{skip_ratio:g}", weights=weights)


def config3(seed: int = 0, dtype: str = "bf16", C: int = 4096, I: int = 14336, B: int = 4,
            weights=None) -> Workload:
    """High-resolution: 4 x (20 text + 48x48 visual + 20 text); visual (r, c) kept iff
    r % 4 == 0 and c % 2 == 0 (87.5 % skipped)."""
    G = 48
    S = 20 + G * G + 20
    v = np.arange(G * G)
    keep = ((v // G) % 4 == 0) & ((v % G) % 2 == 0)
    mask = np.zeros((B, S), dtype=np.uint8)
    mask[:, 20:20 + G * G] = (~keep).astype(np.uint8)
    vis = np.zeros((B, S), dtype=np.uint8)
    vis[:, 20:20 + G * G] = 1
    return _finish("cfg3-highres", dtype, B, S, C, I, mask.reshape(-1), seed,
                   is_visual=vis.reshape(-1), meta={"grid": G}, weights=weights)


def config4(seed: int = 0, dtype: str = "bf16", C: int = 4096, I: int = 14336, n_seq: int = 16,
            weights=None) -> Workload:
    """Packed variable-length batch: per sequence V = 144*U{4..20} visual, T = U{20..200} text laid
    out ``[T//2 text | V visual | rest text]``, skip ratio U[0.5, 0.9] of random visual positions."""
    u = uniform01(seed, TID_LAYOUT, 0, 3 * n_seq)
    cu = [0]
    masks, viss = [], []
    for s in range(n_seq):
        V = 144 * (4 + int(u[3 * s] * 17))
        T = 20 + int(u[3 * s + 1] * 181)
        r = 0.5 + 0.4 * u[3 * s + 2]
        m = np.zeros(T + V, dtype=np.uint8)
        vi = np.zeros(T + V, dtype=np.uint8)
        vi[T // 2:T // 2 + V] = 1
        m[T // 2 + random_subset(seed, s, V, n_skipped(r, V))] = 1
        masks.append(m)
        viss.append(vi)
        cu.append(cu[-1] + T + V)
    mask = np.concatenate(masks)
    return _finish("cfg4-packed", dtype, 1, mask.shape[0], C, I, mask, seed,
                   cu=np.asarray(cu, dtype=np.int32), is_visual=np.concatenate(viss),
                   meta={"n_seq": n_seq}, weights=weights)


SWEEP_RATIOS = (0.0, 0.25, 0.5, 0.75, 0.9, 1.0)
SWEEP_SHAPES = {"llama3-8b": (4096, 14336), "vicuna-13b": (5120, 13824)}


def small_case(seed: int, dtype: str, C: int, I: int, n_seq: int, text: int, n_visual: int,
               skip_ratio: float, name: str = "small") -> Workload:
    """Scaled-down layer with the same token structure; sized for a full CPU-oracle run."""
    return uniform_batch(seed, dtype, C, I, n_seq, text // 2, n_visual, text - text // 2,
                         skip_ratio=skip_ratio, name=name)
