"""ctypes binding of the Skip-FFN C ABI (see ``include/skipffn.h`` for the contract)."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

BF16, FP32 = 0, 1
PATH_DEFAULT, PATH_SIMT = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libskipffn.so")
_lib: Optional[ctypes.CDLL] = None

# every symbol the header declares
EXPORTS = ["skipffn_workspace_bytes", "skipffn_saved_create", "skipffn_saved_destroy",
           "skipffn_plan", "skipffn_forward", "skipffn_backward", "skipffn_get_kept",
           "skipffn_get_intermediate", "skipffn_poll", "skipffn_last_launches", "skipffn_flops",
           "skipffn_strerror", "skipffn_profile_enable", "skipffn_profile_read",
           "skipffn_compact_static", "skipffn_schedule_segment", "skipffn_kv_compact",
           "skipffn_forward_prenorm", "skipffn_backward_prenorm", "skipffn_summary_scratch_bytes",
           "skipffn_summary_forward", "skipffn_summary_backward", "skipffn_token_merge_scratch_bytes",
           "skipffn_token_merge", "skipffn_tune", "skipffn_saved_bytes", "skipffn_scratch_bytes",
           "skipffn_workspace_bytes_kept", "skipffn_saved_create_kept", "skipffn_saved_create_split",
           "skipffn_token_merge_poll", "skipffn_schedule_plan_segment"]
STATIC_MAX_TOKENS = 65536   # SKIPFFN_STATIC_MAX_TOKENS

TUNABLES = {"tile_n": 0, "streamk": 1, "stages": 2, "lose_handover": 3, "one_box": 4, "tma_stores": 5, "gather": 6,
            "panel_sync": 7}
PROFILE_SLOTS = ["compact", "route_x", "gateup", "down", "route_dout", "dh", "dw_down", "dw_gate",
                 "dw_up", "dx", "norm_bwd", "recompute"]


class SkipFFNError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {skipffn_strerror(status)} (status {status})")


class _Config(ctypes.Structure):
    _fields_ = [("C", ctypes.c_int32), ("I", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("dense", ctypes.c_int32), ("grad_dtype_fp32", ctypes.c_int32),
                ("accumulate_dw", ctypes.c_int32), ("path", ctypes.c_int32),
                ("prenorm", ctypes.c_int32), ("debug", ctypes.c_int32), ("recompute", ctypes.c_int32)]


def load_library() -> ctypes.CDLL:
    """Load ``libskipffn.so`` (built in-tree by ``paper_2503_21817_b200.build.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with "
                           "`python -m paper_2503_21817_b200.build` (there is no fallback path)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    cfgp = ctypes.POINTER(_Config)
    lib.skipffn_workspace_bytes.restype = ctypes.c_size_t
    lib.skipffn_workspace_bytes.argtypes = [cfgp, i64]
    lib.skipffn_saved_create.restype = i32
    lib.skipffn_saved_create.argtypes = [ctypes.POINTER(vp), cfgp, vp, ctypes.c_size_t, i64]
    for fn in (lib.skipffn_saved_bytes, lib.skipffn_scratch_bytes, lib.skipffn_workspace_bytes_kept):
        fn.restype = ctypes.c_size_t
        fn.argtypes = [cfgp, i64, i64]
    lib.skipffn_saved_create_kept.restype = i32
    lib.skipffn_saved_create_kept.argtypes = [ctypes.POINTER(vp), cfgp, vp, ctypes.c_size_t, i64, i64]
    lib.skipffn_saved_create_split.restype = i32
    lib.skipffn_saved_create_split.argtypes = [ctypes.POINTER(vp), cfgp, vp, ctypes.c_size_t, vp, ctypes.c_size_t, i64, i64]
    lib.skipffn_saved_destroy.restype = None
    lib.skipffn_saved_destroy.argtypes = [vp]
    lib.skipffn_plan.restype = i32
    lib.skipffn_plan.argtypes = [vp, vp, i64, vp]
    lib.skipffn_tune.restype = i32
    lib.skipffn_tune.argtypes = [vp, i32, i32]
    lib.skipffn_forward.restype = i32
    lib.skipffn_forward.argtypes = [vp, vp, vp, i64, i64, vp, i32, vp, vp, vp, vp, vp]
    lib.skipffn_backward.restype = i32
    lib.skipffn_backward.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.skipffn_forward_prenorm.restype = i32
    lib.skipffn_forward_prenorm.argtypes = [vp, vp, vp, i64, i64, vp, i32, vp, ctypes.c_float, vp, vp, vp, vp, vp]
    lib.skipffn_backward_prenorm.restype = i32
    lib.skipffn_backward_prenorm.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    lib.skipffn_get_kept.restype = i32
    lib.skipffn_get_kept.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.skipffn_get_intermediate.restype = i32
    lib.skipffn_get_intermediate.argtypes = [vp, i32, ctypes.POINTER(vp)]
    lib.skipffn_poll.restype = i32
    lib.skipffn_poll.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.skipffn_last_launches.restype = i32
    lib.skipffn_last_launches.argtypes = [vp, i32]
    lib.skipffn_flops.restype = ctypes.c_double
    lib.skipffn_flops.argtypes = [cfgp, i64]
    lib.skipffn_profile_enable.restype = i32
    lib.skipffn_profile_enable.argtypes = [vp, i32]
    lib.skipffn_profile_read.restype = i32
    lib.skipffn_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.skipffn_compact_static.restype = i32
    lib.skipffn_compact_static.argtypes = [vp, i64, vp, vp, vp]
    lib.skipffn_schedule_segment.restype = i32
    lib.skipffn_schedule_segment.argtypes = [i32, i32, i32, i32, i32, i32, ctypes.POINTER(i32)]
    lib.skipffn_kv_compact.restype = i32
    lib.skipffn_kv_compact.argtypes = [vp, vp, vp, i64, i64, i64, vp, i32, vp, vp]
    lib.skipffn_summary_scratch_bytes.restype = ctypes.c_size_t
    lib.skipffn_summary_scratch_bytes.argtypes = [i64, i32]
    lib.skipffn_summary_forward.restype = i32
    lib.skipffn_summary_forward.argtypes = [vp, vp, i32, i64, i32, i32, vp, vp, vp, vp]
    lib.skipffn_summary_backward.restype = i32
    lib.skipffn_summary_backward.argtypes = [vp, vp, i32, i64, i32, i32, vp, vp, vp, vp, vp, i32, vp,
                                             ctypes.c_size_t, vp]
    lib.skipffn_token_merge_scratch_bytes.restype = ctypes.c_size_t
    lib.skipffn_token_merge_scratch_bytes.argtypes = [i64, i32, i32, i32]
    lib.skipffn_token_merge.restype = i32
    lib.skipffn_token_merge.argtypes = [vp, i64, i32, i32, i32, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.skipffn_token_merge_poll.restype = i32
    lib.skipffn_token_merge_poll.argtypes = [vp, i64, i32, i32, i32, vp, ctypes.POINTER(i32)]
    lib.skipffn_strerror.restype = ctypes.c_char_p
    lib.skipffn_strerror.argtypes = [i32]
    _lib = lib
    return lib


def _cfg(C, I, dtype=BF16, dense=False, grad_fp32=False, accumulate_dw=False, path=PATH_DEFAULT,
         prenorm=False, debug=False, recompute=False):
    return _Config(int(C), int(I), int(dtype), int(bool(dense)), int(bool(grad_fp32)),
                   int(bool(accumulate_dw)), int(path), int(bool(prenorm)), int(bool(debug)), int(bool(recompute)))


def skipffn_workspace_bytes(C, I, max_tokens, dtype=BF16) -> int:
    c = _cfg(C, I, dtype)
    return int(load_library().skipffn_workspace_bytes(ctypes.byref(c), int(max_tokens)))


def skipffn_flops(C, I, n_kept) -> float:
    c = _cfg(C, I)
    return float(load_library().skipffn_flops(ctypes.byref(c), int(n_kept)))


def skipffn_strerror(status: int) -> str:
    return load_library().skipffn_strerror(int(status)).decode()


def skipffn_schedule(workers: int, tiles: int, k_blocks: int, split_k: bool, worker: int):
    """Segments ``(tile, kb0, kb1, partial, src_lo)`` of one worker's schedule, in processing order
    (``skipffn_schedule_segment``; host only)."""
    lib = load_library()
    seg = (ctypes.c_int32 * 5)()
    n = lib.skipffn_schedule_segment(workers, tiles, k_blocks, int(split_k), worker, -1, seg)
    if n < 0:
        raise SkipFFNError(1, "skipffn_schedule_segment")
    out = []
    for i in range(n):
        lib.skipffn_schedule_segment(workers, tiles, k_blocks, int(split_k), worker, i, seg)
        out.append(tuple(seg))
    return out


def skipffn_schedule_plan(workers: int, panels: int, token_tiles: int, k_blocks: int, min_saving: int,
                          group_mode: int, worker: int):
    """Segments ``(tile, kb0, kb1, partial, first_source_worker, source_stride)`` of one worker's
    schedule of a token problem, worker groups included (``skipffn_schedule_plan_segment``; host only)."""
    lib = load_library()
    seg = (ctypes.c_int32 * 6)()
    args = (workers, panels, token_tiles, k_blocks, min_saving, group_mode, worker)
    n = lib.skipffn_schedule_plan_segment(*args, -1, seg)
    if n < 0:
        raise SkipFFNError(1, "skipffn_schedule_plan_segment")
    out = []
    for i in range(n):
        lib.skipffn_schedule_plan_segment(*args, i, seg)
        out.append(tuple(seg))
    return out


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_of(t):
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream(t.device).cuda_stream)


def summary_forward(X, seg_offsets, w):
    """Adaptive summary tokens (``skipffn_summary_forward``, Eq. 6).  ``X`` ``[n, C]`` packed rows,
    ``seg_offsets`` int32 CUDA tensor ``[n_seg + 1]``, ``w`` ``[C]``.  Returns ``(xs [n_seg, C],
    probs [n] fp32)``; ``probs`` is what the backward needs."""
    import torch
    dtype = BF16 if X.dtype == torch.bfloat16 else FP32
    n, C = X.shape
    n_seg = seg_offsets.numel() - 1
    xs = torch.empty(n_seg, C, dtype=X.dtype, device=X.device)
    probs = torch.empty(max(n, 1), dtype=torch.float32, device=X.device)
    st = load_library().skipffn_summary_forward(_ptr(X), _ptr(seg_offsets), n_seg, n, C, dtype, _ptr(w), _ptr(xs),
                                                _ptr(probs), _stream_of(X))
    if st != 0:
        raise SkipFFNError(st, "skipffn_summary_forward")
    return xs, probs[:n]


def summary_backward(X, seg_offsets, w, probs, dxs, dw_fp32=False):
    """``(dX, dw)`` of the adaptive summary layer (``skipffn_summary_backward``)."""
    import torch
    lib = load_library()
    dtype = BF16 if X.dtype == torch.bfloat16 else FP32
    n, C = X.shape
    n_seg = seg_offsets.numel() - 1
    dX = torch.empty_like(X)
    dw = torch.empty(C, dtype=torch.float32 if (dw_fp32 or dtype == FP32) else X.dtype, device=X.device)
    nbytes = int(lib.skipffn_summary_scratch_bytes(n, C))
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=X.device)
    st = lib.skipffn_summary_backward(_ptr(X), _ptr(seg_offsets), n_seg, n, C, dtype, _ptr(w), _ptr(probs),
                                      _ptr(dxs), _ptr(dX), _ptr(dw), int(dw_fp32), _ptr(scratch), nbytes,
                                      _stream_of(X))
    if st != 0:
        raise SkipFFNError(st, "skipffn_summary_backward")
    return dX, dw


def token_merge(X, k: int, poll: bool = False):
    """Token merge of section 4.1 (``skipffn_token_merge``): ``(kept [k], assign [n], merged [k, C])``
    for the tokens ``X [n, C]`` (bf16 or fp32 CUDA tensor).  ``poll=True`` synchronises the stream
    afterwards and raises if the tensor-core kernel reported a timed-out wait
    (``skipffn_token_merge_poll``)."""
    import torch
    lib = load_library()
    dtype = BF16 if X.dtype == torch.bfloat16 else FP32
    n, C = X.shape
    kept = torch.empty(k, dtype=torch.int32, device=X.device)
    assign = torch.empty(n, dtype=torch.int32, device=X.device)
    merged = torch.empty(k, C, dtype=X.dtype, device=X.device)
    nbytes = int(lib.skipffn_token_merge_scratch_bytes(n, C, k, dtype))
    scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=X.device)
    sp = (scratch.data_ptr() + 255) // 256 * 256
    st = lib.skipffn_token_merge(_ptr(X), n, C, k, dtype, _ptr(kept), _ptr(assign), _ptr(merged),
                                 ctypes.c_void_p(sp), nbytes, _stream_of(X))
    if st != 0:
        raise SkipFFNError(st, "skipffn_token_merge")
    if poll:
        site = ctypes.c_int32(0)
        st = lib.skipffn_token_merge_poll(ctypes.c_void_p(sp), n, C, k, dtype, _stream_of(X), ctypes.byref(site))
        if st != 0:
            raise SkipFFNError(st, f"skipffn_token_merge_poll (site {site.value})")
    return kept, assign, merged


def skipffn_compact_static(skip_mask, idx, nk) -> None:
    """Kept-row list for callers that cannot allocate device memory (``skipffn_compact_static``).

    All three arguments are CUDA tensors the caller already owns: ``skip_mask`` uint8 ``[N]``,
    ``idx`` int32 with at least N entries (the first Nk receive the ascending kept indices), ``nk``
    int32 with one entry.  Neither this wrapper nor the library call allocates anything; the
    kernel's scratch is a fixed array inside the library, which limits N to ``STATIC_MAX_TOKENS``
    and means that calls overlapping on the GPU must be serialised by the caller.  Enqueued on the
    current torch stream of the tensors' GPU, which is made current for the call."""
    import torch
    N = skip_mask.numel()
    if skip_mask.dtype != torch.uint8 or idx.dtype != torch.int32 or nk.dtype != torch.int32:
        raise ValueError("skip_mask must be uint8, idx and nk int32")
    if not (skip_mask.is_cuda and idx.is_cuda and nk.is_cuda and skip_mask.is_contiguous()
            and idx.is_contiguous()) or idx.numel() < N or nk.numel() < 1:
        raise ValueError("skip_mask, idx (>= N entries) and nk (1 entry) must be contiguous CUDA tensors")
    if idx.device != skip_mask.device or nk.device != skip_mask.device:
        raise ValueError("skip_mask, idx and nk must live on the same GPU")
    # the library resolves its fixed array for the CURRENT device, so make the tensors' GPU current
    with torch.cuda.device(skip_mask.device):
        stream = ctypes.c_void_p(torch.cuda.current_stream(skip_mask.device).cuda_stream)
        st = load_library().skipffn_compact_static(_ptr(skip_mask), N, _ptr(idx), _ptr(nk), stream)
    if st == 2:
        raise SkipFFNError(st, f"skipffn_compact_static: N = {N} exceeds the fixed scratch of "
                               f"{STATIC_MAX_TOKENS} tokens")
    if st != 0:
        raise SkipFFNError(st, "skipffn_compact_static")


class SkipFFN:
    """One Skip-FFN sublayer context: owns the workspace tensor and the ``skipffn_saved`` handle.

    ``forward`` / ``backward`` / ``plan`` / ``poll`` mirror ``skipffn_forward`` /
    ``skipffn_backward`` / ``skipffn_plan`` / ``skipffn_poll``; tensors are CUDA tensors whose
    ``data_ptr()`` is handed to the library, work is enqueued on the current torch stream.
    """

    def __init__(self, C: int, I: int, max_tokens: int, dtype: int = BF16, dense: bool = False,
                 grad_fp32: bool = False, accumulate_dw: bool = False, path: int = PATH_DEFAULT,
                 device="cuda", prenorm: bool = False, debug: bool = False, recompute: bool = False,
                 max_kept=None, scratch_from=None):
        """``max_kept`` bounds the kept tokens of any call (default: ``max_tokens``) and sizes the
        compacted arrays.  ``recompute``: the forward keeps no G, U, H.  ``scratch_from``: another
        context of the same configuration whose scratch buffer this one shares (calls of the two
        must not overlap on the GPU)."""
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("Skip-FFN needs a CUDA device (sm_100a); there is no CPU path")
        self._torch = torch
        self.lib = load_library()
        self.C, self.I, self.dtype, self.max_tokens = int(C), int(I), int(dtype), int(max_tokens)
        self.max_kept = self.max_tokens if max_kept is None else int(max_kept)
        self.grad_fp32 = bool(grad_fp32) or dtype == FP32
        self.prenorm = bool(prenorm)
        self.cfg = _cfg(C, I, dtype, dense, grad_fp32, accumulate_dw, path, prenorm, debug, recompute)
        self.device = torch.device(device)
        cfgp = ctypes.byref(self.cfg)
        self.saved_bytes = int(self.lib.skipffn_saved_bytes(cfgp, self.max_tokens, self.max_kept))
        self.scratch_bytes = int(self.lib.skipffn_scratch_bytes(cfgp, self.max_tokens, self.max_kept))
        if self.saved_bytes == 0:
            raise SkipFFNError(1, "skipffn_saved_bytes")

        def aligned(t):
            return (t.data_ptr() + 1023) // 1024 * 1024
        self.workspace = torch.empty(self.saved_bytes + 1024, dtype=torch.uint8, device=self.device)
        if scratch_from is not None:
            if scratch_from.scratch_bytes < self.scratch_bytes:
                raise ValueError("the shared scratch buffer is too small for this context")
            self.scratch = scratch_from.scratch
        else:
            self.scratch = torch.empty(self.scratch_bytes + 1024, dtype=torch.uint8, device=self.device)
        self._ws_ptr = aligned(self.workspace)
        self._saved = ctypes.c_void_p()
        st = self.lib.skipffn_saved_create_split(ctypes.byref(self._saved), cfgp, ctypes.c_void_p(self._ws_ptr),
                                                 self.saved_bytes, ctypes.c_void_p(aligned(self.scratch)),
                                                 self.scratch.numel() - (aligned(self.scratch) - self.scratch.data_ptr()),
                                                 self.max_tokens, self.max_kept)
        if st != 0:
            raise SkipFFNError(st, "skipffn_saved_create_split")
        self._keep = []   # tensors the handle borrows between forward and backward
        self._shape = None

    def __del__(self):
        if getattr(self, "_saved", None) and self._saved.value:
            self.lib.skipffn_saved_destroy(self._saved)
            self._saved = ctypes.c_void_p()

    # ------------------------------------------------------------------ helpers
    @property
    def torch_dtype(self):
        return self._torch.bfloat16 if self.dtype == BF16 else self._torch.float32

    def _stream(self):
        return ctypes.c_void_p(self._torch.cuda.current_stream(self.device).cuda_stream)

    def _check(self, t, name, shape=None, dtype=None):
        if t is None:
            return
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous CUDA tensor")
        if dtype is not None and t.dtype != dtype:
            raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
        if shape is not None and tuple(t.shape) != tuple(shape):
            raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")

    # ------------------------------------------------------------------ C-ABI mirrors
    def tune(self, **knobs):
        """``skipffn_tune``: tile_n, streamk, stages, lose_handover (debug contexts only)."""
        for name, value in knobs.items():
            st = self.lib.skipffn_tune(self._saved, TUNABLES[name], int(value))
            if st != 0:
                raise SkipFFNError(st, f"skipffn_tune({name})")

    def plan(self, skip_mask):
        self._check(skip_mask, "skip_mask", dtype=self._torch.uint8)
        st = self.lib.skipffn_plan(self._saved, _ptr(skip_mask), skip_mask.numel(), self._stream())
        if st != 0:
            raise SkipFFNError(st, "skipffn_plan")

    def forward(self, x, skip_mask, W_gate, W_up, W_down, out=None, cu_seqlens=None, gamma=None,
                eps: float = 1e-5):
        """x: [B, S, C] or [N, C]; skip_mask: uint8 [B, S] / [N] or None (reuse the planned list).
        A context created with ``prenorm=True`` takes the gain vector ``gamma`` [C] and ``eps`` and
        calls ``skipffn_forward_prenorm``."""
        torch, dt = self._torch, self.torch_dtype
        if x.dim() == 2:
            B, S = 1, x.shape[0]
        else:
            B, S = x.shape[0], x.shape[1]
        self._check(x, "x", dtype=dt)
        if x.shape[-1] != self.C:
            raise ValueError("x has the wrong hidden size")
        self._check(W_gate, "W_gate", (self.I, self.C), dt)
        self._check(W_up, "W_up", (self.I, self.C), dt)
        self._check(W_down, "W_down", (self.C, self.I), dt)
        if skip_mask is not None:
            self._check(skip_mask, "skip_mask", dtype=torch.uint8)
            if skip_mask.numel() != B * S:
                raise ValueError("skip_mask must have one byte per token")
        if out is None:
            out = torch.empty_like(x)
        self._check(out, "out", x.shape, dt)
        cu_arr, n_seq = None, 0
        if cu_seqlens is not None:
            vals = [int(v) for v in cu_seqlens]
            n_seq = len(vals) - 1
            cu_arr = (ctypes.c_int32 * len(vals))(*vals)
        cu_p = ctypes.cast(cu_arr, ctypes.c_void_p) if cu_arr is not None else None
        if self.prenorm:
            self._check(gamma, "gamma", (self.C,), dt)
            if gamma is None:
                raise ValueError("a pre-norm context needs gamma")
            st = self.lib.skipffn_forward_prenorm(self._saved, _ptr(x), _ptr(skip_mask), B, S, cu_p, n_seq,
                                                  _ptr(gamma), ctypes.c_float(eps), _ptr(W_gate), _ptr(W_up),
                                                  _ptr(W_down), _ptr(out), self._stream())
        else:
            if gamma is not None:
                raise ValueError("gamma needs a context created with prenorm=True")
            st = self.lib.skipffn_forward(self._saved, _ptr(x), _ptr(skip_mask), B, S, cu_p,
                                          n_seq, _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(out),
                                          self._stream())
        if st != 0:
            raise SkipFFNError(st, "skipffn_forward")
        self._keep = [W_gate, W_up, W_down, gamma]
        self._shape = tuple(x.shape)
        return out

    def backward(self, dout, dx=None, dW_gate=None, dW_up=None, dW_down=None, need_dw=True, dgamma=None):
        """Returns ``(dx, dW_gate, dW_up, dW_down)``; a pre-norm context returns
        ``(dx, dW_gate, dW_up, dW_down, dgamma)``."""
        torch, dt = self._torch, self.torch_dtype
        if self._shape is None:
            raise SkipFFNError(1, "skipffn_backward (no forward has run on this context)")
        self._check(dout, "dout", self._shape, dt)
        if dx is None:
            dx = torch.empty_like(dout)
        self._check(dx, "dx", self._shape, dt)
        gdt = torch.float32 if self.grad_fp32 else dt
        if need_dw:
            if dW_gate is None:
                dW_gate = torch.empty(self.I, self.C, dtype=gdt, device=self.device)
            if dW_up is None:
                dW_up = torch.empty(self.I, self.C, dtype=gdt, device=self.device)
            if dW_down is None:
                dW_down = torch.empty(self.C, self.I, dtype=gdt, device=self.device)
        self._check(dW_gate, "dW_gate", (self.I, self.C), gdt)
        self._check(dW_up, "dW_up", (self.I, self.C), gdt)
        self._check(dW_down, "dW_down", (self.C, self.I), gdt)
        if self.prenorm:
            if dgamma is None and need_dw:
                dgamma = torch.empty(self.C, dtype=gdt, device=self.device)
            self._check(dgamma, "dgamma", (self.C,), gdt)
            st = self.lib.skipffn_backward_prenorm(_ptr(dout), self._saved, _ptr(dx), _ptr(dgamma), _ptr(dW_gate),
                                                   _ptr(dW_up), _ptr(dW_down), self._stream())
            if st != 0:
                raise SkipFFNError(st, "skipffn_backward_prenorm")
            return dx, dW_gate, dW_up, dW_down, dgamma
        st = self.lib.skipffn_backward(_ptr(dout), self._saved, _ptr(dx), _ptr(dW_gate),
                                       _ptr(dW_up), _ptr(dW_down), self._stream())
        if st != 0:
            raise SkipFFNError(st, "skipffn_backward")
        return dx, dW_gate, dW_up, dW_down

    def kv_compact(self, src, dst=None, cu_seqlens=None):
        """Skip KV-cache (``skipffn_kv_compact``, Eq. 7) with the current kept-row list.

        ``src``: contiguous CUDA tensor ``[planes..., N, heads, head_dim]`` (4-D or more) or
        ``[planes..., N, row]``; N must be the token count of the last plan / forward.  ``dst``
        (default: a new tensor shaped like ``src``) receives the kept rows in the first Nk
        positions of its token axis.  Returns ``(dst, kept_cu_seqlens)``; the second is an int32
        CUDA tensor if ``cu_seqlens`` was given, else ``None``."""
        torch = self._torch
        if not src.is_cuda or not src.is_contiguous():
            raise ValueError("src must be a contiguous CUDA tensor")
        tok_axis = src.dim() - 3 if src.dim() >= 4 else src.dim() - 2
        N = src.shape[tok_axis]
        planes = 1
        for d in src.shape[:tok_axis]:
            planes *= d
        row_bytes = src.element_size()
        for d in src.shape[tok_axis + 1:]:
            row_bytes *= d
        if dst is None:
            dst = torch.empty_like(src)
        dst_rows = dst.shape[tok_axis]
        cu_dev = new_cu = None
        n_seq = 0
        if cu_seqlens is not None:
            cu_dev = torch.as_tensor([int(v) for v in cu_seqlens], dtype=torch.int32, device=self.device)
            new_cu = torch.empty_like(cu_dev)
            n_seq = cu_dev.numel() - 1
        st = self.lib.skipffn_kv_compact(self._saved, _ptr(src), _ptr(dst), planes, row_bytes, dst_rows,
                                         _ptr(cu_dev), n_seq, _ptr(new_cu), self._stream())
        if st != 0:
            raise SkipFFNError(st, "skipffn_kv_compact")
        return dst, new_cu

    def poll(self):
        """Synchronise the stream and raise if a kernel reported a device-side problem."""
        site = ctypes.c_int32(0)
        st = self.lib.skipffn_poll(self._saved, self._stream(), ctypes.byref(site))
        if st != 0:
            raise SkipFFNError(st, f"skipffn_poll (site {site.value})")

    def kept(self):
        """(idx, nk): the ascending kept-row index list as an int32 CUDA tensor view, and Nk."""
        torch = self._torch
        idx_p, nk_p = ctypes.c_void_p(), ctypes.c_void_p()
        st = self.lib.skipffn_get_kept(self._saved, ctypes.byref(idx_p), ctypes.byref(nk_p))
        if st != 0:
            raise SkipFFNError(st, "skipffn_get_kept")
        torch.cuda.current_stream(self.device).synchronize()
        nk = int(self._view(nk_p.value, 1, torch.int32)[0].item())
        return self._view(idx_p.value, nk, torch.int32).clone(), nk

    def intermediate(self, which: int, rows: int):
        """Copy of a compacted intermediate: 0 G, 1 U, 2 H, 3 dG, 4 dU ([rows, I]); 5 Xk, 6 dOk ([rows, C])."""
        p = ctypes.c_void_p()
        st = self.lib.skipffn_get_intermediate(self._saved, which, ctypes.byref(p))
        if st != 0:
            raise SkipFFNError(st, "skipffn_get_intermediate")
        cols = self.I if which < 5 else self.C   # 5 Xk, 6 dOk, 7 normalised Xk
        return self._view(p.value, rows * cols, self.torch_dtype).view(rows, cols).clone()

    def _view(self, ptr, numel, dtype):
        """Tensor view of `numel` elements of the handle's memory starting at device address `ptr`."""
        torch = self._torch
        nbytes = numel * torch.empty(0, dtype=dtype).element_size()
        for buf in (self.workspace, self.scratch):
            off = ptr - buf.data_ptr()
            if 0 <= off and off + nbytes <= buf.numel():
                return buf[off:off + nbytes].view(dtype)
        raise ValueError("address outside the handle's buffers")

    def profile(self, step_fn, steps: int):
        """Run ``step_fn`` ``steps`` times with CUDA events around every kernel launch; returns the
        mean milliseconds per launch slot (``PROFILE_SLOTS`` names)."""
        st = self.lib.skipffn_profile_enable(self._saved, 1)
        if st != 0:
            raise SkipFFNError(st, "skipffn_profile_enable")
        acc = [0.0] * len(PROFILE_SLOTS)
        buf = (ctypes.c_float * len(PROFILE_SLOTS))()
        try:
            for _ in range(steps):
                step_fn()
                st = self.lib.skipffn_profile_read(self._saved, buf)
                if st != 0:
                    raise SkipFFNError(st, "skipffn_profile_read")
                for i in range(len(PROFILE_SLOTS)):
                    acc[i] += buf[i]
        finally:
            self.lib.skipffn_profile_enable(self._saved, 0)
        return {n: a / steps for n, a in zip(PROFILE_SLOTS, acc) if a > 0}

    def launches(self):
        return (int(self.lib.skipffn_last_launches(self._saved, 0)),
                int(self.lib.skipffn_last_launches(self._saved, 1)))
