"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "skipffn.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(skipffn_[a-z_]+)\s*\(", src)))


def test_header_symbols_are_exported_and_bound():
    from paper_2503_21817_b200 import build as b
    import paper_2503_21817_b200 as sk
    b.build()
    lib = ctypes.CDLL(b.LIB)
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(sk.EXPORTS) == names


def test_host_only_entry_points():
    import paper_2503_21817_b200 as sk
    # flop count = 2 x the paper's 3*N*C*M multiply-adds for forward, twice that again for backward
    C, I, nk = 4096, 14336, 1472
    assert sk.skipffn_flops(C, I, nk) == 18.0 * nk * C * I
    assert sk.skipffn_flops(C, I, nk) / 3 == 2 * (3 * nk * C * I)
    assert sk.skipffn_workspace_bytes(C, I, 4928) > 5 * 4928 * I * 2
    assert sk.skipffn_workspace_bytes(C, I, 4928, sk.FP32) > sk.skipffn_workspace_bytes(C, I, 4928)
    assert sk.skipffn_workspace_bytes(0, I, 10) == 0
    assert sk.skipffn_strerror(0) == "ok" and "workspace" in sk.skipffn_strerror(3)
    lib = sk.load_library()
    saved = ctypes.c_void_p()
    from paper_2503_21817_b200.binding import _cfg
    c = _cfg(C, I)
    # null workspace, misaligned workspace, too-small workspace, unsupported shape
    assert lib.skipffn_saved_create(ctypes.byref(saved), ctypes.byref(c), None, 0, 16) == 1
    assert lib.skipffn_saved_create(ctypes.byref(saved), ctypes.byref(c), ctypes.c_void_p(4096 + 8), 1 << 40, 16) == 1
    assert lib.skipffn_saved_create(ctypes.byref(saved), ctypes.byref(c), ctypes.c_void_p(4096), 1024, 16) == 3
    c2 = _cfg(100, I)
    assert lib.skipffn_saved_create(ctypes.byref(saved), ctypes.byref(c2), ctypes.c_void_p(4096), 1 << 40, 16) == 2
    # a handle over a (never dereferenced) address: host-side argument checks only
    assert lib.skipffn_saved_create(ctypes.byref(saved), ctypes.byref(c), ctypes.c_void_p(1 << 20), 1 << 40, 16) == 0
    try:
        assert lib.skipffn_backward(None, saved, None, None, None, None, None) == 1     # no forward yet
        assert lib.skipffn_forward(saved, None, None, 1, 32, None, 0, None, None, None, None, None) == 1
        assert lib.skipffn_plan(saved, None, 17, None) == 1                              # > max_tokens
        assert lib.skipffn_get_kept(saved, None, None) == 1                              # nothing planned
        assert lib.skipffn_last_launches(saved, 2) == -1
    finally:
        lib.skipffn_saved_destroy(saved)


def test_no_cpu_fallback():
    import torch
    import paper_2503_21817_b200 as sk
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        sk.SkipFFN(256, 688, 80)
