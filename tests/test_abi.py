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


def test_memory_modes_sizes_and_host_side_checks():
    # host-only: saved / scratch sizes of the memory modes, handle creation over two buffers, knobs
    import paper_2503_21817_b200 as sk
    from paper_2503_21817_b200.binding import _cfg
    lib = sk.load_library()
    C, I, N, nk = 4096, 14336, 4928, 1472
    plain, rec, dbg = _cfg(C, I), _cfg(C, I, recompute=True), _cfg(C, I, debug=True)
    by = lambda fn, c, mk: int(fn(ctypes.byref(c), N, mk))
    sv, sc, ws = lib.skipffn_saved_bytes, lib.skipffn_scratch_bytes, lib.skipffn_workspace_bytes_kept
    # one buffer = saved + scratch; the classic size is the kept-sized one with max_kept = max_tokens
    assert by(ws, plain, N) == by(sv, plain, N) + by(sc, plain, N) == sk.skipffn_workspace_bytes(C, I, N)
    # compacted arrays scale with the kept bound: G, U, H (saved) and dG, dU, dOk (scratch)
    assert by(sv, plain, nk) < 0.35 * by(sv, plain, N) and by(sc, plain, nk) < 0.4 * by(sc, plain, N)
    assert by(sv, plain, nk) > 3 * 1536 * I * 2
    # recompute: G, U, H move from saved to scratch; what is saved is the kept rows of x and two index arrays
    assert by(sv, rec, nk) < 1536 * C * 2 + 2 * 5120 * 4 + 16384
    assert by(sv, rec, nk) + by(sc, rec, nk) == by(sv, plain, nk) + by(sc, plain, nk)
    # debug handles pay for their guard bands; invalid bounds give size 0
    assert by(sv, dbg, nk) > by(sv, plain, nk)
    assert by(sv, plain, N + 1) == 0 and int(sv(ctypes.byref(plain), -1, 0)) == 0
    saved = ctypes.c_void_p()
    a, b = ctypes.c_void_p(1 << 20), ctypes.c_void_p(1 << 30)
    cr = lib.skipffn_saved_create_split
    assert cr(ctypes.byref(saved), ctypes.byref(rec), a, by(sv, rec, nk) - 1, b, 1 << 40, N, nk) == 3    # saved too small
    assert cr(ctypes.byref(saved), ctypes.byref(rec), a, 1 << 40, b, by(sc, rec, nk) - 1, N, nk) == 3    # scratch too small
    assert cr(ctypes.byref(saved), ctypes.byref(rec), a, 1 << 40, None, 1 << 40, N, nk) == 1             # no scratch
    assert cr(ctypes.byref(saved), ctypes.byref(rec), a, 1 << 40, b, 1 << 40, N, N + 1) == 1             # bound > tokens
    assert cr(ctypes.byref(saved), ctypes.byref(rec), a, by(sv, rec, nk), b, by(sc, rec, nk), N, nk) == 0
    try:
        assert lib.skipffn_tune(saved, 0, 128) == 0 and lib.skipffn_tune(saved, 99, 1) == 1
        assert lib.skipffn_tune(saved, sk.binding.TUNABLES["lose_handover"], 1) == 1                      # debug handles only
    finally:
        lib.skipffn_saved_destroy(saved)
    assert lib.skipffn_token_merge_poll(None, 10, 64, 4, 0, None, None) == 1


def test_no_cpu_fallback():
    import torch
    import paper_2503_21817_b200 as sk
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        sk.SkipFFN(256, 688, 80)
