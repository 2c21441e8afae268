"""Host check of the GEMM kernels' work distribution (tiles x K-blocks over persistent workers):
every K-block of every tile is computed exactly once, hand-overs are consistent, the load is
balanced, and no wait can be circular."""
import itertools

import pytest

import paper_2503_21817_b200 as sk

CASES = [
    # (workers, tiles, k_blocks)
    (74, 96, 224),    # down projection at the 8B shape, Nk = 1472
    (74, 96, 448),    # dX
    (74, 672, 64),    # gate/up
    (74, 336, 64),    # dH
    (74, 896, 23),    # weight gradients
    (74, 32, 224),    # fewer tiles than workers
    (74, 148, 10), (74, 74, 5), (74, 75, 3), (5, 1, 11), (2, 1, 1), (3, 7, 1), (74, 1, 300),
    (74, 0, 10), (74, 10, 0), (1, 5, 7), (7, 23, 2),
]


def _all(workers, tiles, kb, split):
    return [sk.skipffn_schedule(workers, tiles, kb, split, w) for w in range(workers)]


@pytest.mark.parametrize("W,T,KB", CASES)
@pytest.mark.parametrize("split", [False, True])
def test_schedule_covers_every_k_block_once(W, T, KB, split):
    sched = _all(W, T, KB, split)
    if KB == 0:
        # empty reduction: every tile still gets one (empty) segment so that zeros are written
        tiles = sorted(s[0] for segs in sched for s in segs)
        assert tiles == list(range(T))
        return
    cover = {}
    for w, segs in enumerate(sched):
        partials = [s for s in segs if s[3]]
        assert len(partials) <= 1                      # one hand-over slot per worker
        if partials:
            assert segs[0][3] == 1                     # and it is filled first: producers never wait
        for tile, kb0, kb1, partial, src_lo in segs:
            assert 0 <= tile < T and 0 <= kb0 < kb1 <= KB
            assert (kb1 < KB) == bool(partial)
            if not split:
                assert (kb0, kb1, partial) == (0, KB, 0)
            for k in range(kb0, kb1):
                assert (tile, k) not in cover
                cover[(tile, k)] = w
    assert len(cover) == T * KB
    # hand-overs: the finisher of a tile started mid-way sums exactly the workers that hold its
    # earlier K-blocks, all of them lower-numbered (so waits form no cycle)
    for w, segs in enumerate(sched):
        for tile, kb0, kb1, partial, src_lo in segs:
            if partial or kb0 == 0:
                continue
            holders = sorted({cover[(tile, k)] for k in range(kb0)})
            nonempty = [q for q in range(src_lo, w) if sched[q]]
            with_partial_here = [q for q in nonempty if sched[q][0][3] and sched[q][0][0] == tile]
            assert holders == with_partial_here == nonempty
            assert all(q < w for q in holders)
    if split and T:
        load = [sum(s[2] - s[1] for s in segs) for segs in sched]
        assert max(load) - min(load) <= max(KB, 1) if T % W == 0 else max(load) - min(load) <= 1


def test_schedule_bad_arguments():
    lib = sk.load_library()
    assert lib.skipffn_schedule_segment(0, 1, 1, 1, 0, 0, None) == -1
    assert lib.skipffn_schedule_segment(4, 1, 1, 1, 4, 0, None) == -1
