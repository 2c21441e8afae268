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


PLAN_CASES = [
    # (workers, panels, token tiles, k_blocks): down / dX of the benchmark shapes and edge cases
    (74, 16, 6, 224), (74, 16, 6, 448), (74, 16, 4, 224), (74, 16, 2, 448), (74, 20, 6, 216), (74, 16, 9, 224),
    (74, 16, 11, 224), (74, 32, 3, 4), (74, 2, 2, 64), (74, 1, 5, 300), (74, 16, 1, 224), (7, 3, 2, 5),
    (6, 5, 3, 40), (16, 4, 16, 33), (5, 2, 6, 64), (74, 0, 6, 10), (74, 16, 6, 0),
]


@pytest.mark.parametrize("W,P,NT,KB", PLAN_CASES)
@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("min_saving", [0, 1, 40])
def test_plan_with_worker_groups_covers_every_k_block_once(W, P, NT, KB, mode, min_saving):
    plan = [sk.skipffn_schedule_plan(W, P, NT, KB, min_saving, mode, w) for w in range(W)]
    T = P * NT
    if KB == 0:
        assert sorted(s[0] for segs in plan for s in segs) == list(range(T))
        return
    strides = {s[5] for segs in plan for s in segs}
    assert len(strides) <= 1
    gw = strides.pop() if strides else 1
    grouped = gw > 1
    if grouped:
        assert gw == NT and mode > 0 and min_saving > 0 and 2 <= NT <= 16 and NT <= W
    if mode == 2 and min_saving > 0 and 2 <= NT <= min(16, W) and T:
        assert grouped
    if mode == 0 or min_saving == 0:
        assert not grouped
    cover = {}
    for w, segs in enumerate(plan):
        assert sum(1 for s in segs if s[3]) <= 1 and (not any(s[3] for s in segs) or segs[0][3] == 1)
        if grouped and w >= (W // gw) * gw:
            assert segs == []                       # workers beyond the last whole group
        for tile, kb0, kb1, partial, src, stride in segs:
            assert 0 <= tile < T and 0 <= kb0 < kb1 <= KB and (kb1 < KB) == bool(partial)
            if grouped:
                assert tile % NT == w % gw          # member j of a group works on token tile j
            for k in range(kb0, kb1):
                assert (tile, k) not in cover
                cover[(tile, k)] = w
    assert len(cover) == T * KB
    # members of a group hold the same panel and K range at the same position of their schedules
    if grouped:
        for g in range(W // gw):
            shapes = {tuple((t // NT, a, b, pt) for t, a, b, pt, _, _ in plan[g * gw + j]) for j in range(gw)}
            assert len(shapes) == 1
    # hand-overs: a finisher that starts mid-way adds exactly the workers that hold the tile's earlier
    # K-blocks; they are src, src + stride, ... below it, each with its partial segment first
    for w, segs in enumerate(plan):
        for tile, kb0, kb1, partial, src, stride in segs:
            if partial or kb0 == 0:
                continue
            holders = sorted({cover[(tile, k)] for k in range(kb0)})
            cands = [q for q in range(src, w, stride) if plan[q]]
            assert (w - src) % stride == 0
            assert holders == cands and all(q < w for q in holders)
            assert all(plan[q][0][3] == 1 and plan[q][0][0] == tile for q in holders)
    # balance: all working workers carry the same number of K-blocks to within one tile
    load = [sum(s[2] - s[1] for s in segs) for segs in plan if segs]
    if load and min_saving == 1:
        assert max(load) - min(load) <= KB


def test_plan_picks_groups_for_the_benchmark_shapes_only_when_cheap():
    # cfg2 down / dX: 16 panels x 6 token tiles on 74 SM pairs -> 12 groups of 6 (+2.8 % K-blocks)
    assert {s[5] for w in range(74) for s in sk.skipffn_schedule_plan(74, 16, 6, 224, 40, 1, w)} == {6}
    # 11 token tiles (r = 0.5) would idle 8 of 74 pairs: not chosen; the dense case has T >= 2W
    assert {s[5] for w in range(74) for s in sk.skipffn_schedule_plan(74, 16, 11, 224, 40, 1, w)} == {1}
    assert {s[5] for w in range(74) for s in sk.skipffn_schedule_plan(74, 16, 20, 224, 40, 1, w)} == {1}
    # short reductions stay with one run per worker
    assert {s[5] for w in range(74) for s in sk.skipffn_schedule_plan(74, 16, 6, 16, 40, 1, w)} == {1}
    lib = sk.load_library()
    assert lib.skipffn_schedule_plan_segment(0, 1, 1, 1, 1, 1, 0, 0, None) == -1
    assert lib.skipffn_schedule_plan_segment(4, 1, 0, 1, 1, 1, 0, 0, None) == -1
