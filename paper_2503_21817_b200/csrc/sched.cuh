// Work distribution of the persistent tensor-core GEMM kernels: which K-blocks of which tiles a
// worker (a CTA, or a CTA pair) processes, in which order.  Pure integer logic, usable on the host
// (skipffn_schedule_segment, for tests) and on the device.
#pragma once

#if defined(__CUDACC__)
#define SKIPFFN_HD __host__ __device__ inline
#else
#define SKIPFFN_HD inline
#endif

namespace skipffn {

// One unit of a worker's schedule: K-blocks [kb0, kb1) of tile `tile`.
//   partial = 1: the run stops before the tile's last K-block; the accumulator goes to this
//                worker's slot.
//   partial = 0: the run ends the tile; if kb0 > 0 the slots of workers src_lo .. w-1 (those with a
//                non-empty run) hold the rest of the tile and are added before the epilogue.
struct Seg { int tile, kb0, kb1, partial, src_lo; };

struct Sched {
    int w, W, T, KB, n_dp, sk_tile0, t_first, has_partial, n_fin;
    long long usk, u0, u1;
    SKIPFFN_HD long long bound(int p) const { return (long long)p * usk / W; }
    SKIPFFN_HD void init(int w_, int W_, int T_, int KB_, int streamk)
    {
        w = w_; W = W_; T = T_; KB = KB_;
        const int full = T / W, rem = T % W;
        int dp_waves;
        if (!streamk || KB == 0 || rem == 0) { dp_waves = (T + W - 1) / W; usk = 0; }
        else { dp_waves = full > 0 ? full - 1 : 0; usk = (long long)(T - dp_waves * W) * KB; }
        sk_tile0 = dp_waves * W;
        n_dp = usk ? dp_waves : (w < T ? (T - w + W - 1) / W : 0);
        u0 = bound(w); u1 = bound(w + 1);
        t_first = 0; has_partial = 0; n_fin = 0;
        if (u1 > u0) {
            t_first = (int)(u0 / KB);
            const int t_last = (int)((u1 - 1) / KB);
            has_partial = (u1 % KB) != 0;
            n_fin = t_last - t_first + 1 - has_partial;
        }
    }
    SKIPFFN_HD int count() const { return has_partial + n_dp + n_fin; }
    SKIPFFN_HD Seg get(int i) const
    {
        Seg s;
        s.partial = 0; s.src_lo = w;
        if (has_partial) {
            if (i == 0) {
                const int t = (int)((u1 - 1) / KB);
                const long long ts = (long long)t * KB;
                s.tile = sk_tile0 + t;
                s.kb0 = (int)((u0 > ts ? u0 : ts) - ts);
                s.kb1 = (int)(u1 - ts);
                s.partial = 1;
                return s;
            }
            --i;
        }
        if (i < n_dp) { s.tile = i * W + w; s.kb0 = 0; s.kb1 = KB; return s; }
        i -= n_dp;
        const int t = t_first + i;
        const long long ts = (long long)t * KB;
        s.tile = sk_tile0 + t;
        s.kb0 = (int)((u0 > ts ? u0 : ts) - ts);
        s.kb1 = KB;
        if (s.kb0 > 0) {
            int p = w - 1;
            while (p > 0 && bound(p) > ts) --p;
            s.src_lo = p;
        }
        return s;
    }
};

// Whether cutting the last waves along K pays: the idle time it removes, (W - T mod W) / W of a
// tile's main loop, must be worth `min_saving` K-blocks per worker (0 = never cut).
SKIPFFN_HD bool split_pays(int T, int W, int KB, int min_saving)
{
    const int rem = T % W;
    return min_saving > 0 && rem != 0 && (long long)(W - rem) * KB >= (long long)min_saving * W;
}

// The schedule of one worker of a launch, with the worker groups of the down / dX launches.
// Token problems order their tiles with the token-tile index fastest: tile = panel * n_tok + column,
// a panel being all token tiles of one block of weight rows.  With groups (gw = n_tok > 1) the
// W workers form W / gw groups of gw; a group takes the place of a worker and a panel the place of
// a tile in `Sched`, and member `col` of a group works on token tile `col` of whatever panel and
// K range its group has, so the members read the same weight bytes at the same time.  Workers
// beyond the last whole group get nothing.  Hand-overs go from member `col` of one group to member
// `col` of the next: schedule worker q of `src_lo .. w-1` is real worker slot_worker(q).
struct Plan {
    Sched s;
    int gw, col;
    // group_mode: 0 never, 1 when all tiles would be cut anyway (T < 2W), K has at least 32 blocks
    // and groups cost under 6 % more K-blocks per worker, 2 always (n_tok between 2 and 16, <= W)
    SKIPFFN_HD void init(int worker, int W, int panels, int n_tok, int KB, int min_saving, int group_mode)
    {
        const int T = panels * n_tok;
        gw = 1;
        if (group_mode && min_saving > 0 && n_tok >= 2 && n_tok <= 16 && n_tok <= W && KB > 0) {
            const int ng = W / n_tok;
            const long long plain = ((long long)T * KB + W - 1) / W;
            const long long grouped = ((long long)panels * KB + ng - 1) / ng;
            if (group_mode == 2 || (T < 2 * W && KB >= 32 && grouped * 100 <= plain * 106)) gw = n_tok;
        }
        col = gw > 1 ? worker % gw : 0;
        if (gw > 1) {
            const int ng = W / gw, sw = worker / gw;
            if (sw < ng) s.init(sw, ng, panels, KB, split_pays(panels, ng, KB, min_saving));
            else s.init(0, 1, 0, KB, 0);   // spare worker: nothing to do
        } else {
            s.init(worker, W, T, KB, split_pays(T, W, KB, min_saving));
        }
    }
    SKIPFFN_HD int count() const { return s.count(); }
    SKIPFFN_HD Seg get(int i) const
    {
        Seg sg = s.get(i);
        if (gw > 1) sg.tile = sg.tile * gw + col;
        return sg;
    }
    // real worker behind schedule worker q (a hand-over source of this worker)
    SKIPFFN_HD int slot_worker(int q) const { return gw > 1 ? q * gw + col : q; }
    SKIPFFN_HD bool had_run(int q) const { return s.bound(q + 1) != s.bound(q); }
    SKIPFFN_HD int self() const { return s.w; }
};

}  // namespace skipffn
