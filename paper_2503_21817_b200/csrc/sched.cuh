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

}  // namespace skipffn
