#!/usr/bin/env python
"""Skip-FFN forward+backward benchmark on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg2|cfg3|cfg4|sweep] [--skip-ratio r] [--shape llama3-8b|vicuna-13b]

One step = one pass of the whole hot path (mask compaction, row routing, gate/up GEMM + SiLU*mul,
down GEMM + residual scatter, and the backward GEMMs dH, dW_down, dW_gate, dW_up, dX) over one
batch of seeded synthetic input.  Default workload: the LLaMA3-8B-shaped layer, 8 x (576 visual +
40 text) tokens, 75 % of the visual tokens skipped, bf16 with fp32 accumulation.

Prints ONE JSON line (rank 0).  `value` is kept tokens per second over all ranks with inputs
resident in HBM; `e2e` is the same metric with the step's inputs copied from pinned host memory
and its results copied back inside the timed region; `roofline` describes the kernel with the
largest share of the step; `cpu_baseline` is the fp64 CPU oracle timed on a bounded sample.
With N > 1 (torchrun) every rank runs an independent replica (no collective on the data path).

At N = 1 the same line carries, measured after and outside the headline timed region:
  sustained  the same step repeated for at least 3 s: ms per step, TFLOP/s against the sustained
             library peak, SM clock median and throttle reasons of that region, per-kernel times
  cfg3/cfg4  the high-resolution and the packed variable-length workloads
  sweep      skip ratios {0, .25, .5, .75, .9, 1} at both shapes against the in-library dense
             comparator on the same inputs
  host_us_per_step  host time of the eight launches of one step (no synchronisation)
  step_times median and best of 50 steps timed one by one, and a step with a cold L2
  graph_replay  the same step replayed from a captured CUDA graph
  seeds      the same workload drawn from two more seeds
(`--no-extras` leaves them out.)
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "skipffn_fwd_bwd_kept_tokens_per_s"
UNIT = "kept tokens/s"
KERNEL_NAMES = ["compact", "route_x", "gateup", "down", "route_dout", "dh", "dw_down", "dw_gate",
                "dw_up", "dx"]
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of each GEMM kernel at the
# default workload, from the ncu captures summarised under profiles/; None until captured.
NCU_TRAFFIC_BYTES = {"gateup": 416.5e6, "down": 224.8e6, "dh": 276.2e6, "dw_down": 501.2e6,
                     "dx": 443.2e6, "route_x": 42.1e6, "route_dout": 41.8e6}
# sha256 prefix of csrc/umma.cu when those counters were taken; once the kernel source differs the
# counters no longer describe it and `traffic` is reported as null
NCU_TRAFFIC_SOURCE_SHA = "ebcdf372e46ce66e"


def ncu_traffic(kernel):
    import hashlib
    src = os.path.join(ROOT, "paper_2503_21817_b200", "csrc", "umma.cu")
    try:
        cur = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    return NCU_TRAFFIC_BYTES.get(kernel) if cur == NCU_TRAFFIC_SOURCE_SHA else None


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def make_workload(args, rank):
    C, I = wl.SWEEP_SHAPES[args.shape]
    seed = args.seed + rank
    if args.workload == "cfg2":
        return wl.config2(seed=seed, skip_ratio=args.skip_ratio, C=C, I=I)
    if args.workload == "cfg3":
        return wl.config3(seed=seed, C=C, I=I)
    if args.workload == "cfg4":
        return wl.config4(seed=seed, C=C, I=I)
    raise ValueError(args.workload)


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        rows = [r for t, r in self.rows if t0 - 0.05 <= t <= t1 + 0.15] or [r for _, r in self.rows]
        for r in rows:
            f = [c.strip() for c in r.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------ oracle legs
def oracle_sample_rate(w, n_tokens):
    """kept tokens / s of the fp64 CPU oracle (forward + backward, as it stands) on the first
    `n_tokens` tokens of the workload."""
    import oracle
    m = w.skip_mask[:n_tokens]
    x64, wg, wu, wd, do = (a.astype(np.float64) for a in (w.x[:n_tokens], w.W_gate, w.W_up, w.W_down,
                                                          w.dout[:n_tokens]))
    t = time.perf_counter()
    oracle.forward(x64, m, wg, wu, wd)
    oracle.backward(x64, m, wg, wu, wd, do)
    dt = time.perf_counter() - t
    kept = int((m == 0).sum())
    return kept / dt, kept, dt, oracle.n_threads()


def run_reference(args):
    """The reference arm: the CPU oracle, timed step by step on a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = make_workload(args, 0)
    budget_s = 150.0
    per_tok = 1.1    # seconds per kept token of this oracle at the 8B shape on ~8 cores (rough)
    n_tok = int(max(1, min(w.N, budget_s / ((args.steps + args.warmup) * per_tok))))
    # text tokens lead every sequence and are always kept, so the first tokens are all FFN work
    rates, kept, cores = [], 0, 0
    for _ in range(args.warmup):
        oracle_sample_rate(w, n_tok)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        r, kept, _, cores = oracle_sample_rate(w, n_tok)
        rates.append(r)
    total = time.perf_counter() - t0
    value = kept * args.steps / total
    sample = f"first {n_tok} tokens of sequence 0 ({kept} kept) per step, full fp64 forward+backward"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(args, w),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(args, w):
    return {"workload": f"{w.name} {args.shape}: C={w.C} I={w.I} N={w.N} tokens "
                        f"({w.meta.get('n_visual', '?')} visual + text per sequence), kept={w.n_kept}",
            "C": w.C, "I": w.I, "tokens": w.N, "kept_tokens": w.n_kept, "skip_ratio": args.skip_ratio,
            "variant": "pre-norm (RMSNorm on the FFN input)" if args.prenorm else "as Eq. 4 (no normalisation)",
            "l2_policy": "inputs larger than L2 (weights 3 x %.0f MB re-read every step)" % (w.C * w.I * 2 / 1e6),
            "parallelism": "replicas only" if args.gpus > 1 else "single GPU"}


# ------------------------------------------------------------------------------ rank aggregation
def max_over_ranks(ms, device=None):
    """Slowest rank's time: replicas finish when the last one does."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(units, device=None):
    """Units (kept tokens) processed per step by the whole job."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return int(units)
    t = torch.tensor([units], device=device, dtype=torch.int64)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())


def job_throughput(units_local, ms_local, steps, device=None):
    """(kept tokens/s of the whole job, ms per step): all ranks' units over the slowest rank's time."""
    ms = max_over_ranks(ms_local, device)
    units = sum_over_ranks(units_local, device)
    return units / (ms / steps * 1e-3), ms / steps


# ------------------------------------------------------------------------------ our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2503_21817_b200 as sk

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    w = make_workload(args, rank)
    N, C, I, nk = w.N, w.C, w.I, w.n_kept

    def h_bf16(a):
        return torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).view(torch.bfloat16).reshape(a.shape)

    # pinned host copies of the step's inputs and results (for the end-to-end leg)
    hx, hdout = h_bf16(w.x).pin_memory(), h_bf16(w.dout).pin_memory()
    hmask = torch.from_numpy(w.skip_mask).pin_memory()
    hout, hdx = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory()
    x, dout, mask = hx.to(dev), hdout.to(dev), hmask.to(dev)
    Wg, Wu, Wd = h_bf16(w.W_gate).to(dev), h_bf16(w.W_up).to(dev), h_bf16(w.W_down).to(dev)
    out, dx = torch.empty_like(x), torch.empty_like(x)
    dWg, dWu, dWd = torch.empty_like(Wg), torch.empty_like(Wu), torch.empty_like(Wd)
    ctx = sk.SkipFFN(C, I, N, dtype=sk.BF16, dense=args.dense, prenorm=args.prenorm, recompute=args.recompute,
                     max_kept=None if (args.dense or not args.kept_sized) else nk)
    if args.tune:       # launch knobs of the handle (skipffn_tune), e.g. --tune one_box=0,streamk=0
        ctx.tune(**{k: int(v) for k, v in (kv.split("=") for kv in args.tune.split(","))})
    if args.dense:
        nk = N
    fwd_kw, bwd_kw = {}, {}
    if args.prenorm:     # pre-norm variant: RMSNorm gain near 1, its gradient as one more output
        gamma = h_bf16(1.0 + 0.1 * wl.normal(args.seed, 9, C)).to(dev)
        fwd_kw = dict(gamma=gamma, eps=1e-5)
        bwd_kw = dict(dgamma=torch.empty_like(gamma))

    def step():
        ctx.forward(x, mask, Wg, Wu, Wd, out=out, **fwd_kw)
        ctx.backward(dout, dx=dx, dW_gate=dWg, dW_up=dWu, dW_down=dWd, **bwd_kw)

    # End-to-end leg: every step copies x, skip_mask and dout from pinned host memory and copies
    # out and dx back.  Two sets of device buffers and three streams (host->device, compute,
    # device->host) let step i+1's input copy and step i-1's result copy run under step i's
    # kernels; events order each buffer's copy -> compute -> copy-back -> reuse.
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    s_comp = torch.cuda.current_stream(dev)
    dbuf = [dict(x=torch.empty_like(x), mask=torch.empty_like(mask), dout=torch.empty_like(dout),
                 out=torch.empty_like(x), dx=torch.empty_like(x),
                 ready_in=torch.cuda.Event(), done=torch.cuda.Event(), copied_out=torch.cuda.Event())
            for _ in range(2)]
    e2e_count = [0]

    def step_e2e():
        b = dbuf[e2e_count[0] % 2]
        first_use = e2e_count[0] < 2
        e2e_count[0] += 1
        with torch.cuda.stream(s_in):
            if not first_use:
                s_in.wait_event(b["done"])          # the step that last read these inputs has finished
            b["x"].copy_(hx, non_blocking=True)
            b["mask"].copy_(hmask, non_blocking=True)
            b["dout"].copy_(hdout, non_blocking=True)
            b["ready_in"].record(s_in)
        s_comp.wait_event(b["ready_in"])
        if not first_use:
            s_comp.wait_event(b["copied_out"])      # its previous results are on the host
        ctx.forward(b["x"], b["mask"], Wg, Wu, Wd, out=b["out"], **fwd_kw)
        ctx.backward(b["dout"], dx=b["dx"], dW_gate=dWg, dW_up=dWu, dW_down=dWd, **bwd_kw)
        b["done"].record(s_comp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(b["done"])
            hout.copy_(b["out"], non_blocking=True)
            hdx.copy_(b["dx"], non_blocking=True)
            b["copied_out"].record(s_out)

    def timed_e2e(steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(s_in)                              # nothing is in flight: the first copy starts here
        for _ in range(steps):
            step_e2e()
        s_out.wait_stream(s_comp)
        e1.record(s_out)                             # after the last result has reached the host
        barrier()
        return e0.elapsed_time(e1)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0 = time.time()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        t1 = time.time()
        return e0.elapsed_time(e1), t0, t1

    if args.profile_only:      # short launch sequence for ncu: W + K steps, nothing else
        for _ in range(args.warmup + args.steps):
            step()
        ctx.poll()
        print(json.dumps({"profile_only": True, "launches_per_step": sum(ctx.launches())}), flush=True)
        return
    for _ in range(max(args.warmup, 3)):
        step()
    ctx.poll()
    sampler = ClockSampler(local) if rank == 0 else None
    ms, t0, t1 = timed(step, args.steps)
    clocks = sampler.stop(t0, t1) if sampler else None
    ctx.poll()
    launches_per_step = sum(ctx.launches())

    for _ in range(3):
        step_e2e()
    ms_e2e = timed_e2e(args.steps)

    # per-kernel durations: the same steps again with CUDA events recorded around every launch
    prof = ctx.profile(step, args.steps) if hasattr(ctx, "profile") else None
    ctx.poll()

    # whole-job numbers: every rank's kept tokens over the slowest rank's time
    value, ms_step = job_throughput(nk, ms, args.steps, dev)
    value_e2e, ms_step_e2e = job_throughput(nk, ms_e2e, args.steps, dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    tflops = value * sk.skipffn_flops(C, I, 1) / 1e12
    unit_flops = 2.0 * nk * C * I     # one GEMM "unit" of the path: 2 * Nk * C * I
    kernel_units = {"gateup": 2, "down": 1, "dh": 1, "dw_down": 1, "dw_gate": 1, "dw_up": 1, "dx": 2}
    kernels, roofline = {}, None
    if prof and "dw_gate" not in prof and "dw_up" not in prof:
        kernel_units["dw_down"] = 3     # one grouped launch computes all three weight gradients
    if prof:
        total = sum(prof.values())
        for name, kms in prof.items():
            ent = {"ms": kms, "share": kms / total if total else None}
            if name in ("route_x", "route_dout"):
                # every row is read once and written once (kept rows compacted, skipped rows copied)
                ent["gbs"] = (2.0 * N * C * 2 + 4.0 * N) / (kms * 1e-3) / 1e9
                ent["frac_of_measured_hbm"] = ent["gbs"] / pk["hbm_gbs"]
            if name == "compact":
                ent["gbs"] = (N + 4.0 * N + 4.0 * nk) / (kms * 1e-3) / 1e9      # mask in; pos, idx out
                ent["bound"] = "latency (one CTA)"
            if name in kernel_units:
                ent["tflops"] = kernel_units[name] * unit_flops / (kms * 1e-3) / 1e12
                ent["frac_of_measured_bf16_peak"] = ent["tflops"] / pk["bf16_tflops"]
            kernels[name] = ent
        gemms = {k: v for k, v in kernels.items() if k in kernel_units}
        top = max(gemms, key=lambda k: gemms[k]["ms"])
        roofline = {"kernel": f"k_umma_gemm[{top}]", "bound": "tensor", "achieved": gemms[top]["tflops"],
                    "peak": pk["bf16_tflops"], "unit": "TFLOP/s", "frac": gemms[top]["tflops"] / pk["bf16_tflops"],
                    "peak_source": pk["source"] + " (burst cuBLAS bf16)",
                    "traffic": ncu_traffic(top),
                    "all_gemm_kernels": {"tflops": sum(kernel_units[k] for k in gemms) * unit_flops /
                                         (sum(v["ms"] for v in gemms.values()) * 1e-3) / 1e12}}
        roofline["all_gemm_kernels"]["frac"] = roofline["all_gemm_kernels"]["tflops"] / pk["bf16_tflops"]

    extras = {}
    if world == 1 and not args.no_extras:
        # host time of one step's launches: enqueue without synchronising
        torch.cuda.synchronize()
        th = time.perf_counter()
        for _ in range(40):
            step()
        extras["host_us_per_step"] = (time.perf_counter() - th) / 40 * 1e6
        torch.cuda.synchronize()
        # 50 steps timed one by one (events around each step): median and best; then one step with a
        # cold L2 (a 512 MB buffer is written first)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(50)]
        for a, b in evs:
            a.record()
            step()
            b.record()
        torch.cuda.synchronize()
        each = sorted(a.elapsed_time(b) for a, b in evs)
        flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
        cold = []
        for _ in range(3):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            step()
            b.record()
            torch.cuda.synchronize()
            cold.append(a.elapsed_time(b))
        del flush
        extras["step_times"] = {"steps": len(each), "median_ms": each[len(each) // 2], "best_ms": each[0],
                                "cold_l2_ms": sorted(cold)[1],
                                "note": "each step timed alone; cold_l2: median of 3 steps that follow a 512 MB write"}
        # the same step replayed from a CUDA graph (one host call per step instead of eight launches)
        try:
            cap = torch.cuda.Stream(dev)
            cap.wait_stream(torch.cuda.current_stream(dev))
            with torch.cuda.stream(cap):
                step()
            torch.cuda.current_stream(dev).wait_stream(cap)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            for _ in range(3):
                graph.replay()
            ms_g, _, _ = timed(graph.replay, args.steps)
            torch.cuda.synchronize()
            th = time.perf_counter()
            for _ in range(40):
                graph.replay()
            host_g = (time.perf_counter() - th) / 40 * 1e6
            torch.cuda.synchronize()
            extras["graph_replay"] = {"ms_per_step": ms_g / args.steps, "host_us_per_step": host_g}
            del graph
        except Exception as exc:      # capture is a convenience of the harness, not part of the metric
            extras["graph_replay"] = {"error": str(exc)[:200]}
        # other seeds: new activations, gradients and mask positions (same kept count), same weights
        seeds = {}
        for sd in (1, 2):
            ws = wl.config2(seed=args.seed + sd, skip_ratio=args.skip_ratio, C=C, I=I,
                            weights=(w.W_gate, w.W_up, w.W_down)) if args.workload == "cfg2" else None
            if ws is None:
                break
            xs_, ds_, ms_ = h_bf16(ws.x).to(dev), h_bf16(ws.dout).to(dev), torch.from_numpy(ws.skip_mask).to(dev)

            def step_seed():
                ctx.forward(xs_, ms_, Wg, Wu, Wd, out=out)
                ctx.backward(ds_, dx=dx, dW_gate=dWg, dW_up=dWu, dW_down=dWd)
            for _ in range(3):
                step_seed()
            t_sd, _, _ = timed(step_seed, args.steps)
            seeds[str(args.seed + sd)] = {"ms_per_step": t_sd / args.steps, "kept_tokens": ws.n_kept}
            del xs_, ds_, ms_
        if seeds:
            extras["seeds"] = seeds
        ctx.poll()
        # sustained: the same step for at least 3 s, clocks sampled over that region
        n_sus = max(args.steps, int(np.ceil(args.sustained_seconds * 1e3 / ms_step)))
        sampler = ClockSampler(local)
        ms_sus, t0, t1 = timed(step, n_sus)
        clocks_sus = sampler.stop(t0, t1)
        prof_sus = ctx.profile(step, 20)          # straight after, while the part is still power-capped
        ctx.poll()
        ms_s = ms_sus / n_sus
        tf_s = sk.skipffn_flops(C, I, nk) / (ms_s * 1e-3) / 1e12
        sus_kernels = {}
        for name, kms in prof_sus.items():
            ent = {"ms": kms}
            if name in kernel_units:
                ent["tflops"] = kernel_units[name] * unit_flops / (kms * 1e-3) / 1e12
                if pk["bf16_tflops_sustained"]:
                    ent["frac_of_sustained_bf16_peak"] = ent["tflops"] / pk["bf16_tflops_sustained"]
            sus_kernels[name] = ent
        extras["sustained"] = {
            "steps": n_sus, "seconds": ms_sus * 1e-3, "ms_per_step": ms_s, "kept_tokens_per_s": nk / (ms_s * 1e-3),
            "tflops": tf_s, "frac_of_sustained_bf16_peak": tf_s / pk["bf16_tflops_sustained"] if pk["bf16_tflops_sustained"] else None,
            "frac_of_burst_bf16_peak": tf_s / pk["bf16_tflops"], "clocks": clocks_sus,
            "mcycles_per_step": ms_s * clocks_sus["sm_mhz"] * 1e-3 if clocks_sus.get("sm_mhz") else None,
            "kernels": sus_kernels}
        # memory modes: bytes a handle holds between forward and backward (saved) and inside a call
        # (scratch, shareable between layers), and the time of the recomputing mode
        def sizes(**kw):
            c = sk.SkipFFN(C, I, N, **kw)
            return {"saved_bytes": c.saved_bytes, "scratch_bytes": c.scratch_bytes}
        rc = sk.SkipFFN(C, I, N, recompute=True, max_kept=nk)

        def step_rc():
            rc.forward(x, mask, Wg, Wu, Wd, out=out)
            rc.backward(dout, dx=dx, dW_gate=dWg, dW_up=dWu, dW_down=dWd)
        for _ in range(3):
            step_rc()
        ms_def, _, _ = timed(step, args.steps)          # the default mode again, same thermal state
        ms_rc, _, _ = timed(step_rc, args.steps)
        rc.poll()
        extras["memory_modes"] = {
            "token_sized": sizes(), "kept_sized": sizes(max_kept=nk),
            "kept_sized_recompute": {"saved_bytes": rc.saved_bytes, "scratch_bytes": rc.scratch_bytes,
                                     "ms_per_step": ms_rc / args.steps, "time_vs_default": ms_rc / ms_def}}
        del rc
        # the other single-GPU workloads, same weights
        dbuf.clear()
        weights_host = (w.W_gate, w.W_up, w.W_down)
        for name in ("cfg3", "cfg4"):
            if args.workload == name or args.shape != "llama3-8b":
                continue
            wo = (wl.config3 if name == "cfg3" else wl.config4)(seed=args.seed, C=C, I=I, weights=weights_host)
            extras[name] = time_workload(sk, wo, (Wg, Wu, Wd), (dWg, dWu, dWd), args.steps, max(args.warmup, 3), pk)
        extras["sweep"] = sweep_table(sk, args, pk, {args.shape: (Wg, Wu, Wd)})

    cpu = None
    if not args.no_cpu_baseline and world == 1:    # the oracle is timed at N = 1 only
        rate, kept, dt, cores = oracle_sample_rate(w, args.cpu_sample_tokens)
        cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"first {args.cpu_sample_tokens} tokens of sequence 0 ({kept} kept), full fp64 "
                         f"forward+backward, {dt:.1f} s"}

    h2d = hx.numel() * 2 + hdout.numel() * 2 + hmask.numel()
    d2h = hout.numel() * 2 + hdx.numel() * 2
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(args, w), "tflops": tflops,
            "frac_of_measured_bf16_peak": tflops / world / pk["bf16_tflops"],
            "frac_of_nominal_bf16_peak": tflops / world / 2250.0,
            "timed_region": "burst: %d steps, %.0f ms; see `sustained` for the power-capped figure" % (args.steps, ms_step * args.steps),
            "e2e": {"value": value_e2e, "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_step_e2e,
                    "pipeline": "3 streams (H2D, compute, D2H), double-buffered device inputs and results"},
            "gpu_launches": launches_per_step * args.steps, "clocks": clocks, "roofline": roofline,
            "kernels": kernels, "cpu_baseline": cpu}
    line.update(extras)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------ other workloads
def _h_bf16(a):
    import torch
    return torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).view(torch.bfloat16).reshape(a.shape)


def time_ctx(ctx, x, mask, dout, W, bufs, steps, warmup):
    """ms per forward+backward step of `ctx` on resident inputs (CUDA events, after warm-up)."""
    import torch
    out, dx, dWg, dWu, dWd = bufs

    def step():
        ctx.forward(x, mask, W[0], W[1], W[2], out=out)
        ctx.backward(dout, dx=dx, dW_gate=dWg, dW_up=dWu, dW_down=dWd)
    for _ in range(max(warmup, 3)):
        step()
    ctx.poll()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ctx.poll()
    return e0.elapsed_time(e1) / steps


def time_workload(sk, w, W, dW, steps, warmup, pk):
    """One more workload on weights already on the device: ms per step, kept tokens/s, TFLOP/s."""
    import torch
    x, dout, mask = _h_bf16(w.x).cuda(), _h_bf16(w.dout).cuda(), torch.from_numpy(w.skip_mask).cuda()
    ctx = sk.SkipFFN(w.C, w.I, w.N)
    ms = time_ctx(ctx, x, mask, dout, W, [torch.empty_like(x), torch.empty_like(x)] + list(dW), steps, warmup)
    tf = sk.skipffn_flops(w.C, w.I, w.n_kept) / (ms * 1e-3) / 1e12
    return {"workload": w.name, "tokens": w.N, "kept_tokens": w.n_kept, "steps": steps, "ms_per_step": ms,
            "kept_tokens_per_s": w.n_kept / (ms * 1e-3), "tflops": tf,
            "frac_of_measured_bf16_peak": tf / pk["bf16_tflops"]}


# ------------------------------------------------------------------------------ skip-ratio sweep
def sweep_table(sk, args, pk, resident=None):
    """Skip-ratio sweep: visual skip fraction in {0, .25, .5, .75, .9, 1} at the LLaMA3-8B and
    Vicuna-13B shapes (8 x 616 tokens), plus the in-library dense comparator on the same inputs.
    Per point: kept tokens/s, TFLOP/s, time relative to dense, and the floor that time is held
    against: max(kept fraction, time to stream the weights and write the weight gradients once at
    the measured HBM rate / dense time).  `resident`: weights of a shape already on the device."""
    import torch
    table = {}
    for shape, (C, I) in wl.SWEEP_SHAPES.items():
        if resident and shape in resident:
            W = list(resident[shape])
            base = wl.config2(seed=args.seed, skip_ratio=0.0, C=C, I=I,
                              weights=tuple(np.empty((0,), np.float32) for _ in range(3)))
        else:
            base = wl.config2(seed=args.seed, skip_ratio=0.0, C=C, I=I)
            W = [_h_bf16(a).cuda() for a in (base.W_gate, base.W_up, base.W_down)]
        x, dout = _h_bf16(base.x).cuda(), _h_bf16(base.dout).cuda()
        bufs = [torch.empty_like(x), torch.empty_like(x)] + [torch.empty_like(t) for t in W]
        dense = sk.SkipFFN(C, I, base.N, dense=True)
        ms_dense = time_ctx(dense, x, torch.from_numpy(base.skip_mask).cuda(), dout, W, bufs, args.steps, args.warmup)
        del dense
        ctx = sk.SkipFFN(C, I, base.N)
        # weights read by forward and backward, weight gradients written: 9 C I bf16 elements
        ms_weights = 9.0 * C * I * 2 / (pk["hbm_gbs"] * 1e9) * 1e3
        rows = []
        for r in wl.SWEEP_RATIOS:
            m = wl.config2(seed=args.seed, skip_ratio=r, C=8, I=8).skip_mask   # the mask depends on (seed, r) only
            nk = int((m == 0).sum())
            ms = time_ctx(ctx, x, torch.from_numpy(m).cuda(), dout, W, bufs, args.steps, args.warmup)
            tf = sk.skipffn_flops(C, I, nk) / (ms * 1e-3) / 1e12
            floor = max(nk / base.N, ms_weights / ms_dense)
            rows.append({"skip_ratio": r, "kept_tokens": nk, "ms_per_step": ms, "kept_tokens_per_s": nk / (ms * 1e-3),
                         "tflops": tf, "frac_of_measured_bf16_peak": tf / pk["bf16_tflops"],
                         "time_vs_dense": ms / ms_dense, "kept_fraction": nk / base.N,
                         "floor": floor, "time_vs_dense_over_floor": ms / ms_dense / floor})
        tf_dense = sk.skipffn_flops(C, I, base.N) / (ms_dense * 1e-3) / 1e12
        table[shape] = {"C": C, "I": I, "tokens": base.N, "weight_streaming_floor_ms": ms_weights,
                        "dense": {"ms_per_step": ms_dense, "tflops": tf_dense,
                                  "frac_of_measured_bf16_peak": tf_dense / pk["bf16_tflops"]},
                        "points": rows}
        del ctx, W, x, dout, bufs
    return table


def run_sweep(args):
    """The sweep alone, as one JSON line."""
    import torch
    import paper_2503_21817_b200 as sk
    torch.cuda.set_device(0)
    pk = peaks()
    print(json.dumps({"sweep": "skip ratio", "steps": args.steps, "dtype": "bf16", "data": "synthetic",
                      "peak_tflops": pk["bf16_tflops"], "peak_source": pk["source"],
                      "shapes": sweep_table(sk, args, pk)}), flush=True)


# ------------------------------------------------------------------------------ skip KV-cache
def run_kv(args):
    """Skip KV-cache (Eq. 7) at the LLaMA3-8B cache shape: 32 layers x {K, V} planes of
    [tokens, 8 heads x 128] bf16 rows, cfg2 mask.  One JSON line: kept rows/s, achieved GB/s against
    the measured HBM copy rate, and the oracle on a bounded sample of planes."""
    import torch
    import oracle
    import paper_2503_21817_b200 as sk
    torch.cuda.set_device(0)
    pk = peaks()
    mask = wl.config2(seed=args.seed, skip_ratio=args.skip_ratio, C=8, I=8).skip_mask
    N, nk = mask.size, int((mask == 0).sum())
    planes, heads, d = 64, 8, 128
    src = torch.empty(planes, N, heads, d, dtype=torch.bfloat16, device="cuda")
    one = wl.to_bf16_bits(wl.normal(args.seed, wl.TID_X, N * heads * d)).view(np.int16).reshape(N, heads, d)
    src.view(torch.int16)[:] = torch.from_numpy(one).cuda()          # same seeded plane, repeated
    dst = torch.empty_like(src)
    ctx = sk.SkipFFN(64, 64, N)
    ctx.plan(torch.from_numpy(mask).cuda())
    for _ in range(max(args.warmup, 3)):
        ctx.kv_compact(src, dst=dst)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        ctx.kv_compact(src, dst=dst)
    e1.record()
    torch.cuda.synchronize()
    ctx.poll()
    ms = e0.elapsed_time(e1) / args.steps
    row_bytes = heads * d * 2
    moved = 2.0 * planes * nk * row_bytes                              # kept rows read once, written once
    gbs = moved / (ms * 1e-3) / 1e9
    host = np.ascontiguousarray(np.stack([one, one]))                  # the same seeded planes, from the host copy
    t = time.perf_counter()
    ref = oracle.kv_compact(host, mask)
    dt = time.perf_counter() - t
    ok = np.array_equal(dst[:2, :nk].view(torch.int16).cpu().numpy(), ref)
    print(json.dumps({"metric": "skip_kv_cache_kept_rows_per_s", "value": planes * nk / (ms * 1e-3), "unit": "rows/s",
                      "ms": ms, "dtype": "u8", "data": "synthetic",
                      "config": {"workload": f"KV cache of LLaMA3-8B: {planes} planes x {N} tokens x {row_bytes} B rows, "
                                             f"{nk} kept (cfg2 mask)", "cache_bytes": planes * N * row_bytes,
                                 "l2_policy": "cache (646 MB) larger than L2"},
                      "roofline": {"kernel": "k_kv_compact", "bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"],
                                   "unit": "GB/s", "frac": gbs / pk["hbm_gbs"], "peak_source": pk["source"],
                                   "traffic": None},
                      "parity_sampled_planes_bit_exact": bool(ok),
                      "cpu_baseline": {"value": 2 * nk / dt, "unit": "rows/s", "cores": 1, "kind": "oracle",
                                       "sample": f"2 of {planes} planes, {dt * 1e3:.1f} ms"}}), flush=True)


# ------------------------------------------------------------------------------ summary token
def run_summary(args):
    """Adaptive summary token (Eq. 6) at the cfg2 layout: 8 samples, each with a segment of 144
    retained and one of 432 skipped visual tokens, C = 4096, bf16; forward + backward."""
    import torch
    import oracle
    import paper_2503_21817_b200 as sk
    torch.cuda.set_device(0)
    pk = peaks()
    C = wl.SWEEP_SHAPES[args.shape][0]
    sizes = [144, 432] * 8
    n = sum(sizes)
    X = wl.round_to(wl.normal(args.seed, wl.TID_X, n * C), "bf16").reshape(n, C)
    w = wl.round_to(wl.normal(args.seed, wl.TID_WGATE, C, 0.02), "bf16")
    dxs = wl.round_to(wl.normal(args.seed, wl.TID_DOUT, len(sizes) * C), "bf16").reshape(len(sizes), C)
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    bf = lambda a: torch.from_numpy(wl.to_bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16).reshape(a.shape)
    Xd, wd, gd, offd = bf(X), bf(w), bf(dxs), torch.from_numpy(off).cuda()

    def step():
        xs, probs = sk.summary_forward(Xd, offd, wd)
        return xs, sk.summary_backward(Xd, offd, wd, probs, gd)
    for _ in range(max(args.warmup, 3)):
        step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        xs, (dX, dw) = step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    moved = 3.0 * n * C * 2              # X read by forward and by backward, dX written
    t = time.perf_counter()
    ref_xs, _ = oracle.summary_forward(X[:off[2]], off[:3], w)
    ref_dX, _ = oracle.summary_backward(X[:off[2]], off[:3], w, dxs[:2])
    dt = time.perf_counter() - t
    err = float(np.linalg.norm(xs[:2].float().cpu().numpy() - ref_xs) / np.linalg.norm(ref_xs))
    gbs = moved / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "summary_token_fwd_bwd_rows_per_s", "value": n / (ms * 1e-3), "unit": "rows/s", "ms": ms,
                      "dtype": "bf16", "data": "synthetic", "gpu_launches": 4,
                      "config": {"workload": f"{len(sizes)} segments (8 samples x [144 retained | 432 skipped]), "
                                             f"{n} rows, C={C}", "l2_policy": "X (38 MB) fits in L2: second reads hit L2"},
                      "roofline": {"kernel": "summary forward+backward (4 launches)", "bound": "hbm", "achieved": gbs,
                                   "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": gbs / pk["hbm_gbs"],
                                   "peak_source": pk["source"], "traffic": None},
                      "xs_rel_error_first_sample": err,
                      "cpu_baseline": {"value": int(off[2]) / dt, "unit": "rows/s", "cores": 1, "kind": "oracle",
                                       "sample": f"first sample (2 segments, {int(off[2])} rows), {dt:.2f} s"}}), flush=True)


# ------------------------------------------------------------------------------ token merge
def run_merge(args):
    """Token merge (section 4.1) of one high-resolution sample: 2304 skipped tokens merged into 288."""
    import torch
    import oracle
    import paper_2503_21817_b200 as sk
    torch.cuda.set_device(0)
    pk = peaks()
    C = wl.SWEEP_SHAPES[args.shape][0]
    n, k, clusters = 2304, 288, 64
    centers = wl.normal(args.seed, wl.TID_WGATE, clusters * C).reshape(clusters, C)
    which = (wl.raw_u64(args.seed, wl.TID_LAYOUT, 0, n) % np.uint64(clusters)).astype(np.int64)
    X = wl.round_to(centers[which] + 0.35 * wl.normal(args.seed, wl.TID_X, n * C).reshape(n, C), "bf16")
    Xd = torch.from_numpy(wl.to_bf16_bits(X).view(np.int16)).cuda().view(torch.bfloat16).reshape(n, C)
    for _ in range(max(args.warmup, 3)):
        sk.token_merge(Xd, k)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        kept, assign, merged = sk.token_merge(Xd, k)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    ns = 256                                           # oracle on a bounded sample: the first 256 tokens, 32 kept
    t = time.perf_counter()
    oracle.token_merge(X[:ns].astype(np.float64), 32)
    dt = time.perf_counter() - t
    flops = 2.0 * (n - k) * k * C + 4.0 * n * C
    moved = (4.0 * n + k) * C * 2                      # X read by norms, mean, averages, gather and merge
    print(json.dumps({"metric": "token_merge_rows_per_s", "value": n / (ms * 1e-3), "unit": "rows/s", "ms": ms,
                      "dtype": "bf16", "data": "synthetic", "gpu_launches": 11,
                      "config": {"workload": f"{n} tokens of {clusters} noisy clusters, C={C}, keep {k}",
                                 "l2_policy": "X (19 MB) stays in L2 after the first pass"},
                      "roofline": {"kernel": "token merge (11 launches)", "bound": "hbm",
                                   "achieved": moved / (ms * 1e-3) / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s",
                                   "frac": moved / (ms * 1e-3) / 1e9 / pk["hbm_gbs"], "peak_source": pk["source"],
                                   "traffic": None, "gemm_tflops": flops / (ms * 1e-3) / 1e12},
                      "cpu_baseline": {"value": ns / dt, "unit": "rows/s", "cores": 1, "kind": "oracle",
                                       "sample": f"first {ns} tokens, keep 32, {dt:.2f} s"}}), flush=True)


# ------------------------------------------------------------------------------ role cycle counters
def run_role_cycles(args):
    """Where the tensor-core GEMM kernels spend their cycles, per role: needs the instrumented
    library (python -m paper_2503_21817_b200.build --role-cycles).  For each GEMM launch of one
    step, averaged over the SM pairs: the MMA issuer's cycles waiting for operand stages and for a
    free accumulator and its total, the TMA producer's cycles waiting for a free stage, and one
    epilogue warp's cycles waiting for a finished accumulator and busy."""
    import paper_2503_21817_b200.binding as binding
    from paper_2503_21817_b200.build import LIB_ROLE_CYCLES
    if not os.path.exists(LIB_ROLE_CYCLES):
        raise SystemExit("build the instrumented library first: python -m paper_2503_21817_b200.build --role-cycles")
    binding._LIB_PATH = LIB_ROLE_CYCLES
    import torch
    import paper_2503_21817_b200 as sk
    torch.cuda.set_device(0)
    w = make_workload(args, 0)
    x, dout, Wg, Wu, Wd = (_h_bf16(a).cuda() for a in (w.x, w.dout, w.W_gate, w.W_up, w.W_down))
    mask = torch.from_numpy(w.skip_mask).cuda()
    ctx = sk.SkipFFN(w.C, w.I, w.N)
    if args.tune:
        ctx.tune(**{k: int(v) for k, v in (kv.split("=") for kv in args.tune.split(","))})
    out, dx = torch.empty_like(x), torch.empty_like(x)
    dW = [torch.empty_like(t) for t in (Wg, Wu, Wd)]

    def step():
        ctx.forward(x, mask, Wg, Wu, Wd, out=out)
        ctx.backward(dout, dx=dx, dW_gate=dW[0], dW_up=dW[1], dW_down=dW[2])
    for _ in range(max(args.warmup, 3)):
        step()
    ctx.poll()
    status = ctx._view(ctx._ws_ptr, 64, torch.int32)     # the handle's status block; counters from word 16
    status[16:64] = 0
    torch.cuda.synchronize()
    for _ in range(args.steps):
        step()
    ctx.poll()
    v = status.cpu().numpy().astype(np.float64)
    res = {}
    for e, name in enumerate(["gateup", "down", "dh", "dw", "dx"]):
        c = v[16 + 8 * e: 24 + 8 * e]
        k = max(c[7], 1.0)
        res[name] = {"issuer_wait_operands": 16 * c[0] / k, "issuer_wait_accumulator": 16 * c[1] / k,
                     "issuer_total": 16 * c[2] / k, "producer_wait_free_stage": 16 * c[3] / k,
                     "epilogue_warp_wait": 16 * c[4] / k, "epilogue_warp_busy": 16 * c[5] / k}
    print(json.dumps({"role_cycles": "SM cycles per SM pair per launch, mean over %d steps" % args.steps,
                      "config": workload_config(args, w), "kernels": res}), flush=True)


# ------------------------------------------------------------------------------ library yardstick
def run_yardstick(args):
    """Not part of the metric: times the vendor library's plain GEMMs (torch.matmul) on the five
    contraction shapes of the path, same box, same timing method, for context beside the fused
    kernels (which also write G, U, H, apply SiLU*mul / its derivative and scatter residual rows)."""
    import torch
    torch.cuda.set_device(0)
    C, I = wl.SWEEP_SHAPES[args.shape]
    nk = wl.config2(seed=args.seed, skip_ratio=args.skip_ratio, C=8, I=8).n_kept
    bf, dev = torch.bfloat16, "cuda"
    g = torch.Generator(device=dev).manual_seed(0)
    rnd = lambda *sh: torch.randn(*sh, device=dev, dtype=bf, generator=g)
    X, dO, H, dG, dGU = rnd(nk, C), rnd(nk, C), rnd(nk, I), rnd(nk, I), rnd(nk, 2 * I)
    Wgu, Wd = rnd(2 * I, C), rnd(C, I)
    cases = [("gateup", lambda: X @ Wgu.T, 2), ("down", lambda: H @ Wd.T, 1), ("dh", lambda: dO @ Wd, 1),
             ("dw_down", lambda: dO.T @ H, 1), ("dw_gate", lambda: dG.T @ X, 1), ("dw_up", lambda: dG.T @ X, 1),
             ("dx", lambda: dGU @ Wgu, 2)]
    out = {}
    for name, fn, units in cases:
        for _ in range(max(args.warmup, 3)):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        out[name] = {"ms": ms, "tflops": units * 2.0 * nk * C * I / (ms * 1e-3) / 1e12}
    print(json.dumps({"yardstick": "torch.matmul bf16, plain GEMMs of the path's shapes", "kept_tokens": nk,
                      "C": C, "I": I, "sum_ms": sum(v["ms"] for v in out.values()), "gemms": out}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg2", "cfg3", "cfg4"])
    ap.add_argument("--shape", default="llama3-8b", choices=list(wl.SWEEP_SHAPES))
    ap.add_argument("--skip-ratio", type=float, default=0.75)
    ap.add_argument("--dense", action="store_true", help="in-library dense comparator (mask ignored)")
    ap.add_argument("--prenorm", action="store_true",
                    help="pre-norm variant: out = x + FFN(RMSNorm(x) * gamma), with dgamma in the backward")
    ap.add_argument("--recompute", action="store_true",
                    help="memory mode: the forward keeps no G, U, H, the backward runs the gate/up GEMM again")
    ap.add_argument("--kept-sized", action="store_true", help="size the compacted arrays by the workload's kept count")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--cpu-sample-tokens", type=int, default=24)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tune", default="", help="comma-separated skipffn_tune knobs for the headline context, e.g. one_box=0")
    ap.add_argument("--no-extras", action="store_true",
                    help="leave out the sustained / cfg3 / cfg4 / sweep keys (N = 1 only carries them)")
    ap.add_argument("--sustained-seconds", type=float, default=3.0)
    ap.add_argument("--profile-only", action="store_true",
                    help="run warmup+steps steps and exit (launch sequence for an ncu capture)")
    ap.add_argument("--sweep", action="store_true",
                    help="skip-ratio sweep at both shapes against the dense comparator (1 GPU)")
    ap.add_argument("--role-cycles", action="store_true",
                    help="per-role cycle counters of the GEMM kernels (needs the instrumented library build)")
    ap.add_argument("--yardstick", action="store_true",
                    help="time the vendor library's plain GEMMs on the path's shapes (context only)")
    ap.add_argument("--kv", action="store_true", help="skip KV-cache compaction (Eq. 7) at the 8B cache shape")
    ap.add_argument("--summary", action="store_true", help="adaptive summary token (Eq. 6), forward + backward")
    ap.add_argument("--merge", action="store_true", help="token merge of section 4.1 on one high-resolution sample")
    args = ap.parse_args()
    if args.role_cycles:
        run_role_cycles(args)
    elif args.merge:
        run_merge(args)
    elif args.summary:
        run_summary(args)
    elif args.kv:
        run_kv(args)
    elif args.yardstick:
        run_yardstick(args)
    elif args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
