#!/usr/bin/env python
"""Benchmark of the draft LM-head forward (low-rank head, fused log-softmax / top-k).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extra]
    python bench.py --sweep        (d=8192 rank / batch sweep: one line per point, then a table)

One step = one call of slimspec_head_topk: down-projection, the streamed up-projection,
online log-softmax, top-k and the slab merge, on the 8B-class head at M = 1
(d=4096, r=512, V=128256, k=10).  The metric is microseconds per call (lower is better).
Weights rotate through several distinct copies (more than 4x the L2 capacity in total), so
every call streams cold weights from HBM.  With N > 1 every rank runs an independent
replica of the same workload (the path has no exchange step); the value is then the time
divided by the calls of all ranks.

`--impl reference` times the fp64 CPU oracle on the host cores instead (rank 0 only).
Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "lm_head_us_per_call_M1"
UNIT = "us/call"
WORKLOAD = "c1"                      # d=4096, r=512, V=128256, k=10
L2_BYTES = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# DRAM traffic per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture on this workload, see profiles/fma_head_c1_m1.md), keyed by the SHA-256 of the kernel's source
# files at the time of the capture: a changed source reports null.
KERNEL_SOURCES = ("stream_fma.cu", "epilogue.cuh", "select.cuh", "ptx.cuh")
KNOWN_TRAFFIC = {
    "97561202ccda3577ebdd709a158455009b1992c9962e46812d9e71cf4467abb5": 139.4e6,      # 135.63 MB read + 3.6-3.9 MB written, three launches
}


def kernel_traffic():
    import hashlib
    h = hashlib.sha256()
    try:
        for name in KERNEL_SOURCES:
            with open(os.path.join(ROOT, "paper_2605_10453_b200", "csrc", name), "rb") as f:
                h.update(f.read())
    except OSError:
        return None
    return KNOWN_TRAFFIC.get(h.hexdigest())


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"]))}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def head_bytes(M, d, r, V, k):
    """Algorithmic bytes of one low-rank call: A, B and h read once, top-k written."""
    return 2 * (d * r + r * V) + 2 * M * d + 8 * M * k


def head_flops(M, d, r, V):
    return 2 * M * (d * r + r * V)


def fullhead_bytes(M, d, V, k):
    """Algorithmic bytes of one full-rank call: W and h read once, top-k written."""
    return 2 * d * V + 2 * M * d + 8 * M * k


def fullhead_flops(M, d, V):
    return 2 * M * d * V


def bytes_ratio_target(d, r, V):
    """The speed-up over the full-rank head the low-rank head should reach: 0.8 of the ratio of weights read."""
    return 0.8 * (d * V) / (d * r + r * V)


# --------------------------------------------------------------------------- clocks

class ClockSampler:
    """nvidia-smi in the background, one sample every 100 ms, for the GPU this rank uses."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="clocks_", suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            # the busiest half of the samples stands for "under load"
            top = sorted(sm)[len(sm) // 2:]
            out["sm_mhz"] = statistics.median(top)
            out["sm_max_mhz"] = max(mx)
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# --------------------------------------------------------------------------- reference arm

def oracle_step_time(cfg, M, frac_cols=1.0, reps=1):
    """Seconds per oracle call of the low-rank head on the first frac_cols of the vocabulary."""
    import oracle
    from paper_2605_10453_b200 import synth
    V = max(cfg.k + 1, int(round(cfg.V * frac_cols)))
    x = synth.make_inputs(M, cfg.d, cfg.r, V, seed=cfg.seed, logit_scale=cfg.logit_scale)
    b = {k: oracle.bf16_bits(v) for k, v in x.items()}
    times = []
    for _ in range(reps):
        t0 = time.perf_counter()
        oracle.head_topk(b["h"], b["A"], b["B"], cfg.k)
        times.append(time.perf_counter() - t0)
    return times, V


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2605_10453_b200 import synth
    cfg = synth.CONFIGS[WORKLOAD]
    M = 1
    oracle.build()
    threads_used = min(oracle.threads(), M)
    # size the per-step sample so that the whole run stays within about two minutes
    probe, _ = oracle_step_time(cfg, M, 1.0, reps=1)
    total_full = probe[0] * (args.steps + args.warmup)
    frac = min(1.0, 120.0 / max(total_full, 1e-9))
    times, Vs = oracle_step_time(cfg, M, frac, reps=args.steps + args.warmup)
    timed = times[args.warmup:]
    scale = cfg.V / Vs
    us = statistics.mean(timed) * scale * 1e6
    sample = ("full call" if Vs == cfg.V else
              "first %d of %d vocabulary columns per step, time scaled by %.2f" % (Vs, cfg.V, scale))
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s M=%d d=%d r=%d V=%d k=%d" % (WORKLOAD, M, cfg.d, cfg.r, cfg.V, cfg.k)},
        "cpu_baseline": {"value": us, "unit": UNIT, "cores": threads_used, "kind": "oracle", "sample": sample},
        "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- our arm

NOMINAL_HBM_GBS = 8000.0             # B200 HBM3e, nominal: reported beside the measured copy bandwidth


def time_calls(torch, fn, n):
    """CUDA-event time of n back-to-back calls on the current stream, in milliseconds."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(n):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def time_stats(torch, fn, n, groups=10):
    """n calls timed as `groups` event pairs (each around n // groups back-to-back calls):
    microseconds per call as (median, min, max) over the groups."""
    per = max(1, n // groups)
    vals = []
    for g in range(groups):
        vals.append(time_calls(torch, lambda i: fn(g * per + i), per) * 1e3 / per)
    return {"median": statistics.median(vals), "min": min(vals), "max": max(vals), "calls": per * groups}


def max_over_ranks(dist, ms, device):
    """The slowest rank's time: what a job of independent replicas takes.  dist None = one process."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_us_per_call(ms_max, steps, world):
    """Whole-job microseconds per call: `world` replicas finish steps * world calls in ms_max."""
    return ms_max * 1e3 / (steps * world)


def copies_needed(nbytes):
    return max(2, -(-4 * L2_BYTES // nbytes))


def clock_sample(gpu_index):
    """One read-only nvidia-smi query of the SM clock and the throttle reasons (changes nothing)."""
    try:
        out = subprocess.run(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + ClockSampler.QUERY,
                              "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=20).stdout
        f = [x.strip() for x in out.strip().split(",")]
        reasons = [n for n, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9])
                   if v.lower().startswith("active")]
        return {"sm_mhz": float(f[1]), "sm_max_mhz": float(f[2]), "reasons": reasons}
    except Exception:
        return None


def check_against_oracle(kind, x, ids, lp, k, rows):
    """Compare a timed point's outputs with the CPU oracle on the given rows (outside any timed region).
    Returns the largest log-prob error and whether every rule of the parity tests held."""
    import oracle
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from parity import check_topk
    hb = oracle.bf16_bits(x["h"])[rows]
    if kind == "full":
        ref = oracle.fullhead_topk(hb, oracle.bf16_bits(x["W"]), k)
    else:
        ref = oracle.head_topk(hb, oracle.bf16_bits(x["A"]), oracle.bf16_bits(x["B"]), k)
    try:
        st = check_topk(ref, ids.cpu().numpy(), lp.cpu().numpy(), rows=rows)
        return {"rows_checked": len(rows), "max_logprob_err": st["max_lp_err"], "ok": True}
    except AssertionError as e:
        return {"rows_checked": len(rows), "ok": False, "why": str(e)[:120]}


def sample_rows(M):
    return sorted({0, M // 2, M - 1})


def run_ours(args):
    import torch
    from paper_2605_10453_b200 import binding, build, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the head has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    build.build()
    peaks, peaks_kind = load_peaks()

    cfg = synth.CONFIGS[WORKLOAD]
    M, d, r, V, k = 1, cfg.d, cfg.r, cfg.V, cfg.k
    ctx = binding.Context(max_M=512, max_d=8192, max_V=160000, max_k=16)
    x = synth.make_inputs(M, d, r, V, seed=cfg.seed)
    R = copies_needed(2 * (d * r + r * V))
    h = x["h"].to(dev)
    As = [x["A"].to(dev).clone() for _ in range(R)]
    Bs = [x["B"].to(dev).clone() for _ in range(R)]
    ids = torch.empty((M, k), dtype=torch.int32, device=dev)
    lp = torch.empty((M, k), dtype=torch.float32, device=dev)
    h_pin = x["h"].pin_memory()
    ids_pin = torch.empty((M, k), dtype=torch.int32).pin_memory()
    lp_pin = torch.empty((M, k), dtype=torch.float32).pin_memory()

    def step(i):
        ctx.slimspec_head_topk(h, As[i % R], Bs[i % R], k, out_ids=ids, out_logprobs=lp)

    def step_host(i):
        ctx.slimspec_head_topk_host(h_pin, As[i % R], Bs[i % R], k, out_ids_host=ids_pin, out_logprobs_host=lp_pin)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    K, W = args.steps, max(args.warmup, 3)
    sampler = ClockSampler(local)
    for i in range(W):
        step(i)
    barrier()
    clk_before = clock_sample(local)
    sampler.start()
    # ---- the timed region: exactly K steps
    n0 = ctx.launch_count()
    ms = time_calls(torch, step, K)
    launches = ctx.launch_count() - n0
    barrier()
    ms = max_over_ranks(dist, ms, dev)
    # ---- the dominant kernel alone, events recorded by the library around it, same K steps
    ctx.kernel_timing(True)
    for i in range(K):
        step(i)
    kms, kn = ctx.kernel_timing_read()
    ctx.kernel_timing(False)
    # ---- end to end: host activations in, host results out, every step
    for i in range(3):
        step_host(i)
    barrier()
    e2e_ms = max_over_ranks(dist, time_calls(torch, step_host, K), dev)
    clocks = sampler.stop()
    clk_after = clock_sample(local)
    if clocks["samples"] == 0:
        # the background sampler's period is longer than a short timed region: fall back on the two
        # synchronous reads taken directly before and after it
        got = [c for c in (clk_before, clk_after) if c]
        if got:
            clocks = {"sm_mhz": statistics.median([c["sm_mhz"] for c in got]), "sm_max_mhz": max(c["sm_max_mhz"] for c in got),
                      "reasons": sorted({r_ for c in got for r_ in c["reasons"]}), "samples": len(got)}
    if ctx.last_error() != binding.OK:
        raise SystemExit("device-side wait timed out during the benchmark")

    us_call = job_us_per_call(ms, K, world)
    e2e_us = job_us_per_call(e2e_ms, K, world)
    # One call of this workload is ONE launch of k_fma_head (both projections, softmax, top-k), so the
    # kernel's average launch duration over the timed region is the region's time per call; the same kernel
    # bracketed by events launch by launch (nothing of a call overlaps its neighbours then) is reported beside it.
    iso_us = kms * 1e3 / max(kn, 1)
    one_launch = int(launches) == K
    kern_us = us_call * world if one_launch else iso_us
    kern_bytes = head_bytes(M, d, r, V, k) if one_launch else 2 * r * V + 8 * r * M
    achieved = kern_bytes / (kern_us * 1e-6) / 1e9
    call_gbs = head_bytes(M, d, r, V, k) / (us_call * world * 1e-6) / 1e9

    line = {
        "metric": METRIC, "value": us_call, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 weights, f32 accumulate", "data": "synthetic",
        "config": {"workload": "%s M=%d d=%d r=%d V=%d k=%d" % (WORKLOAD, M, d, r, V, k),
                   "parallelism": "replicas only" if world > 1 else "1 gpu",
                   "cache": "weights rotate through %d copies (%.0f MB > 4x L2): every call is cold" %
                            (R, R * 2 * (d * r + r * V) / 1e6),
                   "path": {1: "generic", 2: "stream", 3: "tensor"}.get(ctx.last_path(), "?")},
        "e2e": {"value": e2e_us, "unit": UNIT, "h2d_bytes_per_step": M * d * 2, "d2h_bytes_per_step": M * k * 8},
        "gpu_launches": int(launches),
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"],
                   "samples": clocks["samples"]},
        "roofline": {"bound": "hbm", "kernel": "k_fma_head", "achieved": achieved, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": kernel_traffic(),
                     "peak_kind": "of " + peaks_kind, "bytes_per_launch": kern_bytes, "us_per_launch": kern_us,
                     "us_per_launch_isolated": iso_us,
                     "frac_of_nominal_8tbs": achieved / NOMINAL_HBM_GBS,
                     "whole_call_frac": call_gbs / peaks["hbm_gbs"],
                     "whole_call_frac_of_nominal_8tbs": call_gbs / NOMINAL_HBM_GBS},
    }

    if rank == 0 and world == 1 and not args.no_extra:
        line["parity_check"] = check_against_oracle("low", x, ids, lp, k, [0])
        line["extra"] = extra_points(torch, ctx, synth, binding, dev, peaks)
        line["cpu_baseline"] = cpu_baseline(cfg, M)
    ctx.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


def cpu_baseline(cfg, M):
    """The oracle as it stands, timed on the host cores for about ten seconds."""
    import oracle as _o
    from paper_2605_10453_b200 import synth
    _o.build()
    x = synth.make_inputs(M, cfg.d, cfg.r, cfg.V, seed=cfg.seed, logit_scale=cfg.logit_scale)
    b = {kk: _o.bf16_bits(v) for kk, v in x.items()}
    times = []
    t_end = time.perf_counter() + 10.0
    while len(times) < 3 or time.perf_counter() < t_end:
        t0 = time.perf_counter()
        _o.head_topk(b["h"], b["A"], b["B"], cfg.k)
        times.append(time.perf_counter() - t0)
    return {"value": statistics.mean(times) * 1e6, "unit": UNIT, "cores": min(_o.threads(), M), "kind": "oracle",
            "sample": "%d full calls of the same workload (M=%d)" % (len(times), M)}


def extra_points(torch, ctx, synth, binding, dev, peaks):
    """The other points of the metric, each timed cold with CUDA events (median / min over ten event
    pairs), with the kernel that streams the weights timed by itself, and checked once against the
    oracle on sampled rows: the small head, the 8B-class head at 1 / 8 / 512 rows, the
    larger-vocabulary head at 1 / 16 rows, the full-rank baseline."""
    out = {}
    paths = {1: "generic", 2: "stream", 3: "tensor"}

    def timed(fn, n, byt, flo, M):
        for i in range(5):
            fn(i)
        st = time_stats(torch, fn, n)
        ctx.kernel_timing(True)
        for i in range(min(n, 50)):
            fn(i)
        kms, kn = ctx.kernel_timing_read()
        ctx.kernel_timing(False)
        t_hbm = byt / (peaks["hbm_gbs"] * 1e9) * 1e6
        t_mma = flo / (peaks["bf16_tflops"] * 1e12) * 1e6
        roof = max(t_hbm, t_mma)
        us = st["median"]
        return {"us_per_call": us, "us_min": st["min"], "us_max": st["max"], "calls": st["calls"],
                "rows_per_s": M / (us * 1e-6), "roofline_us": roof, "roofline_frac": roof / us,
                "bound": "hbm" if t_hbm >= t_mma else "tensor",
                "frac_of_nominal": max(byt / (NOMINAL_HBM_GBS * 1e9), flo / 2.25e15) * 1e6 / us,
                "weights_kernel_us": kms * 1e3 / max(kn, 1), "path": paths.get(ctx.last_path(), "?")}

    def lowrank(name, cfgname, Ms, n_by_M, logits_too=False):
        c = synth.CONFIGS[cfgname]
        d, r, V, k = c.d, c.r, c.V, c.k
        x = synth.make_inputs(max(Ms), d, r, V, seed=c.seed, logit_scale=c.logit_scale)
        R = copies_needed(2 * (d * r + r * V))
        As = [x["A"].to(dev).clone() for _ in range(R)]
        Bs = [x["B"].to(dev).clone() for _ in range(R)]
        for M in Ms:
            xm = dict(x, h=x["h"][:M].contiguous())
            h = xm["h"].to(dev)
            ids = torch.empty((M, k), dtype=torch.int32, device=dev)
            lp = torch.empty((M, k), dtype=torch.float32, device=dev)
            fn = lambda i: ctx.slimspec_head_topk(h, As[i % R], Bs[i % R], k, out_ids=ids, out_logprobs=lp)
            pt = timed(fn, n_by_M[M], head_bytes(M, d, r, V, k), head_flops(M, d, r, V), M)
            torch.cuda.synchronize()
            pt["parity_check"] = check_against_oracle("low", xm, ids, lp, k, sample_rows(M))
            out["%s_M%d" % (name, M)] = pt
            if logits_too:
                lg = torch.empty((M, V), dtype=torch.float32, device=dev)
                fl = lambda i: ctx.slimspec_head_logits(h, As[i % R], Bs[i % R], out_logits=lg)
                out["%s_logits_M%d" % (name, M)] = timed(fl, n_by_M[M], 2 * (d * r + r * V) + 2 * M * d + 4 * M * V,
                                                          head_flops(M, d, r, V), M)
        del As, Bs

    lowrank("c0", "c0", (1,), {1: 200}, logits_too=True)
    lowrank("slimspec", "c1", (1, 8, 512), {1: 200, 8: 200, 512: 40})
    lowrank("c2", "c2", (1, 16), {1: 200, 16: 200})
    # full-rank baseline: W is 1.05 GB, eight times the L2, so one copy is cold by itself
    c1 = synth.CONFIGS["c1"]
    d, r, V, k = c1.d, c1.r, c1.V, c1.k
    xw = {"W": synth.make_W(d, V, c1.seed)}
    Wd = xw["W"].to(dev)
    for M, n in ((1, 50), (8, 50), (512, 10)):
        hh = synth.make_h(M, d, c1.seed)
        h = hh.to(dev)
        ids = torch.empty((M, k), dtype=torch.int32, device=dev)
        lp = torch.empty((M, k), dtype=torch.float32, device=dev)
        fn = lambda i: ctx.fullhead_topk(h, Wd, k, out_ids=ids, out_logprobs=lp)
        pt = timed(fn, n, fullhead_bytes(M, d, V, k), fullhead_flops(M, d, V), M)
        torch.cuda.synchronize()
        pt["parity_check"] = check_against_oracle("full", {"h": hh, "W": xw["W"]}, ids, lp, k, sample_rows(M)[:2])
        out["fullhead_M%d" % M] = pt
    for M in (1, 8, 512):
        out["speedup_vs_fullhead_M%d" % M] = out["fullhead_M%d" % M]["us_per_call"] / out["slimspec_M%d" % M]["us_per_call"]
    out["bytes_ratio_target"] = bytes_ratio_target(d, r, V)
    return out


def run_point(args):
    """One other point of the metric by itself (the 8B-class shapes at --point M rows, cold rotating
    weights, --warmup untimed then --steps timed calls): the command the profiler captures are made with."""
    import torch
    from paper_2605_10453_b200 import binding, build, synth
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    build.build()
    peaks, kind = load_peaks()
    c1 = synth.CONFIGS["c1"]
    d, r, V, k, M = c1.d, c1.r, c1.V, c1.k, args.point
    x = synth.make_inputs(8, d, r, V, seed=c1.seed)
    R = copies_needed(2 * (d * r + r * V))
    As = [x["A"].to(dev).clone() for _ in range(R)]
    Bs = [x["B"].to(dev).clone() for _ in range(R)]
    ctx = binding.Context(max_M=max(M, 8), max_d=d, max_V=V, max_k=k)
    h = synth.make_h(M, d, c1.seed).to(dev)
    ids = torch.empty((M, k), dtype=torch.int32, device=dev)
    lp = torch.empty((M, k), dtype=torch.float32, device=dev)
    fn = lambda i: ctx.slimspec_head_topk(h, As[i % R], Bs[i % R], k, out_ids=ids, out_logprobs=lp)
    for i in range(max(args.warmup, 3)):
        fn(i)
    us = time_calls(torch, fn, args.steps) * 1e3 / args.steps
    if ctx.last_error() != binding.OK:
        raise RuntimeError("device-side wait timed out")
    t_hbm = head_bytes(M, d, r, V, k) / (peaks["hbm_gbs"] * 1e9)
    t_mma = head_flops(M, d, r, V) / (peaks["bf16_tflops"] * 1e12)
    print(json.dumps({"point": "c1 shapes, M=%d" % M, "us_per_call": us, "rows_per_s": M / (us * 1e-6),
                      "roofline_us": max(t_hbm, t_mma) * 1e6, "roofline_frac": max(t_hbm, t_mma) * 1e6 / us,
                      "bound": "hbm" if t_hbm >= t_mma else "tensor", "peaks": kind, "steps": args.steps,
                      "path": {1: "generic", 2: "stream", 3: "tensor"}.get(ctx.last_path(), "?")}))
    ctx.close()


def run_sweep(args):
    """The rank / batch sweep (d=8192, V=128256, r in {d/16, d/8, d/4} and full rank, M in {1..1024}):
    one JSON line per point with us/call and the fraction of the roofline, then a markdown table.
    Weights are drawn on the device from a seeded generator (values do not change the timing)."""
    import torch
    from paper_2605_10453_b200 import binding, build, synth
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    build.build()
    peaks, kind = load_peaks()
    d, V, k = synth.SWEEP_D, synth.SWEEP_V, 10
    ctx = binding.Context(max_M=max(synth.SWEEP_MS), max_d=d, max_V=V, max_k=16)
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)

    def draw(rows, cols, std):
        return (torch.randn((rows, cols), generator=gen, device=dev, dtype=torch.float32) * std).to(torch.bfloat16)

    rows_out = []
    for r in list(synth.SWEEP_RANKS) + [0]:
        full = r == 0
        nbytes = 2 * d * V if full else 2 * (d * r + r * V)
        R = max(1, min(4, -(-2 * L2_BYTES // nbytes)))
        if full:
            Ws = [draw(d, V, d ** -0.5) for _ in range(R)]
        else:
            As = [draw(d, r, d ** -0.5) for _ in range(R)]
            Bs = [draw(r, V, r ** -0.5) for _ in range(R)]
        for M in synth.SWEEP_MS:
            h = draw(M, d, 1.0)
            ids = torch.empty((M, k), dtype=torch.int32, device=dev)
            lp = torch.empty((M, k), dtype=torch.float32, device=dev)
            if full:
                fn = lambda i: ctx.fullhead_topk(h, Ws[i % R], k, out_ids=ids, out_logprobs=lp)
                byt, flo = 2 * d * V + 2 * M * d, 2 * M * d * V
            else:
                fn = lambda i: ctx.slimspec_head_topk(h, As[i % R], Bs[i % R], k, out_ids=ids, out_logprobs=lp)
                byt, flo = head_bytes(M, d, r, V, k), head_flops(M, d, r, V)
            n = max(3, min(100, int(2e4 / (byt / (peaks["hbm_gbs"] * 1e3) + flo / (peaks["bf16_tflops"] * 1e6)))))
            for i in range(3):
                fn(i)
            us = time_calls(torch, fn, n) * 1e3 / n
            t_hbm, t_mma = byt / (peaks["hbm_gbs"] * 1e9) * 1e6, flo / (peaks["bf16_tflops"] * 1e12) * 1e6
            roof = max(t_hbm, t_mma)
            row = {"sweep": "c4", "rank": "full" if full else r, "M": M, "us_per_call": us, "roofline_us": roof,
                   "roofline_frac": roof / us, "bound": "hbm" if t_hbm >= t_mma else "tensor", "peaks": kind,
                   "path": {1: "generic", 2: "stream", 3: "tensor"}.get(ctx.last_path(), "?"), "calls": n}
            if ctx.last_error() != binding.OK:
                raise SystemExit("device-side wait timed out in the sweep")
            rows_out.append(row)
            print(json.dumps(row), flush=True)
        if full:
            del Ws
        else:
            del As, Bs
        torch.cuda.empty_cache()
    print("| rank | M | path | us/call | roofline us | fraction | bound |")
    print("|---|---|---|---|---|---|---|")
    for r_ in rows_out:
        print("| %s | %d | %s | %.1f | %.1f | %.2f | %s |" % (r_["rank"], r_["M"], r_["path"], r_["us_per_call"],
                                                          r_["roofline_us"], r_["roofline_frac"], r_["bound"]))
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the extra points and the CPU baseline")
    ap.add_argument("--sweep", action="store_true", help="run the rank / batch sweep instead of the benchmark line")
    ap.add_argument("--point", type=int, default=0, metavar="M",
                    help="time only the 8B-class shapes at M rows (for profiler captures) instead of the benchmark line")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
    elif args.point > 0:
        run_point(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
