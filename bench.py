#!/usr/bin/env python
"""Benchmark of the HCCS hot path (hccs_forward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config C]

A step is one pass of the whole hot path (row max, clamped distance, score, row sum, reciprocal,
normalise and store) over one batch of synthetic int8 logits: one hccs_forward call.  The headline
workload is the small-edge-transformer shape [4096, 4, 64, 64] (uint8 output, exact divide);
`--config 3|4|5` makes another workload the headline.  Inputs rotate over several buffer sets so
that the working set exceeds the 126 MB L2.  Rank 0 prints one JSON line.

How a rate is timed: W warm-up launches, then back-to-back launches for a fixed wall-clock time
(so that clocks and the launch queue are in their steady state), then, without a gap, R regions of
exactly K steps each, separated by CUDA events on the launching stream.  `ms_per_step` is the
median region divided by K; the fastest and slowest region are reported beside it.  The clock
sampler runs from before the pre-warm to after the last region and only samples taken while the
GPU was under this load are counted.

With the default headline (one GPU) the same line also carries, under `workloads`, the other
standalone workloads, the three other output/reciprocal modes and the fused attention workload,
each timed the same way and each compared in full with the CPU oracle, and a fidelity report.

`--impl reference` times the plain-C CPU oracle on the host cores (there is no other reference
implementation of this method); it is a deliberately slow baseline.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126 * 1000 * 1000
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
METRIC = "hccs_forward rows/s (int8 logits -> uint8 probabilities, exact divide)"
FUSED_METRIC = "hccs_attention_fused query rows/s (int8 Q.K^T -> requantise -> HCCS u8 -> P.V int32)"
MODE_FLAGS = {"u8div": 0, "u8clb": 2, "u16div": 1, "u16clb": 3}

# dram__bytes_read.sum + dram__bytes_write.sum per launch, from one-pass ncu captures of launches in
# the middle of the rotating-buffer loop without a cache flush in front of them (so that the lines
# evicted by a launch are counted like in the timed loop); see profiles/.  None: not captured for
# the kernel as it stands.
NCU_TRAFFIC_BYTES = {"config2": 135.1e6, "config3": 67.0e6, "config4": 400.0e6, "config5": 176.0e6}

# Fused kernel: warp instructions on the integer (ALU) pipe per launch of workload 5, from the ncu
# capture under profiles/ (sm__inst_executed_pipe_alu).  The pipe issues one warp instruction per
# two cycles and scheduler (16 lanes per SM sub-partition), so its peak on 148 SMs x 4 schedulers at
# 1.965 GHz is 148 * 4 * 1.965e9 / 2 warp instructions per second.
FUSED_ALU_WARP_INSTR = {"config5": 59.7e6}
ALU_PIPE_PEAK_WARP_INSTR_S = 148 * 4 * 1.965e9 / 2


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi; every sample carries its time, so
    that a summary can be restricted to the interval a timed region ran in."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int, period_ms: int = 50):
        self.gpu = gpu_index
        self.period_ms = period_ms
        self.proc = None
        self.samples = []          # (host time, sm MHz, max MHz, power W, [reasons])
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", str(self.gpu), "-lms", str(self.period_ms)], stdout=subprocess.PIPE,
                stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm, mx = float(parts[1]), float(parts[2])
            except ValueError:
                continue
            t = time.time()                 # if the tool's own time stamp cannot be read: the time the line arrived
            for fmt in ("%Y/%m/%d %H:%M:%S.%f", "%Y/%m/%d %H:%M:%S"):
                try:
                    t = datetime.datetime.strptime(parts[0], fmt).timestamp()
                    break
                except ValueError:
                    pass
            try:
                power = float(parts[3])
            except ValueError:
                power = None
            reasons = [n for n, v in zip(self.NAMES, parts[5:9]) if v.lower().startswith("active")]
            self.samples.append((t, sm, mx, power, reasons))

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)

    def summary(self, intervals):
        """Median SM clock and the throttle reasons seen over the samples that fall into one of
        the (t0, t1) host-time intervals (the GPU was under the timed load throughout each)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        inside = [s for s in self.samples if any(t0 <= s[0] <= t1 for t0, t1 in intervals)]
        sm = sorted(s[1] for s in inside)
        reasons = sorted({r for s in inside for r in s[4]})
        power = [s[3] for s in inside if s[3] is not None]
        mx = [s[2] for s in self.samples]
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_min_mhz": sm[0] if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "samples_total": len(self.samples), "power_w_max": max(power) if power else None,
                "reasons": reasons, "window": "samples taken during the pre-warm and the timed regions"}


def time_regions(launch, stream, steps, warmup, prewarm_s, timed_s, min_repeats=25, max_repeats=2000,
                 barrier=None):
    """Times `launch(i)` (one step) on `stream`: `warmup` untimed steps, a time-based pre-warm, then R
    back-to-back regions of exactly `steps` steps between CUDA events.  Returns the per-region
    times in ms and the host-time interval in which the GPU was under this load."""
    import torch
    for i in range(warmup):
        launch(i)
    repeats = min_repeats
    if max_repeats > min_repeats:
        # a first estimate of the step time picks the number of regions
        probe = max(8, min(64, steps))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(probe):
            launch(i)
        b.record(stream)
        torch.cuda.synchronize()
        est_ms = max(a.elapsed_time(b) / probe, 1e-4)
        repeats = int(min(max_repeats, max(min_repeats, timed_s * 1e3 / (est_ms * steps) + 1)))
    if barrier is not None:
        barrier()
    events = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    t_load0 = time.time()
    i = 0
    t_end = time.perf_counter() + prewarm_s
    while time.perf_counter() < t_end:          # the host runs ahead of the GPU: no idle gap follows
        launch(i)
        i += 1
    h0 = time.perf_counter()
    events[0].record(stream)
    for r in range(repeats):
        for _ in range(steps):
            launch(i)
            i += 1
        events[r + 1].record(stream)
    h1 = time.perf_counter()
    torch.cuda.synchronize()
    t_load1 = time.time()
    if barrier is not None:
        barrier()
    regions = [events[r].elapsed_time(events[r + 1]) for r in range(repeats)]
    return {"regions_ms": regions, "interval": (t_load0 + 0.1, t_load1), "prewarm_launches": i - repeats * steps,
            "host_enqueue_us_per_step": 1e6 * (h1 - h0) / (repeats * steps)}


def region_stats(regions_ms, steps):
    med = statistics.median(regions_ms)
    return {"ms_per_step": med / steps, "ms_per_step_min": min(regions_ms) / steps,
            "ms_per_step_max": max(regions_ms) / steps, "ms_per_step_mean": statistics.fmean(regions_ms) / steps,
            "repeats": len(regions_ms)}


def workload_for(args):
    from paper_2604_02292_b200 import workloads
    if args.shape:
        shape = tuple(int(v) for v in args.shape.split(","))
        if args.config == 5:
            return workloads.make_attention(12345, shape)
        wl = workloads.make_rows(12345, shape, kind="gauss")
        wl.name = "rows" + "x".join(str(v) for v in shape)
        return wl
    return workloads.make_config(args.config)


def buffer_sets(wl, osz):
    """Number of rotating buffer sets of a standalone workload: at least four, and enough for four
    times the L2 size."""
    return min(64, max(4, -(-4 * L2_BYTES // ((1 + osz) * wl.elements))))


def config_dict(wl, mode):
    """The `config` object; both arms print the same one for the same workload and mode."""
    if wl.logits is None:
        Bt, H, L, d = wl.shape
        return {"workload": wl.name, "shape": list(wl.shape), "flags": int(wl.flags), "mode": "u8div",
                "cache": f"GPU arm: 3 rotating buffer sets of {7 * Bt * H * L * d >> 20} MiB; CPU arm: the one "
                         "host copy"}
    flags = int(wl.flags) | MODE_FLAGS[mode]
    osz = 2 if flags & 1 else 1
    n = buffer_sets(wl, osz)
    total = (1 + osz) * wl.elements * n
    note = "> L2" if total > L2_BYTES else "fits the L2: a launch-bound workload, not a bandwidth figure"
    return {"workload": wl.name, "shape": list(wl.shape), "flags": flags, "mode": mode,
            "cache": f"GPU arm: {n} rotating buffer sets ({total >> 20} MiB) {note}; CPU arm: the one host copy"}


def algorithmic_bytes(wl, flat: bool):
    """Bytes one launch must move.  flat: 1 B read + 1 B written per element (the metric's
    2 B/element); otherwise causal rows count only the valid prefix that has to be read."""
    Bt, H, Lq, Lk = wl.shape
    n = Bt * H * Lq * Lk
    if flat or not (wl.flags & 4):
        return 2 * n
    valid = sum(min(max(i + (Lk - Lq) + 1, 0), Lk) for i in range(Lq))
    return Bt * H * valid + n


def oracle_mode_of(orc, flags):
    return (orc.MODE_CAUSAL if flags & 4 else 0) | (orc.MODE_U16 if flags & 1 else 0) | \
        (orc.MODE_CLB if flags & 2 else 0)


def cpu_oracle_rate(wl, flags, min_seconds: float, threads: int):
    """rows/s of the oracle as it stands on the host cores over whole passes of the workload."""
    from oracle import hccs_oracle as orc
    mode = oracle_mode_of(orc, flags)
    orc.forward(wl.logits[:1], wl.theta, mode)                 # load the library
    passes, t0 = 0, time.perf_counter()
    while True:
        orc.forward(wl.logits, wl.theta, mode, threads=threads)
        passes += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds:
            break
    return wl.rows * passes / dt, passes, dt


def run_reference(args):
    """The CPU oracle as the reference arm (rank 0 only): a step is one pass of the oracle over the
    whole workload on all host cores."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = workload_for(args)
    from oracle import hccs_oracle as orc
    cores = os.cpu_count() or 1
    if wl.logits is None:
        Bt, H, L, d = wl.shape
        rows = Bt * H * L

        def step():
            orc.attention(wl.Q, wl.K, wl.V, wl.requant_mult, wl.requant_shift, wl.theta, threads=cores)
        metric, mode = FUSED_METRIC, "u8div"
    else:
        rows = wl.rows
        omode = oracle_mode_of(orc, wl.flags | MODE_FLAGS[args.mode])

        def step():
            orc.forward(wl.logits, wl.theta, omode, threads=cores)
        metric, mode = METRIC, args.mode
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = rows * args.steps / dt
    sample = f"the whole workload per step ({rows} rows), {args.steps} steps in {dt:.2f} s"
    print(json.dumps({
        "impl": "reference", "metric": metric, "value": value, "unit": "rows/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic", "config": config_dict(wl, mode),
        "cpu_baseline": {"value": value, "unit": "rows/s", "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "rows/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


class Timing:
    """What the legs of one run share: protocol parameters, the clock sampler, the load intervals."""

    def __init__(self, args, sampler, barrier=None):
        self.steps, self.warmup = args.steps, max(args.warmup, 3)
        self.kernel_only = args.kernel_only
        self.sampler, self.barrier = sampler, barrier
        self.intervals = []

    def run(self, launch, stream, steps=None, prewarm_s=0.5, timed_s=0.4):
        steps = self.steps if steps is None else steps
        if self.kernel_only:        # profiler captures: few launches, no time-based pre-warm
            t = time_regions(launch, stream, steps, self.warmup, 0.0, 0.0, min_repeats=1, max_repeats=1,
                             barrier=self.barrier)
        else:
            t = time_regions(launch, stream, steps, self.warmup, prewarm_s, timed_s, barrier=self.barrier)
        self.intervals.append(t["interval"])
        out = region_stats(t["regions_ms"], steps)
        out["interval"] = t["interval"]
        out["steps"] = steps
        out["host_enqueue_us_per_step"] = t["host_enqueue_us_per_step"]
        out["prewarm_launches"] = t["prewarm_launches"]
        return out


def time_forward(ctx, wl, mode, timing, dev, keep=None):
    """One standalone leg: hccs_forward on workload `wl` in `mode`, device-resident, plus the full
    comparison of one output buffer with the oracle.  Returns (stats, tensors kept for the caller)."""
    import torch
    flags = int(wl.flags) | MODE_FLAGS[mode]
    osz = 2 if flags & 1 else 1
    odt = torch.uint16 if osz == 2 else torch.uint8
    nbuf = buffer_sets(wl, osz)
    host_x = torch.from_numpy(wl.logits).pin_memory()
    xs = [host_x.to(dev, non_blocking=True) for _ in range(nbuf)]
    ps = [torch.empty(wl.logits.shape, dtype=odt, device=dev) for _ in range(nbuf)]
    stream = torch.cuda.current_stream()
    sptr = stream.cuda_stream
    torch.cuda.synchronize()
    n0 = ctx.hccs_launch_count()

    def launch(i):
        ctx.hccs_forward(xs[i % nbuf], ps[i % nbuf], flags, stream=sptr)

    st = timing.run(launch, stream)
    st["launches_total"] = ctx.hccs_launch_count() - n0
    st["flags"], st["mode"], st["nbuf"], st["osz"] = flags, mode, nbuf, osz
    if osz == 1 and not timing.kernel_only:
        # yardstick: the runtime's device-to-device copy of the same tensor, same buffers, same protocol
        def copy(i):
            ps[i % nbuf].view(torch.int8).copy_(xs[i % nbuf], non_blocking=True)
        st["memcpy_d2d_ms"] = timing.run(copy, stream, prewarm_s=0.2, timed_s=0.2)["ms_per_step"]
        for i in range(nbuf):              # the copies went into the output buffers: compute them again
            launch(i)
        torch.cuda.synchronize()
    if keep is not None:
        keep.update(host_x=host_x, xs=xs, ps=ps, flags=flags, odt=odt, osz=osz, nbuf=nbuf)
    return st, ps[nbuf - 1]


def rates(wl, st, world=1):
    """Derived figures of a standalone leg."""
    peak, peak_kind = measured_peak()
    s = st["ms_per_step"] * 1e-3
    flat = algorithmic_bytes(wl, True) + (st["osz"] - 1) * wl.elements
    true_bytes = algorithmic_bytes(wl, False) + (st["osz"] - 1) * wl.elements
    gbs = flat / s / 1e9
    return {"rows_per_s": world * wl.rows / s, "elements_per_s": world * wl.elements / s, "gbs": gbs,
            "frac_of_measured": gbs / peak, "peak_kind": peak_kind, "peak": peak,
            "frac_of_nominal_8TBs": (2 * wl.elements / s / 1e9) / NOMINAL_HBM_GBS,
            "bytes_per_launch": flat, "true_bytes_per_launch": true_bytes, "gbs_true_bytes": true_bytes / s / 1e9}


def full_parity(wl, flags, got_tensor):
    """Mismatches of one whole output tensor against the oracle (all host cores)."""
    from oracle import hccs_oracle as orc
    want = orc.forward(wl.logits, wl.theta, oracle_mode_of(orc, flags), threads=os.cpu_count() or 1)
    return int((got_tensor.cpu().numpy() != want).sum())


def fidelity_arrays(logits, probs, flags, T, alpha=1.0 / 16, max_rows=4096):
    """Max-abs error and KL of integer probability rows (scale T) against an fp64 exp-softmax of alpha * x
    on a seeded row sample (a report, not a gate)."""
    import numpy as np
    Bt, H, Lq, Lk = logits.shape
    rows = Bt * H * Lq
    rng = np.random.default_rng(0)
    pick = np.sort(rng.choice(rows, size=min(max_rows, rows), replace=False))
    x = logits.reshape(-1, Lk)[pick].astype(np.float64)
    p = probs.reshape(-1, Lk)[pick].astype(np.float64)
    qi = pick % Lq
    valid = (np.arange(Lk)[None, :] <= qi[:, None] + (Lk - Lq)) if flags & 4 else np.ones(x.shape, bool)
    z = np.where(valid, alpha * x, -np.inf)
    z = z - z.max(axis=1, keepdims=True)
    e = np.exp(z)
    sm = e / e.sum(axis=1, keepdims=True)
    err = np.abs(p / float(T) - sm).max(axis=1)
    q = np.where(valid, np.maximum(p, 1e-12), 0.0)
    q = q / q.sum(axis=1, keepdims=True)
    with np.errstate(divide="ignore", invalid="ignore"):
        kl = np.where(sm > 0, sm * (np.log(sm) - np.log(np.where(q > 0, q, 1.0))), 0.0).sum(axis=1)
    return {"alpha": alpha, "rows": int(pick.size), "mean_max_abs": float(err.mean()),
            "worst_max_abs": float(err.max()), "mean_kl": float(kl.mean())}


def fidelity(wl, probs_u8, alpha=1.0 / 16, max_rows=4096):
    """The kernel's uint8 rows of a whole workload against fp64 softmax(alpha x); theta is uncalibrated."""
    out = fidelity_arrays(wl.logits, probs_u8, wl.flags, 255, alpha, max_rows)
    out["note"] = "uint8 output / 255 against fp64 softmax(alpha x); theta uniform in the band, uncalibrated"
    return out


def calibrated_fidelity(ctx, wl, dev, alpha=1.0 / 16):
    """The paper's offline calibration on synthetic logits: theta per head by the grid scan (hccs_calibrate)
    on the first 64 batch entries, fidelity of the int16 path on the next 64 with the workload's
    uniformly drawn theta and with the calibrated one."""
    import torch
    import paper_2604_02292_b200 as pkg
    x = torch.from_numpy(wl.logits[:128]).to(dev)
    t0 = time.perf_counter()
    theta_cal, kl_cal = pkg.hccs_calibrate(x[:64].contiguous(), alpha, (2, 127, 1, 0, 127, 1, 1))
    dt = time.perf_counter() - t0
    out = {"alpha": alpha, "calibration_set": "batch entries 0..63", "held_out": "batch entries 64..127",
           "grid": "Dmax 2..127, S 0..127, every B of the band", "calibration_s": dt,
           "theta_calibrated": theta_cal.tolist(), "objective_on_calibration_set": [float(v) for v in kl_cal]}
    held = x[64:].contiguous()
    for name, theta in (("uniform_in_band", wl.theta), ("calibrated", theta_cal)):
        ctx.hccs_params_upload(theta, wl.n_design)
        p = torch.empty(held.shape, dtype=torch.uint16, device=dev)
        ctx.hccs_forward(held, p, int(wl.flags) | 1)
        torch.cuda.synchronize()
        out[name] = fidelity_arrays(wl.logits[64:128], p.cpu().numpy(), wl.flags, 32767, alpha)
    ctx.hccs_params_upload(wl.theta, wl.n_design)
    return out


def fused_leg(ctx, wl, timing, with_e2e, with_parity):
    """hccs_attention_fused on workload `wl` (one GPU): device-resident rate, optional end-to-end
    leg through torch copies, and the comparison of every (batch, head) slice with the oracle."""
    import torch
    Bt, H, L, d = wl.shape
    ctx.hccs_params_upload(wl.theta, wl.n_design)
    hq, hk, hv = (torch.from_numpy(t).pin_memory() for t in (wl.Q, wl.K, wl.V))
    nbuf = 3                                       # 3 x (75 MB in + 100 MB out) > L2
    bufs = [tuple(t.cuda() for t in (hq, hk, hv)) + (torch.empty(wl.shape, dtype=torch.int32, device="cuda"),)
            for _ in range(nbuf)]
    stream = torch.cuda.current_stream()
    sptr = stream.cuda_stream
    n0 = ctx.hccs_launch_count()

    def launch(i):
        q, k, v, o = bufs[i % nbuf]
        ctx.hccs_attention_fused(q, k, v, o, wl.requant_mult, wl.requant_shift, 0, stream=sptr)

    st = timing.run(launch, stream, steps=min(timing.steps, 50))
    st["launches_total"] = ctx.hccs_launch_count() - n0
    s = st["ms_per_step"] * 1e-3
    rows, logits = Bt * H * L, Bt * H * L * L
    alu = FUSED_ALU_WARP_INSTR.get(wl.name)
    out = dict(st)
    out.update({
        "rows_per_s": rows / s, "logits_per_s": logits / s,
        "tensor_int8_tops_algorithmic": 2 * 2 * logits * d / s / 1e12,
        "hbm_gbs_algorithmic": (3 * rows * d + 4 * rows * d) / s / 1e9,
        "roofline": {"bound": "alu", "unit": "warp instructions/s on the integer pipe",
                     "achieved": alu / s if alu else None, "peak": ALU_PIPE_PEAK_WARP_INSTR_S,
                     "frac": alu / s / ALU_PIPE_PEAK_WARP_INSTR_S if alu else None,
                     "peak_kind": "derived: 148 SMs x 4 schedulers x 1.965 GHz / 2 cycles per warp instruction "
                                  "(measured issue rate of the integer pipe)",
                     "traffic": NCU_TRAFFIC_BYTES.get(wl.name)},
    })
    if with_e2e:
        # end to end: host tensors in, host result out (there is no host-buffer entry point for
        # the fused call: the copies go through torch on the same stream)
        ho = torch.empty(wl.shape, dtype=torch.int32).pin_memory()
        q, k, v, o = bufs[0]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2e_steps = 5
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(e2e_steps):
            q.copy_(hq, non_blocking=True); k.copy_(hk, non_blocking=True); v.copy_(hv, non_blocking=True)
            ctx.hccs_attention_fused(q, k, v, o, wl.requant_mult, wl.requant_shift, 0, stream=sptr)
            ho.copy_(o, non_blocking=True)
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_ms = e0.elapsed_time(e1) / e2e_steps
        out["e2e"] = {"value": rows / (e2e_ms * 1e-3), "unit": "rows/s", "h2d_bytes_per_step": 3 * rows * d,
                      "d2h_bytes_per_step": 4 * rows * d, "ms_per_step": e2e_ms, "steps": e2e_steps}
    if with_parity:
        # every (batch, head) slice against the oracle; its one pass over the workload on the host
        # cores is this workload's CPU baseline
        from oracle import hccs_oracle as orc
        cores = os.cpu_count() or 1
        got = bufs[nbuf - 1][3].cpu().numpy()
        t0 = time.perf_counter()
        want = orc.attention(wl.Q, wl.K, wl.V, wl.requant_mult, wl.requant_shift, wl.theta, threads=cores)
        dt = time.perf_counter() - t0
        out["parity_mismatches"] = int((got != want).sum())
        out["parity_checked"] = f"all {Bt * H} (batch, head) slices"
        out["cpu_baseline"] = {"value": rows / dt, "unit": "rows/s", "cores": cores, "kind": "oracle",
                               "sample": f"the whole workload once in {dt:.1f} s"}
    out["device_status"] = ctx.hccs_device_status()
    del bufs
    torch.cuda.empty_cache()
    return out


def link_rates(dev, nbytes):
    """Plain pinned-memory copy rates of this machine (GB/s): host to device alone, device to host
    alone, and both at once on two streams; the yardstick of the end-to-end leg."""
    import torch
    h_in = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    h_out = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    d_in = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    d_out = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    res = {}

    def timed(fn, reps=5):
        fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(reps):
            fn()
        torch.cuda.synchronize()
        return (time.perf_counter() - t0) / reps

    def h2d():
        with torch.cuda.stream(s1):
            d_in.copy_(h_in, non_blocking=True)

    def d2h():
        with torch.cuda.stream(s2):
            h_out.copy_(d_out, non_blocking=True)

    def both():
        h2d()
        d2h()

    res["h2d_gbs"] = nbytes / timed(h2d) / 1e9
    res["d2h_gbs"] = nbytes / timed(d2h) / 1e9
    res["both_gbs_each_way"] = nbytes / timed(both) / 1e9
    return res


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2604_02292_b200 as pkg
    from paper_2604_02292_b200 import workloads

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(v):
        if world == 1:
            return v
        t = torch.tensor([v], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    full = not args.kernel_only
    sampler = ClockSampler(local)
    if rank == 0 and full:
        sampler.start()
    timing = Timing(args, sampler, barrier=barrier if world > 1 else None)
    ctx = pkg.Context(local)
    wl = workload_for(args)
    fused_headline = wl.logits is None
    extras = (full and world == 1 and args.config == 2 and not args.shape and args.mode == "u8div"
              and not args.no_extras)
    line = None

    if fused_headline:
        # Workload 5 as the headline (one GPU; other ranks of a multi-rank launch have no work)
        if rank == 0:
            f = fused_leg(ctx, wl, timing, with_e2e=full, with_parity=full)
            line = {
                "metric": FUSED_METRIC, "value": f["rows_per_s"], "unit": "rows/s", "n_gpus": 1,
                "steps": f["steps"], "warmup": timing.warmup, "ms_per_step": f["ms_per_step"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
                "data": "synthetic", "config": config_dict(wl, "u8div"),
                "timing": {k: f[k] for k in ("repeats", "ms_per_step_min", "ms_per_step_max", "ms_per_step_mean",
                                             "host_enqueue_us_per_step", "prewarm_launches")},
                "gpu_launches": int(f["repeats"] * f["steps"]),
            }
            for k in ("logits_per_s", "tensor_int8_tops_algorithmic", "hbm_gbs_algorithmic", "roofline", "e2e",
                      "parity_mismatches", "parity_checked", "cpu_baseline", "device_status"):
                if k in f:
                    line[k] = f[k]
    else:
        # Rows are independent: every rank owns one workload-sized shard of a world-times larger
        # batch and nothing is exchanged on the data path (weak scaling).
        ctx.hccs_params_upload(wl.theta, wl.n_design)
        keep = {}
        st, last_out = time_forward(ctx, wl, args.mode, timing, dev, keep=keep)
        for k in ("ms_per_step", "ms_per_step_min", "ms_per_step_max", "ms_per_step_mean"):
            st[k] = max_over_ranks(st[k])
        r = rates(wl, st, world)
        flags, osz, nbuf = keep["flags"], keep["osz"], keep["nbuf"]
        xs, ps, host_x = keep["xs"], keep["ps"], keep["host_x"]
        stream = torch.cuda.current_stream()
        sptr = stream.cuda_stream

        # ---------------- end to end: host tensors in, host tensors out, through hccs_forward_host
        e2e = None
        if full:
            host_p = torch.empty(wl.logits.shape, dtype=keep["odt"]).pin_memory()
            e2e_steps = max(3, min(args.steps, 10))
            for _ in range(2):
                ctx.hccs_forward_host(host_x, host_p, xs[0], ps[0], flags, stream=sptr)
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for s in range(e2e_steps):
                ctx.hccs_forward_host(host_x, host_p, xs[s % nbuf], ps[s % nbuf], flags, stream=sptr)
            e1.record(stream)
            barrier()
            e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps
            e2e = {"value": world * wl.rows / (e2e_ms * 1e-3), "unit": "rows/s", "h2d_bytes_per_step": wl.elements,
                   "d2h_bytes_per_step": wl.elements * osz, "ms_per_step": e2e_ms, "steps": e2e_steps,
                   "gbs_each_way": wl.elements / (e2e_ms * 1e-3) / 1e9}
        status = ctx.hccs_device_status()

        if rank == 0:
            mism = full_parity(wl, flags, last_out)
            if full:
                mism += full_parity(wl, flags, host_p)
                e2e["link"] = link_rates(dev, wl.elements)
            line = {
                "metric": METRIC, "value": r["rows_per_s"], "unit": "rows/s", "n_gpus": world,
                "steps": st["steps"], "warmup": timing.warmup, "ms_per_step": st["ms_per_step"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
                "data": "synthetic", "config": config_dict(wl, args.mode),
                "timing": {"protocol": "W warm-up steps, back-to-back launches for 0.5 s, then R regions of exactly K "
                                       "steps between CUDA events on the launching stream with no gap; ms_per_step "
                                       "is the median region / K",
                           "repeats": st["repeats"], "ms_per_step_min": st["ms_per_step_min"],
                           "ms_per_step_max": st["ms_per_step_max"], "ms_per_step_mean": st["ms_per_step_mean"],
                           "host_enqueue_us_per_step": st["host_enqueue_us_per_step"],
                           "prewarm_launches": st["prewarm_launches"]},
                "elements_per_s": r["elements_per_s"], "gbs_algorithmic": r["gbs"] * world,
                "frac_of_nominal_8TBs": r["frac_of_nominal_8TBs"],
                "roofline": {"bound": "hbm", "achieved": r["gbs"], "peak": r["peak"], "unit": "GB/s",
                             "frac": r["frac_of_measured"], "peak_kind": f"of {r['peak_kind']}",
                             "traffic": NCU_TRAFFIC_BYTES.get(wl.name) if args.mode == "u8div" else None,
                             "algorithmic_bytes_per_launch": r["bytes_per_launch"],
                             "true_bytes_per_launch": r["true_bytes_per_launch"],
                             "achieved_true_bytes": r["gbs_true_bytes"]},
                "gpu_launches": int(st["repeats"] * st["steps"]),
                "parity_mismatches": mism,
                "parity_checked": "every element of one device-resident output" +
                                  (" and of the end-to-end output" if full else ""),
                "device_status": status,
            }
            if e2e is not None:
                line["e2e"] = e2e
            if osz == 1 and full:
                line["fidelity"] = fidelity(wl, last_out.cpu().numpy())
            if "memcpy_d2d_ms" in st:
                line["timing"]["memcpy_d2d_ms"] = st["memcpy_d2d_ms"]
            if world == 1 and full:
                cores = os.cpu_count() or 1
                cpu_rate, cpu_passes, cpu_dt = cpu_oracle_rate(wl, flags, 10.0, cores)
                one_rate, one_passes, one_dt = cpu_oracle_rate(wl, flags, 2.0, 1)
                line["cpu_baseline"] = {"value": cpu_rate, "unit": "rows/s", "cores": cores, "kind": "oracle",
                                        "sample": f"{cpu_passes} whole passes of the workload in {cpu_dt:.1f} s",
                                        "single_thread": {"value": one_rate, "unit": "rows/s", "cores": 1,
                                                          "sample": f"{one_passes} whole passes in {one_dt:.1f} s"}}
        del keep, xs, ps, last_out
        torch.cuda.empty_cache()

        # ---------------- the other workloads and modes, same protocol, same line
        if extras and rank == 0:
            others = {}
            line["fidelity_calibrated_int16"] = calibrated_fidelity(ctx, wl, dev)
            for mode in ("u8clb", "u16div", "u16clb"):
                s2, out2 = time_forward(ctx, wl, mode, timing, dev)
                r2 = rates(wl, s2)
                others[f"config2_{mode}"] = leg_summary(wl, s2, r2, full_parity(wl, s2["flags"], out2), timing)
                del out2
                torch.cuda.empty_cache()
            for c in (3, 4):
                w = workloads.make_config(c)
                ctx.hccs_params_upload(w.theta, w.n_design)
                s2, out2 = time_forward(ctx, w, "u8div", timing, dev)
                r2 = rates(w, s2)
                others[w.name] = leg_summary(w, s2, r2, full_parity(w, s2["flags"], out2), timing)
                others[w.name]["fidelity"] = fidelity(w, out2.cpu().numpy())
                del out2, w
                torch.cuda.empty_cache()
            w = workloads.make_config(1)
            ctx.hccs_params_upload(w.theta, w.n_design)
            s2, out2 = time_forward(ctx, w, "u8div", timing, dev)
            others[w.name] = leg_summary(w, s2, rates(w, s2), full_parity(w, s2["flags"], out2), timing)
            others[w.name]["note"] = "32 KiB: launch-bound, reported only"
            w5 = workloads.make_config(5)
            f = fused_leg(ctx, w5, timing, with_e2e=False, with_parity=True)
            others[w5.name] = {k: f[k] for k in ("ms_per_step", "ms_per_step_min", "ms_per_step_max", "repeats",
                                                 "steps", "rows_per_s", "logits_per_s",
                                                 "tensor_int8_tops_algorithmic", "hbm_gbs_algorithmic", "roofline",
                                                 "parity_mismatches", "parity_checked", "cpu_baseline",
                                                 "device_status")}
            others[w5.name]["config"] = config_dict(w5, "u8div")
            line["workloads"] = others

    if rank == 0 and line is not None:
        sampler.stop()
        if full:
            clocks = sampler.summary(timing.intervals[:1])       # the headline leg's pre-warm and timed regions
            line["clocks"] = clocks
            if clocks.get("sm_mhz"):
                line["timing"]["ms_per_step_x_sm_mhz"] = line["ms_per_step"] * clocks["sm_mhz"]
        else:
            line["clocks"] = None
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    ctx.close()


def leg_clock(timing, st):
    """Median SM clock over the samples taken while this leg's launches ran."""
    time.sleep(0.06)                       # let the sampler deliver the last samples of the interval
    c = timing.sampler.summary([st["interval"]])
    return {"sm_mhz": c.get("sm_mhz"), "samples": c.get("samples"), "reasons": c.get("reasons")}


def leg_summary(wl, st, r, mismatches, timing=None):
    out = leg_summary_core(wl, st, r, mismatches)
    if timing is not None:
        out["clocks"] = leg_clock(timing, st)
    if "memcpy_d2d_ms" in st:
        out["memcpy_d2d_ms"] = st["memcpy_d2d_ms"]
    return out


def leg_summary_core(wl, st, r, mismatches):
    return {"config": config_dict(wl, st["mode"]), "ms_per_step": st["ms_per_step"],
            "ms_per_step_min": st["ms_per_step_min"], "ms_per_step_max": st["ms_per_step_max"],
            "repeats": st["repeats"], "steps": st["steps"], "rows_per_s": r["rows_per_s"],
            "gbs_algorithmic": r["gbs"], "frac_of_measured": r["frac_of_measured"],
            "frac_of_nominal_8TBs": r["frac_of_nominal_8TBs"], "gbs_true_bytes": r["gbs_true_bytes"],
            "host_enqueue_us_per_step": st["host_enqueue_us_per_step"],
            "parity_mismatches": mismatches, "parity_checked": "every element of one output"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--shape", default="", help="B,H,Lq,Lk: time hccs_forward on seeded Gaussian rows of this "
                                                "shape instead of a named workload (with --config 5: B,H,L,d "
                                                "operands of the fused call)")
    ap.add_argument("--mode", default="u8div", choices=sorted(MODE_FLAGS),
                    help="output type and reciprocal of hccs_forward (the headline is u8div)")
    ap.add_argument("--kernel-only", action="store_true",
                    help="only the device-resident timing of the headline, W + K launches in all (for "
                         "profiler captures): no pre-warm by time, no end-to-end leg, no CPU baseline, no clock "
                         "sampling")
    ap.add_argument("--no-extras", action="store_true",
                    help="leave out the `workloads` legs (other workloads and modes) of the default run")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
