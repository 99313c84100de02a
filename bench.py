#!/usr/bin/env python
"""Benchmark of the HCCS hot path (hccs_forward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config C]

A step is one pass of the whole hot path (row max, clamped distance, score, row sum, reciprocal,
normalise and store) over one batch of synthetic int8 logits: one hccs_forward call.  The default
workload is the small-edge-transformer shape [4096, 4, 64, 64]; `--config 3|4` times the causal
128-key and the 512-key shapes instead.  Inputs rotate over several buffer sets so that the
working set exceeds the 126 MB L2.  One JSON line is printed by rank 0.

`--impl reference` times the plain-C CPU oracle on the host cores (there is no other reference
implementation of this method); it is a deliberately slow baseline.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126 * 1000 * 1000
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (cold L2, so part of the output had not been written back yet); None for workloads
# that were not captured.  Set back to None when the kernel of a workload changes.
NCU_TRAFFIC_BYTES = {"config2": 67.13e6 + 15.2e6, "config3": 33.57e6 + 0.8e6, "config4": 201.34e6 + 153.8e6,
                     "config5": 75.58e6 + 52.65e6}
NOMINAL_HBM_GBS = 8000.0
METRIC = "hccs_forward rows/s (int8 logits -> uint8 probabilities, exact divide)"


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", str(self.gpu), "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL,
                text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def workload_for(args):
    from paper_2604_02292_b200 import workloads
    if args.shape:
        shape = tuple(int(v) for v in args.shape.split(","))
        wl = workloads.make_rows(12345, shape, kind="gauss")
        wl.name = "rows" + "x".join(str(v) for v in shape)
        return wl
    return workloads.make_config(args.config)


def algorithmic_bytes(wl, flat: bool):
    """Bytes one launch must move.  flat: 1 B read + 1 B written per element (the metric's
    2 B/element); otherwise causal rows count only the valid prefix that has to be read."""
    Bt, H, Lq, Lk = wl.shape
    n = Bt * H * Lq * Lk
    if flat or not (wl.flags & 4):
        return 2 * n
    valid = sum(min(max(i + (Lk - Lq) + 1, 0), Lk) for i in range(Lq))
    return Bt * H * valid + n


def cpu_oracle_rate(wl, min_seconds: float, threads: int):
    """rows/s of the oracle as it stands on the host cores over whole passes of the workload."""
    from oracle import hccs_oracle as orc
    mode = orc.MODE_CAUSAL if wl.flags & 4 else 0
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
    """The CPU oracle as the reference arm (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = workload_for(args)
    from oracle import hccs_oracle as orc
    cores = os.cpu_count() or 1
    mode = orc.MODE_CAUSAL if wl.flags & 4 else 0
    # one step = the first `sample_batches` batch entries of the workload
    sample_batches = max(1, min(wl.shape[0], (32 << 20) // (wl.elements // wl.shape[0])))
    x = wl.logits[:sample_batches]
    rows = sample_batches * wl.shape[1] * wl.shape[2]
    for _ in range(args.warmup):
        orc.forward(x, wl.theta, mode, threads=cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.forward(x, wl.theta, mode, threads=cores)
    dt = time.perf_counter() - t0
    value = rows * args.steps / dt
    sample = f"first {sample_batches} of {wl.shape[0]} batch entries per step, {args.steps} steps"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "rows/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic", "config": {"workload": wl.name, "shape": list(wl.shape)},
        "cpu_baseline": {"value": value, "unit": "rows/s", "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "rows/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# Integer operations the method itself spends on one logit of the fused path (tensor-core work
# excluded): requantise (multiply, add, shift, two clamps) 5, row max 1, distance and clamp 2,
# score multiply-add 1, row sum 1, normalise multiply and shift 2.
FUSED_ALU_OPS_PER_LOGIT = 12
ALU_PEAK_TOPS = 148 * 128 * 1.965e9 / 1e12     # 128 integer lanes per SM and clock, nominal


def run_fused(args):
    """Workload 5: hccs_attention_fused on int8 Q, K, V [32, 12, 1024, 64] (one GPU)."""
    import torch
    import paper_2604_02292_b200 as pkg
    from paper_2604_02292_b200 import workloads
    from oracle import hccs_oracle as orc

    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = workloads.make_attention(12345, [int(v) for v in args.shape.split(",")]) if args.shape else workloads.make_config(5)
    Bt, H, L, d = wl.shape
    ctx = pkg.Context(0)
    ctx.hccs_params_upload(wl.theta, wl.n_design)
    hq, hk, hv = (torch.from_numpy(t).pin_memory() for t in (wl.Q, wl.K, wl.V))
    nbuf = 3                                       # 3 x (75 MB in + 100 MB out) > L2
    bufs = [tuple(t.cuda() for t in (hq, hk, hv)) + (torch.empty(wl.shape, dtype=torch.int32, device="cuda"),)
            for _ in range(nbuf)]
    stream = torch.cuda.current_stream()
    sptr = stream.cuda_stream

    def step(i):
        q, k, v, o = bufs[i % nbuf]
        ctx.hccs_attention_fused(q, k, v, o, wl.requant_mult, wl.requant_shift, 0, stream=sptr)

    steps = min(args.steps, 200)
    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    full = not args.kernel_only
    if full:
        sampler.start()
        time.sleep(0.3)
    n0 = ctx.hccs_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    launches = ctx.hccs_launch_count() - n0
    if full:
        t_end = time.time() + 1.0
        while time.time() < t_end:
            for i in range(8):
                step(i)
            torch.cuda.synchronize()
    clocks = sampler.stop() if full else None
    rows = Bt * H * L
    logits = rows * L
    line = {
        "metric": "hccs_attention_fused query rows/s (int8 Q.K^T -> requantise -> HCCS u8 -> P.V int32)",
        "value": rows / (ms * 1e-3), "unit": "rows/s", "n_gpus": 1, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": wl.name, "shape": list(wl.shape),
                   "cache": f"rotating {nbuf} buffer sets > L2"},
        "logits_per_s": logits / (ms * 1e-3),
        "tensor_int8_tops": 2 * 2 * logits * d / (ms * 1e-3) / 1e12,
        "hbm_gbs_algorithmic": (3 * rows * d + 4 * rows * d) / (ms * 1e-3) / 1e9,
        "roofline": {"bound": "alu", "achieved": FUSED_ALU_OPS_PER_LOGIT * logits / (ms * 1e-3) / 1e12,
                     "peak": ALU_PEAK_TOPS, "unit": "Top/s",
                     "frac": FUSED_ALU_OPS_PER_LOGIT * logits / (ms * 1e-3) / 1e12 / ALU_PEAK_TOPS,
                     "peak_kind": "derived: 148 SMs x 128 int lanes x 1.965 GHz",
                     "traffic": NCU_TRAFFIC_BYTES.get(wl.name)},
        "gpu_launches": int(launches), "clocks": clocks, "device_status": ctx.hccs_device_status(),
    }
    if full:
        # end to end: host tensors in, host result out (there is no host-buffer entry point for
        # the fused call: the copies go through torch on the same stream)
        ho = torch.empty(wl.shape, dtype=torch.int32).pin_memory()
        q, k, v, o = bufs[0]
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
        line["e2e"] = {"value": rows / (e2e_ms * 1e-3), "unit": "rows/s", "h2d_bytes_per_step": 3 * rows * d,
                       "d2h_bytes_per_step": 4 * rows * d, "ms_per_step": e2e_ms, "steps": e2e_steps}
        # parity of every (batch, head) slice against the oracle, whose one pass over the workload on
        # the host cores is the CPU baseline (about 40 core-seconds)
        cores = os.cpu_count() or 1
        nsl = Bt * H
        t0 = time.perf_counter()
        want = orc.attention(wl.Q, wl.K, wl.V, wl.requant_mult, wl.requant_shift, wl.theta,
                             bh_range=(0, nsl), threads=cores)
        dt = time.perf_counter() - t0
        got = bufs[0][3].cpu().numpy().reshape(Bt * H, L, d)[:nsl]
        line["parity_mismatches"] = int((got != want.reshape(Bt * H, L, d)[:nsl]).sum())
        line["cpu_baseline"] = {"value": nsl * L / dt, "unit": "rows/s", "cores": cores, "kind": "oracle",
                                "sample": f"all {nsl} (batch, head) slices of the workload, once, in {dt:.1f} s"}
    print(json.dumps(line))
    ctx.close()


def run_ours(args):
    if args.config == 5:
        return run_fused(args)
    import torch
    import torch.distributed as dist
    import paper_2604_02292_b200 as pkg

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

    # Rows are independent: every rank owns one workload-sized shard of a world-times larger
    # batch and nothing is exchanged on the data path (weak scaling).
    wl = workload_for(args)
    ctx = pkg.Context(local)
    ctx.hccs_params_upload(wl.theta, wl.n_design)
    extra = {"u8div": 0, "u8clb": pkg.HCCS_RECIP_CLB, "u16div": pkg.HCCS_OUT_U16,
             "u16clb": pkg.HCCS_OUT_U16 | pkg.HCCS_RECIP_CLB}[args.mode]
    flags = wl.flags | extra
    osz = 2 if flags & pkg.HCCS_OUT_U16 else 1
    odt = torch.uint16 if osz == 2 else torch.uint8
    nbytes = wl.elements
    nbuf = max(4, -(-4 * L2_BYTES // ((1 + osz) * nbytes)))
    nbuf = min(nbuf, 64)
    host_x = torch.from_numpy(wl.logits).pin_memory()
    xs = [host_x.to(dev, non_blocking=True) for _ in range(nbuf)]
    ps = [torch.empty(wl.logits.shape, dtype=odt, device=dev) for _ in range(nbuf)]
    stream = torch.cuda.current_stream()
    sptr = stream.cuda_stream
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------- device-resident throughput
    for s in range(max(args.warmup, 3)):
        ctx.hccs_forward(xs[s % nbuf], ps[s % nbuf], flags, stream=sptr)
    barrier()
    sampler = ClockSampler(local)
    full = not args.kernel_only
    if rank == 0 and full:
        sampler.start()
        time.sleep(0.3)
    launches0 = ctx.hccs_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for s in range(args.steps):
        ctx.hccs_forward(xs[s % nbuf], ps[s % nbuf], flags, stream=sptr)
    e1.record(stream)
    barrier()
    best_ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([best_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        best_ms = float(t.item())
    launches = ctx.hccs_launch_count() - launches0
    # keep the GPU busy long enough for the clock sampler to see it under load
    if rank == 0 and full:
        t_end = time.time() + 1.0
        while time.time() < t_end:
            for s in range(64):
                ctx.hccs_forward(xs[s % nbuf], ps[s % nbuf], flags, stream=sptr)
            torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 and full else None
    ms_per_step = best_ms / args.steps
    rows_per_s = world * wl.rows / (ms_per_step * 1e-3)

    # ---------------- end to end: host tensors in, host tensors out, through hccs_forward_host
    host_p = torch.empty(wl.logits.shape, dtype=odt).pin_memory()
    e2e_steps = max(3, min(args.steps, 10)) if full else 0
    for _ in range(2 if full else 0):
        ctx.hccs_forward_host(host_x, host_p, xs[0], ps[0], flags, stream=sptr)
    barrier()
    e0.record(stream)
    for s in range(e2e_steps):
        ctx.hccs_forward_host(host_x, host_p, xs[s % nbuf], ps[s % nbuf], flags, stream=sptr)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([e2e_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    e2e_rows_per_s = world * wl.rows * e2e_steps / (e2e_ms * 1e-3) if full else None
    status = ctx.hccs_device_status()

    if rank == 0:
        peak, peak_kind = measured_peak()
        kernel_s = ms_per_step * 1e-3
        flat = algorithmic_bytes(wl, True) + (osz - 1) * wl.elements
        true_bytes = algorithmic_bytes(wl, False) + (osz - 1) * wl.elements
        achieved = flat / kernel_s / 1e9
        # parity spot check of the timed launch configuration against the oracle (rank 0)
        from oracle import hccs_oracle as orc
        mode = (orc.MODE_CAUSAL if flags & 4 else 0) | (orc.MODE_U16 if flags & 1 else 0) | \
            (orc.MODE_CLB if flags & 2 else 0)
        nb = max(1, wl.shape[0] // 64)
        want = orc.forward(wl.logits[:nb], wl.theta, mode, threads=os.cpu_count() or 1)
        mism = int((ps[0][:nb].cpu().numpy() != want).sum())
        if full:
            mism += int((host_p[:nb].numpy() != want).sum())
        cpu_cores = os.cpu_count() or 1
        cpu_rate, cpu_passes, cpu_dt = cpu_oracle_rate(wl, 10.0, cpu_cores) if world == 1 and full else (None, 0, 0)
        line = {
            "metric": METRIC, "value": rows_per_s, "unit": "rows/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
            "data": "synthetic",
            "config": {"workload": wl.name, "shape": list(wl.shape), "flags": flags, "mode": args.mode,
                       "cache": f"rotating {nbuf} buffer sets ({2 * nbytes * nbuf >> 20} MiB) > L2",
                       "timing": "CUDA events around the K steps on the launching stream"},
            "elements_per_s": world * wl.elements / kernel_s,
            "gbs_algorithmic": achieved * world,
            "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "traffic": NCU_TRAFFIC_BYTES.get(wl.name) if args.mode == "u8div" else None,
                         "algorithmic_bytes_per_launch": flat,
                         "true_bytes_per_launch": true_bytes,
                         "achieved_true_bytes": true_bytes / kernel_s / 1e9},
            "e2e": {"value": e2e_rows_per_s, "unit": "rows/s", "h2d_bytes_per_step": nbytes,
                    "d2h_bytes_per_step": nbytes * osz,
                    "ms_per_step": e2e_ms / e2e_steps if full else None, "steps": e2e_steps},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "parity_mismatches": mism,
            "device_status": status,
        }
        if cpu_rate is not None:
            line["cpu_baseline"] = {"value": cpu_rate, "unit": "rows/s", "cores": cpu_cores,
                                    "kind": "oracle",
                                    "sample": f"{cpu_passes} whole passes of the workload in {cpu_dt:.1f} s"}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--shape", default="", help="B,H,Lq,Lk: time hccs_forward on seeded Gaussian rows of this "
                                                "shape instead of a named workload (with --config 5: B,H,L,d "
                                                "operands of the fused call)")
    ap.add_argument("--mode", default="u8div", choices=["u8div", "u8clb", "u16div", "u16clb"],
                    help="output type and reciprocal of hccs_forward (the headline is u8div)")
    ap.add_argument("--kernel-only", action="store_true",
                    help="only the device-resident timing (for profiler captures): no end-to-end leg, "
                         "no CPU baseline, no clock sampling")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
