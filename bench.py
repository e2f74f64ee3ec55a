#!/usr/bin/env python
"""Benchmark of the incremental depth-first CNN path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload vgg2d] [--impl ours|reference]

One step = one whole batch of streams pushed through the full net (all rows and the end of input,
idf_stream_push_last).  Prints ONE JSON line on rank 0.  Under torchrun every rank runs its own batch of streams
(weak scaling, no collective on the data path); the time is the maximum over ranks.

`--impl reference` times the CPU oracle (oracle/) on the host cores on a bounded sample of the
same workload.
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
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1804_10727_b200 import workloads  # noqa: E402

METRIC = "input pixels/s through full net (batched streams)"
UNIT = "pixels/s"


def measured_peaks():
    """Roofline denominators: the machine's measured copy bandwidth and cuBLAS bf16 rate, as a burst (a kernel timed
    alone or in a short region) and sustained (seconds under the power cap); an earlier measurement if the file is absent."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


def kernel_source_hash() -> str:
    """Fingerprint of the CUDA sources: a counter record only speaks for the kernels it was taken from."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_1804_10727_b200", "csrc")
    for n in sorted(os.listdir(d)):
        if n.endswith((".cu", ".h")):
            h.update(open(os.path.join(d, n), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic(w):
    """DRAM bytes per step of the conv launches from the last ncu capture (dram__bytes_read.sum + dram__bytes_write.sum),
    kept beside the kernels in dram_traffic.json together with the fingerprint of the sources it was taken from.
    None once the kernels have changed since, or when the capture was of another workload."""
    p = os.path.join(ROOT, "paper_1804_10727_b200", "dram_traffic.json")
    if not os.path.exists(p):
        return None, "no ncu capture recorded"
    rec = json.load(open(p)).get(w.name)
    if not rec:
        return None, "no ncu capture recorded for this workload"
    if rec.get("kernel_source_hash") != kernel_source_hash():
        return None, "the kernels have changed since the ncu capture was taken"
    if rec.get("n_streams") != w.n_streams:
        return None, "the ncu capture was taken at another stream count"
    # (rows in + rows out: proportional to the number of rows when the capture was of fewer rows)
    return rec["bytes_per_row"] * w.H, rec.get("note", "")


def algorithmic_bytes(w, net) -> int:
    """Bytes the method must move per step: the input segments in, the output map out, the parameters once."""
    act = {"f32": 4, "bf16": 2, "i8": 1}[w.dtype]
    r, ow, oc = net.out_shape(w.H)
    out_b = w.n_streams * r * ow * oc * (1 if w.dtype == "i8" else 4)
    par = sum(l.cout * l.cin * l.kh * l.kw * act for l in w.layers if l.kind == "conv")
    return w.n_streams * w.H * w.W * w.C * act + out_b + par


def conv_macs(w: workloads.Workload):
    """Algorithmic multiply-accumulates per stream, per layer (the conventional count: under
    deferred emission every unit receives each of its taps exactly once)."""
    H, W, C = w.H, w.W, w.C
    out = []
    for l in w.layers:
        if l.kind == "conv":
            Ho = (H + 2 * l.pad - l.kh) // l.stride + 1
            Wo = 1 if (W == 1 and l.kw == 1) else (W + 2 * l.pad - l.kw) // l.stride + 1
            out.append(Ho * Wo * l.cout * l.cin * l.kh * l.kw)
            H, W, C = Ho, Wo, l.cout
        else:
            out.append(0)
            H, W = H // 2, (1 if W == 1 else W // 2)
    return out


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln)

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [v.strip() for v in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_rate(w: workloads.Workload, budget_s: float, steps: int = 1):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload.
    Returns (pixels/s, threads used, description of the sample, seconds per step list)."""
    from oracle import oracle
    oracle.build()
    cores = oracle.num_threads()
    n_s = max(1, min(w.n_streams, cores))
    ws, bs = workloads.make_params(w)
    # calibrate on a thin slice, then pick the number of rows that fits the budget
    probe_rows = min(w.H, 24 if w.W > 1 else 1500)
    wp = workloads.get(w.name, n_streams=n_s, H=probe_rows)
    xp = workloads.make_input(wp)
    t0 = time.perf_counter()
    oracle.forward(wp.dtype, wp.layers, xp, ws, bs)
    tp = time.perf_counter() - t0
    rows = w.H
    while rows > probe_rows and tp * rows / probe_rows * steps > budget_s:
        rows //= 2
    rows = max(rows, probe_rows)
    wsamp = workloads.get(w.name, n_streams=n_s, H=rows)
    x = workloads.make_input(wsamp)
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        oracle.forward(wsamp.dtype, wsamp.layers, x, ws, bs)
        times.append(time.perf_counter() - t0)
    px = n_s * rows * w.W
    sample = f"{n_s} of {w.n_streams} streams, first {rows} of {w.H} rows each, {len(times)} pass(es)"
    return px / float(np.mean(times)), min(cores, n_s), sample, times


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    total = args.steps + args.warmup
    rate, cores, sample, times = oracle_rate(w, budget_s=150.0, steps=total)
    timed = times[args.warmup:] if len(times) > args.warmup else times
    from oracle import oracle
    # recompute the rate on the timed passes only
    px_per_pass = rate * float(np.mean(times))
    v = px_per_pass / float(np.mean(timed))
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(timed)), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": {"f32": "f64", "bf16": "f64", "i8": "int32"}[w.dtype],
        "data": "synthetic", "config": {"workload": w.name, "n_streams": w.n_streams, "H": w.H, "W": w.W, "sample": sample},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def rank_input(w, rank: int, world: int) -> np.ndarray:
    """The batch of streams rank `rank` owns: every rank processes w.n_streams streams of its own
    (weak scaling), drawn from a different offset of the same seeded generator."""
    return workloads.make_input(w, first=rank * w.n_streams, count=w.n_streams)


def max_over_ranks(t: torch.Tensor, world: int) -> torch.Tensor:
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t


def whole_job_value(w, world: int, steps: int, ms: float) -> float:
    """Pixels all ranks processed in `steps` steps divided by the (max over ranks) time."""
    return world * w.n_streams * w.H * w.W * steps / (ms * 1e-3)


def time_steps(net, d_seg, d_out, steps, warmup, flush_buf, stream, barrier):
    """Device time of `steps` steps (reset + push_last of the whole batch), L2 flushed before each; returns (ms, launches)."""
    def step():
        net.reset()
        net.push_last(d_seg, d_out)
    for _ in range(max(warmup, 3)):
        step()
    barrier()
    evs, n_launch = [], 0
    for _ in range(steps):
        flush_buf.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        step()
        b.record(stream)
        evs.append((a, b))
        n_launch += net.launches
    barrier()
    return sum(a.elapsed_time(b) for a, b in evs), n_launch


def extra_workloads(args, main_name, dev, flush_buf, stream, barrier, peaks):
    """The other workloads, device-timed the same way (fewer steps), as context beside the headline line."""
    from paper_1804_10727_b200 import idf
    out = {}
    for name in workloads.NAMES:
        if name == main_name:
            continue
        w = workloads.get(name)
        ws, bs = workloads.make_params(w)
        net = idf.net_from_workload(w, ws, bs)
        d_seg = idf.segments_from_maps(workloads.make_input(w), w.dtype).to(dev)
        d_out = net.alloc_out(w.H, dev)
        net.open(dev)
        sampler = ClockSampler(int(dev.split(":")[1]))
        sampler.start()
        time.sleep(0.05)
        steps = 10
        ms, n_launch = time_steps(net, d_seg, d_out, steps, 3, flush_buf, stream, barrier)
        clocks = sampler.stop()
        macs = conv_macs(w)
        flops = 2.0 * sum(macs) * w.n_streams
        ratio = {"bf16": 1.0, "i8": 2.0, "f32": 0.5}[w.dtype]
        tf = flops / (ms / steps * 1e-3) / 1e12
        out[name] = {"value": w.n_streams * w.H * w.W * steps / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms / steps, "steps": steps,
                     "n_streams": w.n_streams, "dtype": w.dtype, "gpu_launches_per_step": n_launch // steps,
                     "dense_equiv_tflops": tf, "frac_of_burst_peak_whole_step": tf / (peaks["bf16_burst"] * ratio),
                     "state_bytes_per_stream": net.state_bytes, "clocks": clocks}
        net.close()
        del d_seg, d_out
        torch.cuda.empty_cache()
    return out


def run_ours(args, w):
    import torch.distributed as dist
    from paper_1804_10727_b200 import idf

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank owns its own batch of streams (weak scaling); data differs per rank via the stream offset
    ws, bs = workloads.make_params(w)
    x = rank_input(w, rank, world)
    net = idf.Net(w.dtype, w.layers, w.W, w.C, w.n_streams, ws, bs, row_block=args.row_block, eager=args.eager)
    h_seg = idf.segments_from_maps(x, w.dtype).pin_memory()
    d_seg = h_seg.to(dev)
    d_out = net.alloc_out(w.H, dev)
    h_out = torch.empty(d_out.shape, dtype=d_out.dtype).pin_memory()
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # larger than the 126 MB L2
    stream = torch.cuda.current_stream()

    net.open(dev)                            # binds the workspace and uploads the parameters, once

    def step():
        net.reset()                          # a new batch of streams: all rolling state back to zero
        net.push_last(d_seg, d_out)          # all segments of the batch and the end of input

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()                      # nvidia-smi needs a moment before its first sample: start it ahead of the warm-up
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    # ---- timed region: device-resident inputs, CUDA events on the launching stream -------------
    evs = []
    barrier()
    l0 = net.launches
    n_launch = 0
    for _ in range(args.steps):
        flush_buf.fill_(1)                                  # evict L2 between iterations (untimed)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        step()
        b.record(stream)
        evs.append((a, b))
        n_launch += net.launches                            # launch counter restarts at every reset
    barrier()
    ms = sum(a.elapsed_time(b) for a, b in evs)
    # ---- end to end through idf_run_host: pinned host in, host out, copies inside --------------
    for _ in range(2):
        net.reset(); net.run_host(h_seg, d_seg, h_out, d_out)
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        net.reset()
        net.run_host(h_seg, d_seg, h_out, d_out)
    barrier()
    e2e_s = time.perf_counter() - t0
    clocks = sampler.stop() if rank == 0 else None
    # ---- streaming mode: one segment per push (the paper's use: rows arrive one at a time) ---------
    per_push = 1 if w.H <= 1024 else (w.H + 1023) // 1024      # long 1D signals: a few samples per push, 1024 pushes

    def stream_step():
        net.reset()
        r = 0
        while r + per_push < w.H:
            net.push(d_seg[r:r + per_push], d_out)
            r += per_push
        net.push_last(d_seg[r:], d_out)
    stream_step()
    barrier()
    sa, sb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush_buf.fill_(1)
    sa.record(stream)
    stream_step()
    sb.record(stream)
    barrier()
    stream_ms = sa.elapsed_time(sb)
    stream_launches = net.launches
    # ---- per-layer device time of the same step (instrumented pass, CUDA events per launch) ----
    net.set_timing(True)
    flush_buf.fill_(1)
    step()
    lms, ln = net.layer_times()
    net.set_timing(False)

    t = max_over_ranks(torch.tensor([ms, e2e_s * 1e3, stream_ms], dtype=torch.float64, device=dev), world)
    ms, e2e_ms, stream_ms = float(t[0]), float(t[1]), float(t[2])
    if rank == 0:
        peaks = measured_peaks()
        px_step = world * w.n_streams * w.H * w.W
        macs = conv_macs(w)
        dense = [i for i, l in enumerate(w.layers) if l.kind == "conv" and macs[i] > 0]
        dom_ms = sum(lms[i] for i in dense)
        dom_launches = sum(ln[i] for i in dense)
        flops = 2.0 * sum(macs[i] for i in dense) * w.n_streams
        achieved = flops / (dom_ms * 1e-3) / 1e12 if dom_ms > 0 else 0.0
        ratio = {"bf16": 1.0, "i8": 2.0, "f32": 0.5}[w.dtype]      # nominal ratio to the bf16 dense peak
        traffic, traffic_note = recorded_traffic(w)
        # which peak applies: a timed region of seconds runs under the power cap (sustained), a short one does not (burst)
        timed_s = ms * 1e-3
        kind = "sustained" if timed_s >= 2.0 else "burst"
        peak = peaks["bf16_" + kind] * ratio
        mhz = clocks.get("sm_mhz") if clocks else None
        line = {
            "metric": METRIC, "value": whole_job_value(w, world, args.steps, ms), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": {"f32": "f32", "bf16": "bf16", "i8": "int8"}[w.dtype], "data": "synthetic",
            "config": {"workload": w.name, "n_streams_per_gpu": w.n_streams, "H": w.H, "W": w.W, "C": w.C,
                       "emission": "eager (every unit announces its change after every segment; CUDA cores)" if args.eager else "deferred",
                       "row_block": args.row_block or "default", "l2": "flushed between iterations (256 MiB write)",
                       "state_bytes_per_stream": net.state_bytes},
            "clocks": clocks,
            "ms_per_step_x_sm_mhz": (ms / args.steps) * mhz if mhz else None,
            "e2e": {"value": px_step * args.steps / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": h_seg.numel() * h_seg.element_size(),
                    "d2h_bytes_per_step": h_out.numel() * h_out.element_size()},
            "gpu_launches": n_launch,
            "streaming": {"value": px_step / (stream_ms * 1e-3), "unit": UNIT, "ms_per_step": stream_ms,
                          "pushes": (w.H + per_push - 1) // per_push, "segments_per_push": per_push,
                          "gpu_launches": stream_launches,
                          "note": "segments pushed as they arrive for all streams, the last push carries the end of input"},
            "roofline": {"bound": "alu" if (args.eager or w.dtype == "f32") else "tensor", "kernel": "dense conv update (all conv layers)", "achieved": achieved,
                         "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak if (peak and dom_ms > 0) else None,
                         "peak_source": f"{peaks['source']} bf16 {kind} x{ratio} (timed region {timed_s:.3f} s)",
                         "frac_of_burst": achieved / (peaks["bf16_burst"] * ratio),
                         "frac_of_sustained": achieved / (peaks["bf16_sustained"] * ratio),
                         "frac_of_burst_whole_step": flops / (ms / args.steps * 1e-3) / 1e12 / (peaks["bf16_burst"] * ratio),
                         "traffic": traffic, "traffic_note": traffic_note,
                         "algorithmic_bytes": algorithmic_bytes(w, net),
                         "launches_per_step": dom_launches, "ms_per_step": dom_ms,
                         "layer_ms": [round(v, 4) for v in lms]},
        }
        if world == 1 and args.extra:
            line["extra"] = extra_workloads(args, w.name, dev, flush_buf, stream, barrier, peaks)
        if world == 1 and not args.no_cpu:
            rate, cores, sample, _ = oracle_rate(w, budget_s=25.0)
            line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vgg2d", choices=list(workloads.NAMES))
    ap.add_argument("--streams", type=int, default=None, help="streams per GPU (default: the workload's)")
    ap.add_argument("--rows", type=int, default=None, help="segments per stream (default: the workload's; shorter runs are for profiling)")
    ap.add_argument("--row-block", type=int, default=0)
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--eager", action="store_true", help="eager (anytime) emission instead of the default deferred emission")
    ap.add_argument("--no-extra", dest="extra", action="store_false",
                    help="skip the other four workloads, which are otherwise timed too (device time only, 10 steps each) under an 'extra' key")
    args = ap.parse_args()
    w = workloads.get(args.workload, n_streams=args.streams, H=args.rows)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
