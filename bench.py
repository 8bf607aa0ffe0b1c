#!/usr/bin/env python
"""Benchmark of the RRM hot path on B200.

Workload: the int8 delta-FC configuration (AlexNet-fc6 shape 9216 -> 4096, int32 accumulation,
32-frame sequences whose frames differ in a fraction rho of the inputs, changed entries in runs
of 32).  One "step" = one frame through the whole hot path of the layer (delta + compaction,
column-gather product, accumulate + snapshot + output), i.e. one rrm_step call.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--rho 0.05] [--impl ours|reference]

Timing: every timed step is preceded by an untimed L2 flush (a 256 MiB device write), and is
bracketed by its own CUDA event pair on the launching stream; ms_per_step is the mean of those
K durations, max over ranks.  N > 1 runs N independent replicas (one video stream and one layer
state per GPU, no data-path collective): weak scaling.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

C_IN, C_OUT, FRAMES = 9216, 4096, 32
DENSE_MACS = C_IN * C_OUT
RHOS = (0.01, 0.05, 0.20)


def pingpong(frames):
    """0,1,..,F-1,F-2,..,1 : replaying it keeps every step's delta density representative."""
    return list(range(frames)) + list(range(frames - 2, 0, -1))


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:  # noqa: BLE001
            pass
    return 6650.0, "fallback"


def committed_traffic(rho):
    """DRAM bytes per launch of the delta-FC kernel from the committed ncu summary, if present."""
    p = os.path.join(ROOT, "profiles", "fc_delta_i8_fc6.txt")
    if not os.path.exists(p):
        return None
    for line in open(p):
        parts = line.split()
        if len(parts) >= 3 and parts[0] == "traffic_bytes_per_launch" and parts[1] == f"rho={rho:g}":
            return float(parts[2])
    return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.samples, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:  # noqa: BLE001
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.t.join(timeout=2)
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            try:
                mhz.append(float(s[0]))
                mx = float(s[1])
                for nme, v in zip(names, s[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(nme)
            except Exception:  # noqa: BLE001
                continue
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz)}


def run_reference(args, rank, world):
    """The CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return
    import workloads as wl
    from oracle import rrm_oracle as orc
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=FRAMES, rho=args.rho, seed=21)
    order = pingpong(FRAMES)
    rec = orc.Recurrence([spec])
    rec.step(seq[0])
    for i in range(args.warmup):
        rec.step(seq[order[(i + 1) % len(order)]])
    t0 = time.perf_counter()
    for i in range(args.steps):
        rec.step(seq[order[(args.warmup + i + 1) % len(order)]])
    dt = time.perf_counter() - t0
    fps = args.steps / dt
    print(json.dumps({
        "impl": "reference", "metric": "frames_per_sec", "value": fps, "unit": "frames/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "i8", "data": "synthetic",
        "config": {"workload": f"cfg2 delta-FC int8 fc6 {C_IN}->{C_OUT}, rho={args.rho:g}, 1 stream"},
        "dense_equiv_gmacs": fps * DENSE_MACS / 1e9,
        "cpu_baseline": {"value": fps, "unit": "frames/s", "cores": orc.threads(), "kind": "oracle",
                         "sample": f"{args.steps} frames of the same sequence through the oracle's Algorithm-1 recurrence"},
        "e2e": {"value": fps, "unit": "frames/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=992)
    ap.add_argument("--warmup", type=int, default=62)
    ap.add_argument("--rho", type=float, default=0.05)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="skip the secondary sweeps (profiling runs)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if args.steps == 992:
            args.steps, args.warmup = 310, 31
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    import workloads as wl
    import paper_1802_09723_b200 as rrm

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    rrm.lib()
    spec = wl.fc6_i8()[0]
    W = torch.from_numpy(spec.weight).cuda()
    B = torch.from_numpy(spec.bias).cuda()
    order = pingpong(FRAMES)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def make(rho, n=1):
        desc = rrm.desc_from_spec(spec, n=n)
        layer = rrm.Net([desc], [W], [B])
        seq = wl.fc_run_sequence(frames=FRAMES, rho=rho, seed=21 + rank, n=n)
        frames = [torch.from_numpy(seq[t]).cuda() for t in range(FRAMES)]
        nnz = [int(np.count_nonzero(seq[order[(i + 1) % len(order)]] != seq[order[i % len(order)]]))
               for i in range(len(order))]
        return layer, seq, frames, float(np.mean(nnz))

    def timed(layer, frames, steps, warmup, cold, dense=False):
        """Returns (mean ms per step, launches).  cold: flush L2 before each step, time each step alone."""
        Y = layer.new_output()
        layer.keyframe(frames[0], Y)
        call = layer.dense if dense else layer.step
        for i in range(warmup):
            call(frames[order[(i + 1) % len(order)]], Y)
        barrier()
        if cold:
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            for i in range(steps):
                flush.fill_(i & 0xff)
                evs[i][0].record(stream)
                call(frames[order[(warmup + i + 1) % len(order)]], Y)
                evs[i][1].record(stream)
            barrier()
            ms = float(np.mean([a.elapsed_time(b) for a, b in evs]))
        else:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(steps):
                call(frames[order[(warmup + i + 1) % len(order)]], Y)
            b.record(stream)
            barrier()
            ms = a.elapsed_time(b) / steps
        if world > 1:
            t = torch.tensor([ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms, steps * (2 if dense else 1)

    def algorithmic_bytes(nnz_mean):
        # gathered weight columns + read/modify/write of P + output + X_t, snapshot read, snapshot write
        return nnz_mean * C_OUT + 8 * C_OUT + 4 * C_OUT + 3 * C_IN

    peak, peak_kind = measured_peaks()

    # ---- primary: one stream, rho as asked, cold L2, per-step events
    layer, seq, frames, nnz_mean = make(args.rho)
    sampler = ClockSampler(local)
    sampler.start()
    ms, launches = timed(layer, frames, args.steps, args.warmup, cold=True)
    clocks = sampler.stop()
    fps = world * 1e3 / ms
    bytes_step = algorithmic_bytes(nnz_mean)
    achieved = bytes_step / (ms * 1e-3) / 1e9
    st = layer.stats(0)

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    xh = [torch.from_numpy(seq[t]).pin_memory() for t in range(FRAMES)]
    yh = torch.empty((1, C_OUT, 1, 1), dtype=torch.int32).pin_memory()
    e2e_steps = 10 if args.quick else min(args.steps, 310)
    for i in range(5):
        layer.step_host(xh[order[(i + 1) % len(order)]], yh)
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        layer.step_host(xh[order[(5 + i + 1) % len(order)]], yh)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
    if world > 1:
        t = torch.tensor([e2e_ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    layer.close()

    extra = {}
    if not args.quick:
        by_rho = {}
        for rho in RHOS:
            L2, _, fr, nz = make(rho)
            c_ms, _ = timed(L2, fr, 310, 31, cold=True)
            w_ms, _ = timed(L2, fr, 310, 31, cold=False)
            d_ms, _ = timed(L2, fr, 124, 10, cold=True, dense=True)
            by_rho[f"{rho:g}"] = {
                "nnz_mean": nz, "cold_us": c_ms * 1e3, "warm_us": w_ms * 1e3, "dense_cold_us": d_ms * 1e3,
                "fps_cold": 1e3 / c_ms, "gmacs_dense_equiv_cold": DENSE_MACS / c_ms / 1e6,
                "speedup_vs_own_dense": d_ms / c_ms,
                "roofline_frac_cold": algorithmic_bytes(nz) / (c_ms * 1e-3) / 1e9 / peak}
            L2.close()
        extra["by_rho"] = by_rho
        streams = {}
        for n in (16, 64):
            L3, _, fr, nz = make(args.rho, n=n)
            c_ms, _ = timed(L3, fr, 124, 10, cold=True)
            streams[str(n)] = {"cold_us_per_step": c_ms * 1e3, "fps_cold": n * 1e3 / c_ms,
                               "algorithmic_gbs": (nz * C_OUT + n * (12 * C_OUT + 3 * C_IN)) / (c_ms * 1e-3) / 1e9}
            L3.close()
        extra["streams_per_call"] = streams

    # ---- CPU oracle on the host cores (rank 0, N = 1 only): a bounded sample of the same workload
    cpu = None
    if rank == 0 and world == 1 and not args.quick:
        from oracle import rrm_oracle as orc
        rec = orc.Recurrence([spec])
        rec.step(seq[0])
        t0 = time.perf_counter()
        cnt = 0
        while cnt < 2 * len(order) and time.perf_counter() - t0 < 20.0:
            rec.step(seq[order[(cnt + 1) % len(order)]])
            cnt += 1
        dt = time.perf_counter() - t0
        cpu = {"value": cnt / dt, "unit": "frames/s", "cores": orc.threads(), "kind": "oracle",
               "sample": f"{cnt} frames of the same sequence through the oracle's Algorithm-1 recurrence (delta path)"}

    if rank == 0:
        line = {
            "metric": "frames_per_sec", "value": fps, "unit": "frames/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "i8", "data": "synthetic",
            "config": {"workload": f"cfg2 delta-FC int8 fc6 {C_IN}->{C_OUT}, rho={args.rho:g}, 1 stream per GPU, "
                                   f"{FRAMES}-frame sequence replayed back and forth",
                       "l2": "flushed before every timed step (256 MiB write); each step timed by its own event pair",
                       "measured_nnz_mean": nnz_mean, "measured_density": nnz_mean / C_IN},
            "dense_equiv_gmacs": fps * DENSE_MACS / 1e9,
            "clocks": clocks,
            "e2e": {"value": world * 1e3 / e2e_ms, "unit": "frames/s", "h2d_bytes_per_step": C_IN,
                    "d2h_bytes_per_step": 4 * C_OUT},
            "gpu_launches": launches,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": committed_traffic(args.rho), "peak_kind": f"of {peak_kind}",
                         "kernel": "fc_delta_i8_kernel", "algorithmic_bytes_per_launch": bytes_step},
            "cpu_baseline": cpu,
            "last_step_stats": st,
        }
        line.update(extra)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
