#!/usr/bin/env python
"""Benchmark of the RRM hot path on B200.

Workload: the int8 delta-FC configuration (AlexNet-fc6 shape 9216 -> 4096, int32 accumulation,
32-frame sequences whose frames differ in a fraction rho of the inputs, changed entries in runs
of 32).  One "step" = one chunk of 32 consecutive frames of one stream through the whole hot path
of the layer (delta + compaction, column-gather product, accumulate + snapshot + output for every
frame), i.e. one rrm_step_seq call = one kernel launch; the reported value is frames per second.
Secondary numbers: the same with one frame per call (rrm_step), the library's dense path, other
densities, several streams per call.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--rho 0.05] [--chunk 32] [--impl ours|reference]

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


def whole_job_rate(units_per_rank_step, ms_max_over_ranks, world):
    """Units per second of the whole job: every rank processes `units_per_rank_step` units per step (weak
    scaling, replicas), and a step takes as long as the slowest rank."""
    return world * units_per_rank_step * 1e3 / ms_max_over_ranks


def max_over_ranks(ms, world, device=None):
    """The slowest rank's time (all-reduce MAX over the process group when there is one)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:  # noqa: BLE001
            pass
    return 6650.0, "fallback"


def measured_tensor_tmacs():
    """int8 tensor-core peak in TMAC/s: the measured bf16 burst TFLOP/s x 2 (nominal int8 : bf16 ratio) / 2 (flops per
    MAC); fallback 1590 TFLOP/s bf16."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["bf16_tflops"]), "measured"
    except Exception:  # noqa: BLE001
        return 1590.0, "fallback"


def committed_traffic(kernel, rho):
    """DRAM bytes per launch of the chunk kernel that ran, from its committed ncu summary, if present."""
    p = os.path.join(ROOT, "profiles", {"fc_seq_kernel": "fc_seq_fc6_chunk32.txt",
                                        "fc_tc_kernel": "fc_tc_fc6_chunk32.txt"}[kernel])
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
    """The CPU oracle, as it stands, on the host cores (rank 0 only).  One reference step is a bounded
    sample of the GPU arm's step: ONE frame of the chunk; ms_per_step is scaled to a whole chunk."""
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
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps * args.chunk,
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "i8", "data": "synthetic",
        "config": {"workload": f"cfg2 delta-FC int8 fc6 {C_IN}->{C_OUT}, rho={args.rho:g}, 1 stream; one step = one chunk "
                               f"of {args.chunk} consecutive frames", "frames_per_step": args.chunk},
        "dense_equiv_gmacs": fps * DENSE_MACS / 1e9,
        "cpu_baseline": {"value": fps, "unit": "frames/s", "cores": orc.threads(), "kind": "oracle",
                         "sample": f"1 frame per step ({args.steps} frames of the same sequence) through the oracle's "
                                   f"Algorithm-1 recurrence; ms_per_step scaled to {args.chunk} frames"},
        "e2e": {"value": fps, "unit": "frames/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------------
# Secondary workloads (the convolution configurations): python bench.py --workload cfg1|cfg3_f32|...
# One step = one frame through rrm_net_step (Algorithm 1, one iteration of the frame loop).
# ------------------------------------------------------------------------------------------------
CONV_WORKLOADS = ("cfg1", "cfg3_f32", "cfg3_i8", "cfg4", "cfg5")
FFMA_TMACS, DP4A_TMACS, POPC_TBITMACS = 37.2, 74.5, 148.9      # derived ALU peaks in TMAC/s: lanes per SM x 148 SMs x 1.965 GHz (FFMA 128, dp4a 64 x 4, popc 16 x 32 bits)


def conv_workload(name, frames=None, streams=None):
    """(layer specs, video [F][n]..., n, dtype label).  `streams` overrides the configuration's stream count."""
    import workloads as wl
    if name == "cfg1":
        n = streams or 1
        return wl.single_conv_f32(), wl.block_redraw_sequence(frames=frames or 8, n=n), n, "f32"
    if name == "cfg3_f32":
        n = streams or 1
        return wl.alexnet_convs("f32"), wl.moving_rect_video(frames=frames or 64, hw=227, dtype="f32", seed=31, n=n), n, "f32"
    if name == "cfg3_i8":
        n = streams or 1
        return wl.alexnet_convs("i8"), wl.moving_rect_video(frames=frames or 64, hw=227, dtype="i8", seed=32, n=n), n, "i8"
    if name == "cfg4":
        n = streams or 4
        return (wl.resnet18_convs(), wl.moving_rect_video(frames=frames or 64, hw=224, dtype="i8", seed=41, n=n,
                                                          bg_redraw=0.02), n, "i8")
    if name == "cfg5":
        n = streams or 1
        return (wl.xnor_alexnet_convs(), wl.moving_rect_video(frames=frames or 128, hw=227, dtype="i8", seed=51, n=n),
                n, "i8+bin")
    raise SystemExit(f"unknown workload {name}")


def run_conv(args):
    import torch
    import workloads as wl
    import paper_1802_09723_b200 as rrm
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    specs, video, n, dtype = conv_workload(args.workload, args.frames, args.streams)
    F = video.shape[0]
    net = rrm.net_from_specs(specs, n=n, variant=args.variant)
    frames = [torch.from_numpy(np.ascontiguousarray(video[t])).cuda() for t in range(F)]
    order = pingpong(F)
    period = len(order)
    out = net.new_output()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    dense_macs = wl.dense_macs(specs) * n

    def timed(call, steps, warmup, cold=True):
        net.keyframe(frames[order[0]], out)
        for i in range(warmup):
            call(frames[order[(i + 1) % period]], out)
        torch.cuda.synchronize()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(steps):
            if cold:
                flush.fill_(i & 0xff)
            evs[i][0].record(stream)
            call(frames[order[(warmup + i + 1) % period]], out)
            evs[i][1].record(stream)
        torch.cuda.synchronize()
        return float(np.mean([a.elapsed_time(b) for a, b in evs]))

    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    ms = timed(net.step, args.steps, args.warmup)
    clocks = sampler.stop()
    per_layer = []
    tot_active = 0
    for l, sp in enumerate(specs):
        st = net.stats(l)
        if st["variant"] == 3:                # the last frame was evaluated densely (high measured activity): nothing counted
            tot_active = None
            per_layer.append({"layer": sp.name, "variant": "dense (measured activity >= 75 %)", "dense_macs": st["dense_macs"]})
            continue
        tot_active += st["active_macs"]
        per_layer.append({"layer": sp.name, "rho": st["nnz_elems"] / max(1, st["in_elems"]),
                          "active_in_pixels": st["active_in_pixels"] / max(1, st["in_pixels"]),
                          "active_out_pixels": st["active_out_pixels"] / max(1, st["out_pixels"]),
                          "active_macs": st["active_macs"], "dense_macs": st["dense_macs"], "variant": st["variant"]})
    # ---- roofline of the last timed step: per layer the slower of (MACs executed at the unit's peak) and (bytes that
    # have to move at the HBM peak), summed over the layers, against the measured step time.  Bytes per layer: the delta
    # rows of the active input pixels once + the projection rows of the pixels to update three times (read and write
    # by the convolution, read by the epilogue); weights stay in L2 and are left out.
    hbm, hbm_kind = measured_peaks()
    tens, tens_kind = measured_tensor_tmacs()
    unit_bytes = {"f32": 4.0, "i8": 1.0, "bin": 1.0 / 8}
    mac_peak = {"f32": FFMA_TMACS, "i8": tens, "bin": tens}         # TMAC/s (int8 and binary layers run on the tensor cores)
    roof_us = mac_us = byte_us = 0.0
    for l, sp in enumerate(specs):
        st = net.stats(l)
        dense_step = st["variant"] == 3
        macs = st["dense_macs"] if dense_step else st["active_macs"]
        fin = 1.0 if dense_step else st["active_in_pixels"] / max(1, st["in_pixels"])
        fout = 1.0 if dense_step else st["active_out_pixels"] / max(1, st["out_pixels"])
        peak_l = mac_peak[sp.dtype] if (sp.dtype == "f32" or st["variant"] in (2, 3)) else (DP4A_TMACS if sp.dtype == "i8" else POPC_TBITMACS)
        t_mac = macs / (peak_l * 1e12) * 1e6
        nbytes = st["in_pixels"] * fin * sp.c_in * unit_bytes[sp.dtype] + st["out_pixels"] * fout * sp.c_out * 4 * (2 if dense_step else 3)
        t_byte = nbytes / (hbm * 1e9) * 1e6
        per_layer[l]["roofline_us"] = max(t_mac, t_byte)
        per_layer[l]["roofline_bound"] = "hbm" if t_byte >= t_mac else ("alu" if sp.dtype == "f32" else "tensor")
        roof_us += max(t_mac, t_byte); mac_us += t_mac; byte_us += t_byte
    roofline = {"bound": "hbm" if byte_us >= mac_us else ("alu" if dtype == "f32" else "tensor"),
                "achieved": roof_us * 1e-3 / ms * (hbm if byte_us >= mac_us else (FFMA_TMACS if dtype == "f32" else tens)),
                "peak": hbm if byte_us >= mac_us else (FFMA_TMACS if dtype == "f32" else tens),
                "unit": "GB/s" if byte_us >= mac_us else "TMAC/s", "frac": roof_us * 1e-3 / ms, "traffic": None,
                "peak_kind": f"of {hbm_kind if byte_us >= mac_us else ('derived' if dtype == 'f32' else tens_kind)}",
                "roofline_us_per_step": roof_us, "mac_us": mac_us, "byte_us": byte_us,
                "note": "sum over the layers of max(executed MACs at the unit's peak, algorithmic bytes at the HBM peak) / "
                        "measured step time; per-layer figures in per_layer_last_step"}
    ms_warm = timed(net.step, args.steps, args.warmup, cold=False)
    ms_dense = timed(net.dense, max(8, args.steps // 4), 3)
    # ---- chunks of --seq consecutive frames per call (rrm_net_step_seq: the frames of a chunk overlap layer by layer)
    seq_extra = {}
    if args.seq and args.seq > 1:
        Tq = args.seq
        total = period * Tq // np.gcd(period, Tq)
        walk = torch.stack([frames[order[(i + 1) % period]] for i in range(total)])     # frame i+1 of the walk
        outs = net.new_output(frames=Tq)
        nchunks = total // Tq

        def timed_seq(call, steps, warmup):
            net.keyframe(frames[order[0]], out)
            for i in range(warmup):
                call(walk[(i % nchunks) * Tq:(i % nchunks + 1) * Tq], outs, Tq)
            torch.cuda.synchronize()
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            for i in range(steps):
                k = (warmup + i) % nchunks
                flush.fill_(i & 0xff)
                evs[i][0].record(stream)
                call(walk[k * Tq:(k + 1) * Tq], outs, Tq)
                evs[i][1].record(stream)
            torch.cuda.synchronize()
            return float(np.mean([a.elapsed_time(b) for a, b in evs]))

        steps_q = max(4, args.steps // Tq)
        # (18 warm-up chunks: a large stack measures its activity with one delta chunk after 15 dense ones, and both
        # chunk graphs are to be captured before the timed region)
        ms_seq = timed_seq(net.step_seq, max(steps_q, 16), 18)
        ms_seq_dense = timed_seq(net.dense_seq, steps_q, 3)
        seq_extra = {"seq": {"frames_per_call": Tq, "ms_per_call": ms_seq, "ms_per_frame_step": ms_seq / Tq,
                             "frames_per_sec": n * Tq * 1e3 / ms_seq, "dense_ms_per_call": ms_seq_dense,
                             "dense_frames_per_sec": n * Tq * 1e3 / ms_seq_dense,
                             "speedup_vs_own_dense": ms_seq_dense / ms_seq,
                             "speedup_vs_frame_by_frame": ms * Tq / ms_seq}}
    line = {
        "metric": "frames_per_sec", "value": n * 1e3 / ms, "unit": "frames/s", "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": dtype, "data": "synthetic",
        "config": {"workload": f"{args.workload}: {len(specs)} conv layers, {n} stream(s), {F}-frame video walked back and forth; "
                               f"one step = one frame of every stream through rrm_net_step", "variant": args.variant,
                   "l2": "flushed before every timed step (256 MiB write); each step timed by its own event pair"},
        "dense_equiv_gmacs": n * 1e3 / ms * (dense_macs / n) / 1e9,
        "ms_per_step_warm": ms_warm, "ms_per_step_dense_path": ms_dense, "speedup_vs_own_dense": ms_dense / ms,
        "active_macs_last_step": tot_active, "dense_macs_per_step": dense_macs,
        "active_gmacs_per_s": None if tot_active is None else tot_active / ms / 1e6,
        "clocks": clocks, "roofline": roofline, "per_layer_last_step": per_layer,
    }
    line.update(seq_extra)
    print(json.dumps(line))
    net.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=310, help="timed steps; one step = one chunk of --chunk frames")
    ap.add_argument("--warmup", type=int, default=31)
    ap.add_argument("--rho", type=float, default=0.05)
    ap.add_argument("--chunk", type=int, default=FRAMES, help="frames per rrm_step_seq call")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="skip the secondary sweeps (profiling runs)")
    ap.add_argument("--workload", default="cfg2", choices=("cfg2",) + CONV_WORKLOADS,
                    help="cfg2 (default) is the contract line; the others are secondary convolution workloads")
    ap.add_argument("--variant", default="auto", choices=["auto", "gather", "tensor", "dense"])
    ap.add_argument("--frames", type=int, default=None, help="frames of the synthetic video (convolution workloads)")
    ap.add_argument("--streams", type=int, default=None, help="independent videos per call (convolution workloads)")
    ap.add_argument("--seq", type=int, default=None, help="also time rrm_net_step_seq with this many frames per call (convolution workloads)")
    args = ap.parse_args()
    if args.workload != "cfg2":
        if args.steps == 310:
            args.steps, args.warmup = 60, 5
        run_conv(args)
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
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
    period = len(order)                                  # 62 frames, then the walk repeats
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    T = args.chunk

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def reduce_max(ms):
        return max_over_ranks(ms, world, "cuda")

    def make(rho, n=1, variant="auto"):
        """Layer + the endless back-and-forth walk over the 32-frame sequence, laid out so that chunk k
        is rows [k*T, (k+1)*T) of one device array (whole number of periods, so it wraps seamlessly)."""
        desc = rrm.desc_from_spec(spec, n=n, variant=variant)
        layer = rrm.Net([desc], [W], [B])
        seq = wl.fc_run_sequence(frames=FRAMES, rho=rho, seed=21 + rank, n=n)
        total = period * T // np.gcd(period, T)
        walk = np.stack([seq[order[(i + 1) % period]] for i in range(total)])      # frame i+1 of the walk
        nnz = np.array([np.count_nonzero(seq[order[(i + 1) % period]] != seq[order[i % period]]) / n
                        for i in range(period)])
        # distinct weight columns one chunk touches (what a cold L2 must fetch), mean over the chunks, stream 0
        uniq = []
        for k in range(total // T):
            touched = np.zeros(C_IN, dtype=bool)
            for i in range(k * T, (k + 1) * T):
                touched |= seq[order[(i + 1) % period]][0] != seq[order[i % period]][0]
            uniq.append(int(touched.sum()))
        return layer, seq, walk, torch.from_numpy(walk).cuda(), float(nnz.mean()), float(np.mean(uniq))

    def timed_chunks(layer, seq, walk_dev, steps, warmup, cold, dense=False, frames_per_call=None):
        """Mean ms per call of rrm_step_seq (or rrm_dense_seq) over chunks of the walk."""
        tc = T if frames_per_call is None else frames_per_call
        nchunks = walk_dev.shape[0] // tc
        Y = layer.new_output(frames=tc)
        layer.keyframe(torch.from_numpy(seq[order[0]]).cuda(), None)
        call = layer.dense_seq if dense else layer.step_seq
        for i in range(warmup):
            call(walk_dev[(i % nchunks) * tc:(i % nchunks + 1) * tc], Y, tc)
        barrier()
        if cold:
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            for i in range(steps):
                k = (warmup + i) % nchunks
                flush.fill_(i & 0xff)
                evs[i][0].record(stream)
                call(walk_dev[k * tc:(k + 1) * tc], Y, tc)
                evs[i][1].record(stream)
            barrier()
            ms = float(np.mean([a.elapsed_time(b) for a, b in evs]))
        else:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(steps):
                k = (warmup + i) % nchunks
                call(walk_dev[k * tc:(k + 1) * tc], Y, tc)
            b.record(stream)
            barrier()
            ms = a.elapsed_time(b) / steps
        return reduce_max(ms)

    def timed_single(layer, seq, frames, steps, warmup, cold, dense=False):
        """Mean ms per rrm_step (one frame per call)."""
        Y = layer.new_output()
        layer.keyframe(frames[0], Y)
        call = layer.dense if dense else layer.step
        for i in range(warmup):
            call(frames[order[(i + 1) % period]], Y)
        barrier()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(steps):
            if cold:
                flush.fill_(i & 0xff)
            evs[i][0].record(stream)
            call(frames[order[(warmup + i + 1) % period]], Y)
            evs[i][1].record(stream)
        barrier()
        return reduce_max(float(np.mean([a.elapsed_time(b) for a, b in evs])))

    def frame_bytes(nnz_mean):
        # per frame: gathered weight columns + read/modify/write of P + output + X_t, snapshot read, snapshot write
        return nnz_mean * C_OUT + 8 * C_OUT + 4 * C_OUT + 3 * C_IN

    def dense_chunk_bytes(frames):
        # the dense evaluation of a chunk: W once, the frames, outputs, stored projection, snapshot
        return C_IN * C_OUT + (frames + 1) * C_IN + frames * 4 * C_OUT + 4 * C_OUT

    EVAL = {1: "column gather", 3: "dense on the tensor cores, W read once (rows x measured density of the previous "
                                   "chunk >= 0.75)"}
    KERNEL = {1: "fc_seq_kernel", 3: "fc_tc_kernel"}

    def chunk_cold_bytes(uniq_cols, frames):
        # what one chunk launch must fetch with a cold L2: every distinct column once, the frames, per-frame
        # projection deltas (write + read) and outputs, the stored projection
        return uniq_cols * C_OUT + (frames + 2) * C_IN + frames * 12 * C_OUT + 8 * C_OUT

    peak, peak_kind = measured_peaks()

    # ---- primary: one stream per GPU, chunks of T frames per call, rho as asked, cold L2, per-step events
    layer, seq, walk, walk_dev, nnz_mean, uniq_mean = make(args.rho)
    sampler = ClockSampler(local)
    sampler.start()
    ms = timed_chunks(layer, seq, walk_dev, args.steps, args.warmup, cold=True)
    clocks = sampler.stop()
    fps = whole_job_rate(T, ms, world)
    bytes_launch = frame_bytes(nnz_mean) * T
    achieved = bytes_launch / (ms * 1e-3) / 1e9
    st = layer.stats(0)
    main_variant = st["variant"]
    own_bytes = dense_chunk_bytes(T) if main_variant == 3 else chunk_cold_bytes(uniq_mean, T)

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    nchunks = walk.shape[0] // T
    xh = torch.from_numpy(walk).pin_memory()
    yh = torch.empty((T, 1, C_OUT, 1, 1), dtype=torch.int32).pin_memory()
    e2e_steps = 10 if args.quick else min(args.steps, 310)
    layer.keyframe(torch.from_numpy(seq[order[0]]).cuda(), None)
    # (a) every call waits for its outputs (latency of one chunk); (b) calls queued without waiting, one wait at the
    # end: the copy-in of chunk k+1 and the copy-out of chunk k-1 overlap the kernels of chunk k.  Both copy every
    # step's frames from pinned host memory and every step's outputs back to it.
    for i in range(5):
        layer.step_seq_host(xh[(i % nchunks) * T:(i % nchunks + 1) * T], yh, T)
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        k = (5 + i) % nchunks
        layer.step_seq_host(xh[k * T:(k + 1) * T], yh, T)
    torch.cuda.synchronize()
    e2e_sync_ms = reduce_max((time.perf_counter() - t0) * 1e3 / e2e_steps)
    for i in range(5):
        layer.step_seq_host_async(xh[((5 + e2e_steps + i) % nchunks) * T:((5 + e2e_steps + i) % nchunks + 1) * T], yh, T)
    layer.host_sync()
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        k = (10 + e2e_steps + i) % nchunks
        layer.step_seq_host_async(xh[k * T:(k + 1) * T], yh, T)
    layer.host_sync()
    e2e_ms = reduce_max((time.perf_counter() - t0) * 1e3 / e2e_steps)
    layer.close()

    extra = {}
    if not args.quick:
        by_rho = {}
        for rho in RHOS:
            L2, sq, wk, wd, nz, un = make(rho)
            fr = [torch.from_numpy(sq[t]).cuda() for t in range(FRAMES)]
            c_ms = timed_chunks(L2, sq, wd, 124, 10, cold=True)
            variant = EVAL.get(L2.stats(0)["variant"], "?")
            w_ms = timed_chunks(L2, sq, wd, 124, 10, cold=False)
            d_ms = timed_chunks(L2, sq, wd, 31, 3, cold=True, dense=True)
            s_ms = timed_single(L2, sq, fr, 310, 31, cold=True)
            sd_ms = timed_single(L2, sq, fr, 124, 10, cold=True, dense=True)
            LG = make(rho, variant="gather")[0]            # the column-gather kernel whatever the density
            g_ms = timed_chunks(LG, sq, wd, 124, 10, cold=True)
            LG.close()
            by_rho[f"{rho:g}"] = {
                "nnz_mean_per_frame": nz, "distinct_columns_per_chunk": un, "chunk_evaluation": variant,
                "chunk_cold_us": c_ms * 1e3, "chunk_warm_us": w_ms * 1e3, "dense_chunk_cold_us": d_ms * 1e3,
                "gather_chunk_cold_us": g_ms * 1e3,
                "fps_cold": T * 1e3 / c_ms, "gmacs_dense_equiv_cold": T * DENSE_MACS / c_ms / 1e6,
                "speedup_vs_own_dense_chunk": d_ms / c_ms, "gather_speedup_vs_own_dense_chunk": d_ms / g_ms,
                "roofline_frac_per_frame_bytes": frame_bytes(nz) * T / (c_ms * 1e-3) / 1e9 / peak,
                "gather_roofline_frac_per_frame_bytes": frame_bytes(nz) * T / (g_ms * 1e-3) / 1e9 / peak,
                "gather_roofline_frac_distinct_bytes": chunk_cold_bytes(un, T) / (g_ms * 1e-3) / 1e9 / peak,
                "dense_chunk_roofline_frac_own_bytes": dense_chunk_bytes(T) / (d_ms * 1e-3) / 1e9 / peak,
                "single_frame_call_cold_us": s_ms * 1e3, "single_frame_dense_cold_us": sd_ms * 1e3,
                "single_frame_speedup_vs_own_dense": sd_ms / s_ms,
                "single_frame_roofline_frac": frame_bytes(nz) / (s_ms * 1e-3) / 1e9 / peak,
                "single_frame_dense_roofline_frac": dense_chunk_bytes(1) / (sd_ms * 1e-3) / 1e9 / peak}
            L2.close()
        extra["by_rho"] = by_rho
        streams = {}
        for n in (4, 16):
            L3, sq, wk, wd, nz, un = make(args.rho, n=n)
            c_ms = timed_chunks(L3, sq, wd, 62, 5, cold=True)
            streams[str(n)] = {"chunk_cold_us": c_ms * 1e3, "fps_cold": n * T * 1e3 / c_ms,
                               "per_frame_bytes_gbs": n * T * frame_bytes(nz) / (c_ms * 1e-3) / 1e9}
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
        while cnt < 2 * period and time.perf_counter() - t0 < 20.0:
            rec.step(seq[order[(cnt + 1) % period]])
            cnt += 1
        dt = time.perf_counter() - t0
        cpu = {"value": cnt / dt, "unit": "frames/s", "cores": orc.threads(), "kind": "oracle",
               "sample": f"{cnt} frames of the same sequence through the oracle's Algorithm-1 recurrence (delta path)"}

    if rank == 0:
        line = {
            "metric": "frames_per_sec", "value": fps, "unit": "frames/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "i8", "data": "synthetic",
            "config": {"workload": f"cfg2 delta-FC int8 fc6 {C_IN}->{C_OUT}, rho={args.rho:g}, 1 stream per GPU; one step = "
                                   f"one chunk of {T} consecutive frames (one rrm_step_seq call) of the {FRAMES}-frame "
                                   f"sequence walked back and forth",
                       "frames_per_step": T, "evaluation": EVAL.get(main_variant, "?"),
                       "l2": "flushed before every timed step (256 MiB write); each step timed by its own event pair",
                       "measured_nnz_mean_per_frame": nnz_mean, "measured_density": nnz_mean / C_IN,
                       "distinct_columns_per_chunk": uniq_mean},
            "dense_equiv_gmacs": fps * DENSE_MACS / 1e9,
            "clocks": clocks,
            "e2e": {"value": world * T * 1e3 / e2e_ms, "unit": "frames/s", "h2d_bytes_per_step": T * C_IN,
                    "d2h_bytes_per_step": T * 4 * C_OUT,
                    "call": "rrm_step_seq_host_async per step, one rrm_host_sync after the last step; steps back to back "
                            "(no L2 flush between them, unlike `value`), timed on the host clock",
                    "value_waiting_every_call": world * T * 1e3 / e2e_sync_ms},
            "gpu_launches": args.steps,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": committed_traffic(KERNEL.get(main_variant, "fc_seq_kernel"), args.rho),
                         "peak_kind": f"of {peak_kind}",
                         "kernel": KERNEL.get(main_variant, "?"), "evaluation": EVAL.get(main_variant, "?"),
                         "algorithmic_bytes_per_launch": bytes_launch,
                         "own_bytes_per_launch": own_bytes, "achieved_own": own_bytes / (ms * 1e-3) / 1e9,
                         "frac_own": own_bytes / (ms * 1e-3) / 1e9 / peak,
                         "note": "algorithmic bytes = the delta-FC's per-frame bytes (gathered columns, projection, "
                                 "frames) x frames per launch; own bytes = what the kernel that ran has to move with a "
                                 "cold L2 (dense evaluation: W once for all frames; gather: every distinct column once)"},
            "cpu_baseline": cpu,
            "last_step_stats": st,
        }
        line.update(extra)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
