#!/usr/bin/env python
"""Benchmark of the RRM hot path on B200.

Workload of the contract line: the int8 delta-FC configuration (AlexNet-fc6 shape 9216 -> 4096, int32
accumulation, 32-frame sequences whose frames differ in a fraction rho of the inputs, changed entries in runs
of 32).  One "step" = one chunk of 32 consecutive frames of one stream through the whole hot path of the layer
(delta + compaction, sparse product, accumulate + snapshot + output for every frame), i.e. one rrm_step_seq call
= one kernel launch; the reported value is frames per second.  The line also carries, under "conv", compact
results of the convolution configurations (cfg1, cfg3 fp32 / int8, cfg4, cfg5) and, under "by_rho" /
"roofline_delta_fc" / "weight_sparse_fc", the column-gather kernel forced at 1 / 5 / 20 % density and the
weight-sparse form on a pruned matrix.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--rho 0.05] [--chunk 32] [--impl ours|reference]
  python bench.py --workload cfg1|cfg3_f32|cfg3_i8|cfg4|cfg5 [--streams N] [--seq T] [--variant auto|tensor|gather]

Timing: every timed step is preceded by an untimed L2 flush (a 256 MiB device write) and bracketed by its own
CUDA event pair on the launching stream; ms_per_step is the MEDIAN of those K durations (mean, min and max are
printed beside it), max over ranks.  N > 1 runs N independent replicas (one video stream and one layer state
per GPU, no data-path collective): weak scaling.
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


def summarize(times_ms):
    """Median (the reported figure: robust against a few slow early steps), mean, min, max of per-step durations."""
    a = np.asarray(times_ms, dtype=np.float64)
    return {"median": float(np.median(a)), "mean": float(a.mean()), "min": float(a.min()), "max": float(a.max()),
            "n": int(a.size)}


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


_ALU = {}


def alu_peaks():
    """FFMA / dp4a / popc peaks in TMAC/s (T bit-MAC/s for popc), measured once per process by the library's
    micro-kernels (rrm_measure_alu_peak) on the current device."""
    if not _ALU:
        import paper_1802_09723_b200 as rrm
        for k in ("ffma", "dp4a", "popc"):
            _ALU[k] = rrm.measure_alu_peak(k) / 1e12
    return dict(_ALU)


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


# ------------------------------------------------------------------------------------------------
# CPU oracle legs (the only places where bench.py executes anything under oracle/)
# ------------------------------------------------------------------------------------------------
def cpu_fc_baseline(spec, seq, order, budget_s=10.0, max_frames=None):
    """The oracle's Algorithm-1 recurrence and its dense definition on frames of the same sequence, timed on the
    host cores.  Returns (recurrence frames/s, frames, dense frames/s, frames, threads)."""
    from oracle import rrm_oracle as orc
    period = len(order)
    rec = orc.Recurrence([spec])
    rec.step(seq[order[0]])                                   # also promotes the weights once (setup, untimed)
    orc.dense_forward([spec], seq[order[0]])
    t0 = time.perf_counter()
    cnt = 0
    while (max_frames is None or cnt < max_frames) and time.perf_counter() - t0 < budget_s:
        rec.step(seq[order[(cnt + 1) % period]])
        cnt += 1
    dt = time.perf_counter() - t0
    t0 = time.perf_counter()
    dcnt = 0
    while dcnt < max(4, cnt // 4) and time.perf_counter() - t0 < budget_s / 2:
        orc.dense_forward([spec], seq[order[(dcnt + 1) % period]])
        dcnt += 1
    ddt = time.perf_counter() - t0
    return cnt / dt, cnt, dcnt / ddt, dcnt, orc.threads()


def cpu_stack_baseline(specs, video, n, frames=2):
    """ms per frame (of every stream) of the oracle's recurrence and of its dense definition on a stack."""
    from oracle import rrm_oracle as orc
    rec = orc.Recurrence(specs, n=n)
    rec.reset_to(video[0])
    t0 = time.perf_counter()
    for t in range(1, 1 + frames):
        rec.step(video[t])
    ms_rec = (time.perf_counter() - t0) * 1e3 / frames
    t0 = time.perf_counter()
    orc.dense_forward(specs, video[1])
    ms_dense = (time.perf_counter() - t0) * 1e3
    return {"recurrence_ms_per_frame": ms_rec, "dense_ms_per_frame": ms_dense, "value": n * 1e3 / ms_rec,
            "dense_value": n * 1e3 / ms_dense, "unit": "frames/s", "cores": orc.threads(), "kind": "oracle",
            "sample": f"{frames} delta frames after a dense start, and 1 dense frame, of the same video"}


def run_reference(args, rank, world):
    """The CPU oracle, as it stands, on the host cores (rank 0 only).  One reference step = one chunk of --chunk
    frames of the same sequence through the oracle's Algorithm-1 recurrence, as in the GPU arm."""
    if rank != 0:
        return
    import workloads as wl
    from oracle import rrm_oracle as orc
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=FRAMES, rho=args.rho, seed=21)
    order = pingpong(FRAMES)
    period = len(order)
    T = args.chunk
    rec = orc.Recurrence([spec])
    rec.step(seq[0])
    pos = 0

    def chunk():
        nonlocal pos
        for _ in range(T):
            pos += 1
            rec.step(seq[order[pos % period]])

    for _ in range(args.warmup):
        chunk()
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        chunk()
        times.append((time.perf_counter() - t0) * 1e3)
    tm = summarize(times)
    fps = T * 1e3 / tm["median"]
    print(json.dumps({
        "impl": "reference", "metric": "frames_per_sec", "value": fps, "unit": "frames/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": tm["median"], "ms_per_step_stats": tm,
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "i8", "data": "synthetic",
        "config": {"workload": f"cfg2 delta-FC int8 fc6 {C_IN}->{C_OUT}, rho={args.rho:g}, 1 stream; one step = one chunk "
                               f"of {T} consecutive frames", "frames_per_step": T},
        "dense_equiv_gmacs": fps * DENSE_MACS / 1e9,
        "cpu_baseline": {"value": fps, "unit": "frames/s", "cores": orc.threads(), "kind": "oracle",
                         "sample": f"{args.steps} chunks of {T} frames of the same sequence through the oracle's "
                                   f"Algorithm-1 recurrence (weights promoted to int64 once, before the timed region)"},
        "e2e": {"value": fps, "unit": "frames/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------------
# Convolution configurations.  One step = one frame of every stream through rrm_net_step (Algorithm 1, one
# iteration of the frame loop).
# ------------------------------------------------------------------------------------------------
CONV_WORKLOADS = ("cfg1", "cfg3_f32", "cfg3_i8", "cfg4", "cfg5", "cfg3_i8_quiet")


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
    if name == "cfg3_i8_quiet":
        # not one of the contract's configurations: the cfg3 stack on a quieter video (one 24-32 px rectangle moving
        # 1-2 px per frame instead of three of 32-64 px moving 1-4 px), to show how the delta path follows the density
        n = streams or 1
        return (wl.alexnet_convs("i8"), wl.moving_rect_video(frames=frames or 64, hw=227, dtype="i8", seed=33, n=n, n_rect=1,
                                                             side=(24, 32), speed=(1, 2)), n, "i8")
    if name == "cfg4":
        n = streams or 4
        return (wl.resnet18_convs(), wl.moving_rect_video(frames=frames or 64, hw=224, dtype="i8", seed=41, n=n,
                                                          bg_redraw=0.02), n, "i8")
    if name == "cfg5":
        n = streams or 1
        return (wl.xnor_alexnet_convs(), wl.moving_rect_video(frames=frames or 128, hw=227, dtype="i8", seed=51, n=n),
                n, "i8+bin")
    raise SystemExit(f"unknown workload {name}")


def conv_measure(name, variant="auto", steps=60, warmup=5, frames=None, streams=None, seq=None, cpu_frames=0,
                 sample_clocks=True, options=None):
    """Times one convolution configuration: delta steps (cold and warm L2), the library's own dense path, per-layer
    densities, Eq. 9 / Eq. 10, the roofline of the step; optionally chunks of `seq` frames and a CPU oracle sample."""
    import torch
    import workloads as wl
    import paper_1802_09723_b200 as rrm
    specs, video, n, dtype = conv_workload(name, frames, streams)
    F = video.shape[0]
    net = rrm.net_from_specs(specs, n=n, variant=variant)
    if options:
        net.set_options(**options)
    fr = [torch.from_numpy(np.ascontiguousarray(video[t])).cuda() for t in range(F)]
    order = pingpong(F)
    period = len(order)
    out = net.new_output()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    dense_macs = wl.dense_macs(specs) * n

    def timed(call, k, w, cold=True):
        net.keyframe(fr[order[0]], out)
        for i in range(w):
            call(fr[order[(i + 1) % period]], out)
        torch.cuda.synchronize()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(k)]
        for i in range(k):
            if cold:
                flush.fill_(i & 0xff)
            evs[i][0].record(stream)
            call(fr[order[(w + i + 1) % period]], out)
            evs[i][1].record(stream)
        torch.cuda.synchronize()
        return summarize([a.elapsed_time(b) for a, b in evs])

    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0"))) if sample_clocks else None
    if sampler:
        sampler.start()
    tm = timed(net.step, steps, warmup)
    clocks = sampler.stop() if sampler else None
    ms = tm["median"]
    # ---- per-layer counters of the last timed step, Eq. 9 (overall sparsity, MAC-weighted) and Eq. 10 (speedup ratio)
    hbm, hbm_kind = measured_peaks()
    tens, tens_kind = measured_tensor_tmacs()
    alu = alu_peaks()
    unit_bytes = {"f32": 4.0, "i8": 1.0, "bin": 1.0 / 8}
    per_layer, stats = [], []
    tot_active = 0
    num_hat = num_in = den = 0.0
    roof_us = mac_us = byte_us = 0.0
    for l, sp in enumerate(specs):
        st = net.stats(l)
        stats.append(st)
        dense_step = st["variant"] == 3
        # density of the layer input itself (what a sparse engine without RRM would see): non-zero share of the
        # tensor the layer reads (binary tensors have no zeros)
        if sp.dtype == "bin":
            rho_in = 1.0
        else:
            src = net.tensor(sp.src if sp.src >= 0 else l)
            rho_in = float(torch.count_nonzero(src).item()) / src.numel()
        entry = {"layer": sp.name, "dense_macs": st["dense_macs"], "rho_input": rho_in,
                 "variant": {1: "gather", 2: "tensor", 3: "dense"}.get(st["variant"], "?")}
        if dense_step:
            tot_active = None
            entry["note"] = "evaluated densely (measured activity above the switch): no delta counters"
        else:
            if tot_active is not None:
                tot_active += st["active_macs"]
            entry.update({"rho": st["nnz_elems"] / max(1, st["in_elems"]),
                          "active_in_pixels": st["active_in_pixels"] / max(1, st["in_pixels"]),
                          "active_out_pixels": st["active_out_pixels"] / max(1, st["out_pixels"]),
                          "active_macs": st["active_macs"]})
            num_hat += entry["rho"] * st["dense_macs"]
        num_in += rho_in * st["dense_macs"]
        den += st["dense_macs"]
        # roofline of this layer: the slower of (MACs executed at the unit's peak) and (bytes that have to move at the
        # HBM peak).  Bytes: delta rows of the active input pixels once + projection rows of the pixels to update
        # three times (read and write by the convolution, read by the epilogue); weights stay in L2 and are left out.
        macs = st["dense_macs"] if dense_step else st["active_macs"]
        fin = 1.0 if dense_step else st["active_in_pixels"] / max(1, st["in_pixels"])
        fout = 1.0 if dense_step else st["active_out_pixels"] / max(1, st["out_pixels"])
        on_tensor = sp.dtype != "f32" and st["variant"] in (2, 3)
        peak_l = tens if on_tensor else {"f32": alu["ffma"], "i8": alu["dp4a"], "bin": alu["popc"]}[sp.dtype]
        t_mac = macs / (peak_l * 1e12) * 1e6
        nbytes = st["in_pixels"] * fin * sp.c_in * unit_bytes[sp.dtype] + st["out_pixels"] * fout * sp.c_out * 4 * (2 if dense_step else 3)
        t_byte = nbytes / (hbm * 1e9) * 1e6
        entry["roofline_us"] = max(t_mac, t_byte)
        entry["roofline_bound"] = "hbm" if t_byte >= t_mac else ("tensor" if on_tensor else "alu")
        roof_us += max(t_mac, t_byte); mac_us += t_mac; byte_us += t_byte
        per_layer.append(entry)
    all_delta = tot_active is not None
    eq = {"S0_without_rrm": 1.0 - num_in / den,
          "S_with_rrm": (1.0 - num_hat / den) if all_delta else None,
          "eta_eq10": (num_in / num_hat) if all_delta and num_hat > 0 else None,
          "dense_over_active_macs": (dense_macs / tot_active) if all_delta and tot_active else None,
          "note": "Eq. 9: MAC-weighted sparsity of the layer inputs (S0) and of their deltas (S); Eq. 10: eta = sum(rho MACs) / "
                  "sum(rho_hat MACs); dense_over_active_macs uses the exact MAC count instead of Table 1's rho x dense MACs"}
    mac_bound = byte_us < mac_us
    peak = (alu["ffma"] if dtype == "f32" else tens) if mac_bound else hbm
    roofline = {"bound": ("alu" if dtype == "f32" else "tensor") if mac_bound else "hbm",
                "achieved": roof_us * 1e-3 / ms * peak, "peak": peak, "unit": "TMAC/s" if mac_bound else "GB/s",
                "frac": roof_us * 1e-3 / ms, "traffic": None,
                "peak_kind": f"of {('measured by rrm_measure_alu_peak' if dtype == 'f32' else tens_kind) if mac_bound else hbm_kind}",
                "roofline_us_per_step": roof_us, "mac_us": mac_us, "byte_us": byte_us,
                "note": "sum over the layers of max(executed MACs at the unit's peak, algorithmic bytes at the HBM peak) / "
                        "median step time; traffic: no ncu capture of a whole step"}
    tm_warm = timed(net.step, max(8, steps // 2), 3, cold=False)
    tm_dense = timed(net.dense, max(8, steps // 3), 3)
    res = {
        "workload": name, "streams": n, "variant_requested": variant, "frames_in_video": F,
        "ms_per_step": ms, "ms_per_step_stats": tm, "frames_per_sec": n * 1e3 / ms,
        "ms_per_step_warm": tm_warm["median"], "ms_per_step_dense_path": tm_dense["median"],
        "speedup_vs_own_dense": tm_dense["median"] / ms,
        "dense_equiv_gmacs": dense_macs / ms / 1e6,
        "active_macs_last_step": tot_active, "dense_macs_per_step": dense_macs,
        "eq9_eq10": eq, "roofline": roofline, "per_layer_last_step": per_layer, "clocks": clocks, "dtype": dtype,
        "alu_peaks_tmacs": alu,
    }
    # ---- chunks of `seq` consecutive frames per call (rrm_net_step_seq: the frames of a chunk overlap layer by layer)
    if seq and seq > 1:
        Tq = seq
        total = period * Tq // np.gcd(period, Tq)
        walk = torch.stack([fr[order[(i + 1) % period]] for i in range(total)])     # frame i+1 of the walk
        outs = net.new_output(frames=Tq)
        nchunks = total // Tq

        def timed_seq(call, k, w):
            net.keyframe(fr[order[0]], out)
            for i in range(w):
                call(walk[(i % nchunks) * Tq:(i % nchunks + 1) * Tq], outs, Tq)
            torch.cuda.synchronize()
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(k)]
            for i in range(k):
                c = (w + i) % nchunks
                flush.fill_(i & 0xff)
                evs[i][0].record(stream)
                call(walk[c * Tq:(c + 1) * Tq], outs, Tq)
                evs[i][1].record(stream)
            torch.cuda.synchronize()
            return summarize([a.elapsed_time(b) for a, b in evs])["median"]

        steps_q = max(4, steps // Tq)
        # (18 warm-up chunks: a large stack measures its activity with one delta chunk after 15 dense ones, and both
        # chunk graphs are to be captured before the timed region)
        ms_seq = timed_seq(net.step_seq, max(steps_q, 16), 18)
        ms_seq_dense = timed_seq(net.dense_seq, steps_q, 3)
        # the delta path alone: the switches that send high-activity chunks to the dense evaluation out of reach
        keep = net.options()
        net.set_options(chunk_dense_activity=2.0, stack_dense_activity=2.0)
        ms_seq_delta = timed_seq(net.step_seq, max(steps_q, 16), 3)
        net.set_options(chunk_dense_activity=keep["chunk_dense_activity"], stack_dense_activity=keep["stack_dense_activity"])
        res["seq"] = {"frames_per_call": Tq, "ms_per_call": ms_seq, "ms_per_frame_step": ms_seq / Tq,
                      "delta_forced_ms_per_call": ms_seq_delta,
                      "frames_per_sec": n * Tq * 1e3 / ms_seq, "dense_ms_per_call": ms_seq_dense,
                      "dense_frames_per_sec": n * Tq * 1e3 / ms_seq_dense,
                      "speedup_vs_own_dense": ms_seq_dense / ms_seq,
                      "speedup_vs_frame_by_frame": ms * Tq / ms_seq}
    net.close()
    del fr, flush
    torch.cuda.empty_cache()
    if cpu_frames:
        res["cpu_baseline"] = cpu_stack_baseline(specs, video, n, cpu_frames)
    return res


def run_conv(args):
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    options = {}
    for kv in args.opt or []:
        k, v = kv.split("=")
        options[k] = int(v) if k in ("wait_limit", "stack_reprobe") else float(v)
    r = conv_measure(args.workload, args.variant, args.steps, args.warmup, args.frames, args.streams, args.seq,
                     cpu_frames=0 if args.quick else 2, options=options)
    n = r["streams"]
    line = {
        "metric": "frames_per_sec", "value": r["frames_per_sec"], "unit": "frames/s", "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": r["ms_per_step"], "ms_per_step_stats": r["ms_per_step_stats"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": r["dtype"], "data": "synthetic",
        "config": {"workload": f"{args.workload}: {len(r['per_layer_last_step'])} conv layers, {n} stream(s), {r['frames_in_video']}-frame video "
                               f"walked back and forth; one step = one frame of every stream through rrm_net_step",
                   "variant": args.variant,
                   "l2": "flushed before every timed step (256 MiB write); each step timed by its own event pair; median"},
    }
    for k in ("dense_equiv_gmacs", "ms_per_step_warm", "ms_per_step_dense_path", "speedup_vs_own_dense", "active_macs_last_step",
              "dense_macs_per_step", "eq9_eq10", "clocks", "roofline", "per_layer_last_step", "alu_peaks_tmacs", "seq", "cpu_baseline"):
        if k in r:
            line[k] = r[k]
    print(json.dumps(line))


def compact_conv(r):
    """The few figures of a convolution configuration that go into the contract line."""
    out = {k: r[k] for k in ("streams", "variant_requested", "ms_per_step", "frames_per_sec", "ms_per_step_dense_path",
                             "speedup_vs_own_dense", "dense_equiv_gmacs")}
    out["rho_per_layer"] = [round(e["rho"], 4) if "rho" in e else None for e in r["per_layer_last_step"]]
    out["active_out_pixels_per_layer"] = [round(e["active_out_pixels"], 4) if "active_out_pixels" in e else None
                                          for e in r["per_layer_last_step"]]
    out["variant_per_layer"] = [e["variant"] for e in r["per_layer_last_step"]]
    out["S"] = r["eq9_eq10"]["S_with_rrm"]
    out["S0"] = r["eq9_eq10"]["S0_without_rrm"]
    out["eta"] = r["eq9_eq10"]["eta_eq10"]
    out["dense_over_active_macs"] = r["eq9_eq10"]["dense_over_active_macs"]
    out["roofline_frac"] = r["roofline"]["frac"]
    out["roofline_bound"] = r["roofline"]["bound"]
    if "seq" in r:
        q = r["seq"]
        out["chunk"] = {"frames_per_call": q["frames_per_call"], "ms_per_frame": q["ms_per_frame_step"],
                        "delta_forced_ms_per_frame": q["delta_forced_ms_per_call"] / q["frames_per_call"],
                        "dense_ms_per_frame": q["dense_ms_per_call"] / q["frames_per_call"], "frames_per_sec": q["frames_per_sec"],
                        "speedup_vs_own_dense": q["speedup_vs_own_dense"], "speedup_vs_frame_by_frame": q["speedup_vs_frame_by_frame"]}
    if "cpu_baseline" in r:
        out["cpu_baseline"] = r["cpu_baseline"]
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=310, help="timed steps; one step = one chunk of --chunk frames")
    ap.add_argument("--warmup", type=int, default=31)
    ap.add_argument("--rho", type=float, default=0.05)
    ap.add_argument("--chunk", type=int, default=FRAMES, help="frames per rrm_step_seq call")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="skip the secondary sweeps and the CPU legs (profiling runs)")
    ap.add_argument("--workload", default="cfg2", choices=("cfg2",) + CONV_WORKLOADS,
                    help="cfg2 (default) is the contract line; the others are the convolution configurations")
    ap.add_argument("--variant", default="auto", choices=["auto", "gather", "tensor", "dense", "sparse_w"],
                    help="rrm_layer_desc.variant of the timed object (default: the library chooses)")
    ap.add_argument("--pruned", type=float, default=None, help="contract workload on a magnitude-pruned matrix (fraction of weights kept); "
                                                               "for profiling the weight-sparse form: --pruned 0.1 --variant sparse_w")
    ap.add_argument("--frames", type=int, default=None, help="frames of the synthetic video (convolution workloads)")
    ap.add_argument("--streams", type=int, default=None, help="independent videos per call (convolution workloads)")
    ap.add_argument("--opt", action="append", help="rrm_options field=value (convolution workloads), e.g. --opt layer_dense_activity=0.9")
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
        if args.steps == 310:
            args.steps, args.warmup = 20, 3
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
    spec = wl.fc6_i8_pruned(keep=args.pruned)[0] if args.pruned else wl.fc6_i8()[0]
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

    def make(rho, n=1, variant="auto", weights=None):
        """Layer + the endless back-and-forth walk over the 32-frame sequence, laid out so that chunk k
        is rows [k*T, (k+1)*T) of one device array (whole number of periods, so it wraps seamlessly)."""
        desc = rrm.desc_from_spec(spec, n=n, variant=variant)
        layer = rrm.Net([desc], [W if weights is None else weights], [B])
        seq = wl.fc_run_sequence(frames=FRAMES, rho=rho, seed=21 + rank, n=n)
        total = period * T // np.gcd(period, T)
        walk = np.stack([seq[order[(i + 1) % period]] for i in range(total)])      # frame i+1 of the walk
        nnz = np.array([np.count_nonzero(seq[order[(i + 1) % period]] != seq[order[i % period]]) / n
                        for i in range(period)])
        # distinct weight columns one chunk touches (what a cold L2 must fetch; the streams share W), mean over the chunks
        uniq = []
        for k in range(total // T):
            touched = np.zeros(C_IN, dtype=bool)
            for i in range(k * T, (k + 1) * T):
                touched |= np.any(seq[order[(i + 1) % period]] != seq[order[i % period]], axis=0).reshape(-1)
            uniq.append(int(touched.sum()))
        return layer, seq, walk, torch.from_numpy(walk).cuda(), float(nnz.mean()), float(np.mean(uniq))

    def timed_chunks(layer, seq, walk_dev, steps, warmup, cold, dense=False, frames_per_call=None):
        """Per-call durations (ms) of rrm_step_seq (or rrm_dense_seq) over chunks of the walk; returns their summary
        with the median reduced to the max over ranks."""
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
            tm = summarize([a.elapsed_time(b) for a, b in evs])
        else:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(steps):
                k = (warmup + i) % nchunks
                call(walk_dev[k * tc:(k + 1) * tc], Y, tc)
            b.record(stream)
            barrier()
            tm = summarize([a.elapsed_time(b) / steps])
        tm["median"] = reduce_max(tm["median"])
        return tm

    def timed_single(layer, seq, frames, steps, warmup, cold, dense=False):
        """Median ms per rrm_step (one frame per call)."""
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
        return reduce_max(summarize([a.elapsed_time(b) for a, b in evs])["median"])

    def frame_bytes(nnz_mean):
        # per frame: gathered weight columns + read/modify/write of P + output + X_t, snapshot read, snapshot write
        return nnz_mean * C_OUT + 8 * C_OUT + 4 * C_OUT + 3 * C_IN

    def dense_chunk_bytes(frames):
        # the dense evaluation of a chunk: W once, the frames, outputs, stored projection, snapshot
        return C_IN * C_OUT + (frames + 1) * C_IN + frames * 4 * C_OUT + 4 * C_OUT

    def chunk_cold_bytes(uniq_cols, frames, n=1):
        # what one gather launch must fetch with a cold L2: every distinct column once (the streams share W), the
        # frames, per-frame projection deltas (write + read) and outputs, the stored projections
        return uniq_cols * C_OUT + n * ((frames + 2) * C_IN + frames * 12 * C_OUT + 8 * C_OUT)

    EVAL = {1: "column gather (the delta method)", 3: "dense on the tensor cores, W read once (rows x measured density of "
                                                     "the previous chunk >= rrm_options.fc_dense_rows)"}
    KERNEL = {1: "fc_seq_kernel", 3: "fc_tc_kernel"}
    peak, peak_kind = measured_peaks()

    # ---- primary: one stream per GPU, chunks of T frames per call, rho as asked, cold L2, per-step events
    layer, seq, walk, walk_dev, nnz_mean, uniq_mean = make(args.rho, variant=args.variant)
    # (setup, untimed and before the W warm-up steps: lets the library measure the density and settle on its
    # evaluation, allocate its pinned read-back buffer and scratch)
    timed_chunks(layer, seq, walk_dev, 4, 4, cold=True)
    sampler = ClockSampler(local)
    sampler.start()
    tm = timed_chunks(layer, seq, walk_dev, args.steps, args.warmup, cold=True)
    clocks = sampler.stop()
    ms = tm["median"]
    fps = whole_job_rate(T, ms, world)
    st = layer.stats(0)
    main_variant = st["variant"]
    own_bytes = dense_chunk_bytes(T) if main_variant == 3 else chunk_cold_bytes(uniq_mean, T)
    achieved = own_bytes / (ms * 1e-3) / 1e9

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
    delta_fc = {}
    if not args.quick:
        by_rho = {}
        for rho in RHOS:
            L2, sq, wk, wd, nz, un = make(rho)
            fr = [torch.from_numpy(sq[t]).cuda() for t in range(FRAMES)]
            c_ms = timed_chunks(L2, sq, wd, 93, 10, cold=True)["median"]
            variant = L2.stats(0)["variant"]
            d_ms = timed_chunks(L2, sq, wd, 31, 3, cold=True, dense=True)["median"]
            s_ms = timed_single(L2, sq, fr, 186, 31, cold=True)
            sd_ms = timed_single(L2, sq, fr, 93, 10, cold=True, dense=True)
            LG = make(rho, variant="gather")[0]            # the column-gather kernel whatever the density
            g_ms = timed_chunks(LG, sq, wd, 93, 10, cold=True)["median"]
            LG.close()
            own = dense_chunk_bytes(T) if variant == 3 else chunk_cold_bytes(un, T)
            by_rho[f"{rho:g}"] = {
                "nnz_mean_per_frame": nz, "distinct_columns_per_chunk": un,
                "chunk_evaluation": EVAL.get(variant, "?"), "chunk_cold_us": c_ms * 1e3,
                "fps_cold": T * 1e3 / c_ms, "gmacs_dense_equiv_cold": T * DENSE_MACS / c_ms / 1e6,
                "chunk_roofline_frac_own_bytes": own / (c_ms * 1e-3) / 1e9 / peak,
                "dense_chunk_cold_us": d_ms * 1e3,
                "dense_chunk_roofline_frac_own_bytes": dense_chunk_bytes(T) / (d_ms * 1e-3) / 1e9 / peak,
                "speedup_vs_own_dense_chunk": d_ms / c_ms,
                "gather_chunk_cold_us": g_ms * 1e3, "gather_speedup_vs_own_dense_chunk": d_ms / g_ms,
                "single_frame_call_cold_us": s_ms * 1e3, "single_frame_dense_cold_us": sd_ms * 1e3,
                "single_frame_speedup_vs_own_dense": sd_ms / s_ms,
                "single_frame_roofline_frac": frame_bytes(nz) / (s_ms * 1e-3) / 1e9 / peak,
                "single_frame_dense_roofline_frac": dense_chunk_bytes(1) / (sd_ms * 1e-3) / 1e9 / peak}
            # the contract's kernel (3), the column gather, on its own: the bytes it must fetch from HBM with a cold
            # L2 (every distinct column of the chunk once) against the HBM peak, and the bytes it serves to the SMs
            # (every frame's columns; repeats come from L2, so this is a rate, not a fraction of the HBM peak)
            delta_fc[f"{rho:g}"] = {
                "kernel": "fc_seq_kernel", "streams": 1, "frames_per_launch": T, "us_per_launch": g_ms * 1e3,
                "distinct_cold_bytes": chunk_cold_bytes(un, T), "per_frame_bytes_x_frames": frame_bytes(nz) * T,
                "frac_distinct_cold_bytes": chunk_cold_bytes(un, T) / (g_ms * 1e-3) / 1e9 / peak,
                "served_gbs_l2_and_hbm": frame_bytes(nz) * T / (g_ms * 1e-3) / 1e9,
                "faster_than_own_dense_chunk": d_ms / g_ms}
            L2.close()
        extra["by_rho"] = by_rho
        # more streams per call: the library's choice, and the column gather forced (the multi-stream operating point
        # of the delta-FC kernel)
        streams = {}
        for n in (4, 16):
            L3, sq, wk, wd, nz, un = make(args.rho, n=n)
            c_ms = timed_chunks(L3, sq, wd, 31, 5, cold=True)["median"]
            v3 = L3.stats(0)["variant"]
            L3.close()
            LG, sq, wk, wd, nz, un = make(args.rho, n=n, variant="gather")
            g_ms = timed_chunks(LG, sq, wd, 31, 5, cold=True)["median"]
            LG.close()
            streams[str(n)] = {"chunk_cold_us": c_ms * 1e3, "fps_cold": n * T * 1e3 / c_ms,
                               "chunk_evaluation": EVAL.get(v3, "?"), "gather_chunk_cold_us": g_ms * 1e3,
                               "gather_fps_cold": n * T * 1e3 / g_ms}
            delta_fc[f"{args.rho:g}_x{n}_streams"] = {
                "kernel": "fc_seq_kernel", "streams": n, "frames_per_launch": T, "us_per_launch": g_ms * 1e3,
                "distinct_cold_bytes": chunk_cold_bytes(un, T, n), "per_frame_bytes_x_frames": n * T * frame_bytes(nz),
                "frac_distinct_cold_bytes": chunk_cold_bytes(un, T, n) / (g_ms * 1e-3) / 1e9 / peak,
                "served_gbs_l2_and_hbm": n * T * frame_bytes(nz) / (g_ms * 1e-3) / 1e9}
        extra["streams_per_call"] = streams
        delta_fc["note"] = ("column gather forced (variant GATHER), one launch per chunk, cold L2 before every launch.  "
                            "frac_distinct_cold_bytes = bytes the launch must fetch from HBM / time / measured HBM peak; "
                            "served_gbs = all gathered bytes (repeats served by L2) per second: a rate, not an HBM fraction")

    # ---- the same delta-FC kernels on a layer large enough to be bound by bytes: 16384 -> 16384 int8 (268 MB of
    # weights, twice the L2: gathered columns come from HBM whatever ran before), one frame per call (rrm_step) and a
    # chunk of 8 frames, the column gather forced.  fc6's 37.7 MB take 5.8 us at the HBM peak, less than the fixed cost
    # of a launch, which is why its fractions stay low; this row shows what the kernels reach once the bytes dominate.
    if not args.quick and rank == 0 and world == 1:
        try:
            CB, KB = 16384, 16384
            big = wl.fc6_i8(seed=7, c_in=CB, c_out=KB)[0]
            Wb = torch.from_numpy(big.weight).cuda()
            Bb = torch.from_numpy(big.bias).cuda()
            rows = {}
            for rho in (0.05, 0.20):
                Lb = rrm.Net([rrm.desc_from_spec(big, n=1, variant="gather")], [Wb], [Bb])
                sq = wl.fc_run_sequence(frames=9, c_in=CB, rho=rho, seed=77)
                fr = [torch.from_numpy(sq[t]).cuda() for t in range(9)]
                ordb = pingpong(9)
                Yb = Lb.new_output()
                Lb.keyframe(fr[0], Yb)
                for i in range(4):
                    Lb.step(fr[ordb[(i + 1) % len(ordb)]], Yb)
                torch.cuda.synchronize()
                evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(24)]
                for i in range(24):
                    flush.fill_(i & 0xff)
                    evs[i][0].record(stream)
                    Lb.step(fr[ordb[(5 + i) % len(ordb)]], Yb)
                    evs[i][1].record(stream)
                torch.cuda.synchronize()
                us = summarize([a.elapsed_time(b) for a, b in evs])["median"] * 1e3
                nnz = float(np.mean([np.count_nonzero(sq[ordb[(k + 1) % len(ordb)]] != sq[ordb[k % len(ordb)]]) for k in range(len(ordb))]))
                nbytes = nnz * KB + 12 * KB + 3 * CB
                rows[f"{rho:g}"] = {"kernel": "fc_delta_i8_kernel", "frames_per_launch": 1, "nnz_mean_per_frame": nnz,
                                    "us_per_launch": us, "algorithmic_bytes_per_launch": nbytes,
                                    "achieved_gbs": nbytes / (us * 1e-6) / 1e9, "frac": nbytes / (us * 1e-6) / 1e9 / peak}
                # chunks of Tb frames per launch (fc_seq_kernel): distinct columns of the chunk once from HBM, repeats from L2
                for Tb in (4, 8):
                    walkb = np.stack([sq[ordb[(i + 1) % len(ordb)]] for i in range(len(ordb) * Tb)])
                    wdb = torch.from_numpy(walkb).cuda()
                    ncb = wdb.shape[0] // Tb
                    Ycb = Lb.new_output(frames=Tb)
                    Lb.keyframe(fr[0], Yb)
                    for i in range(3):
                        Lb.step_seq(wdb[(i % ncb) * Tb:(i % ncb + 1) * Tb], Ycb, Tb)
                    torch.cuda.synchronize()
                    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(16)]
                    for i in range(16):
                        k = (3 + i) % ncb
                        flush.fill_(i & 0xff)
                        evs[i][0].record(stream)
                        Lb.step_seq(wdb[k * Tb:(k + 1) * Tb], Ycb, Tb)
                        evs[i][1].record(stream)
                    torch.cuda.synchronize()
                    usc = summarize([a.elapsed_time(b) for a, b in evs])["median"] * 1e3
                    uniq = []
                    for k in range(ncb):
                        touched = np.zeros(CB, dtype=bool)
                        for i in range(k * Tb, (k + 1) * Tb):
                            prev = walkb[i - 1] if i else sq[ordb[0]]
                            touched |= (walkb[i] != prev).reshape(-1)
                        uniq.append(int(touched.sum()))
                    db = float(np.mean(uniq)) * KB + Tb * (12 * KB + CB) + 2 * CB
                    rows[f"{rho:g}_chunk{Tb}"] = {"kernel": "fc_seq_kernel", "frames_per_launch": Tb, "us_per_launch": usc,
                                                  "distinct_cold_bytes": db, "per_frame_bytes_x_frames": Tb * nbytes,
                                                  "frac_distinct_cold_bytes": db / (usc * 1e-6) / 1e9 / peak,
                                                  "served_gbs_l2_and_hbm": Tb * nbytes / (usc * 1e-6) / 1e9}
                    del wdb
                Lb.close()
            rows["note"] = (f"int8 FC {CB}->{KB} (268 MB of weights, larger than L2), one stream, column gather forced, cold L2, "
                            f"medians; one frame per rrm_step call (bytes = gathered columns + projection + frames, all from HBM) "
                            f"and chunks of 4 / 8 frames per rrm_step_seq call (distinct columns once from HBM)")
            extra["roofline_delta_fc_large_layer"] = rows
            del Wb, Bb
            torch.cuda.empty_cache()
        except Exception as e:  # noqa: BLE001
            extra["roofline_delta_fc_large_layer"] = {"error": str(e)}

    # ---- weight-sparse x delta-sparse (Sec. 3.5 / 4.3): fc6 magnitude-pruned to 10 %, the weight-sparse form against
    # the column gather and the dense tensor-core pass on the same pruned matrix
    if not args.quick:
        pr = wl.fc6_i8_pruned(keep=0.10)[0]
        Wp = torch.from_numpy(pr.weight).cuda()
        kept = float(np.mean(pr.weight != 0))
        groups = float(np.mean(np.any(pr.weight.reshape(C_OUT // 4, 4, C_IN) != 0, axis=1)))   # non-zero groups of four outputs
        sw = {"weights_kept": kept, "nonzero_groups_of_4": groups,
              "bytes_per_gathered_column": {"dense": C_OUT, "weight_sparse": groups * C_OUT + 32 * (C_OUT // 512)}}
        for rho in RHOS:
            row = {}
            for nm, var in (("weight_sparse", "sparse_w"), ("column_gather", "gather"), ("library_auto", "auto")):
                Lp, sq, wk, wd, nz, un = make(rho, variant=var, weights=Wp)
                row[nm + "_us"] = timed_chunks(Lp, sq, wd, 62, 10, cold=True)["median"] * 1e3
                Lp.close()
            row["nnz_mean_per_frame"] = nz
            row["weight_sparse_bytes_per_chunk"] = T * (nz * sw["bytes_per_gathered_column"]["weight_sparse"] + 12 * C_OUT + 3 * C_IN)
            row["column_gather_bytes_per_chunk"] = T * frame_bytes(nz)
            row["speedup_vs_column_gather"] = row["column_gather_us"] / row["weight_sparse_us"]
            row["speedup_vs_library_auto"] = row["library_auto_us"] / row["weight_sparse_us"]
            sw[f"{rho:g}"] = row
        Lp, sq, wk, wd, nz, un = make(args.rho, n=16, variant="sparse_w", weights=Wp)
        s16 = timed_chunks(Lp, sq, wd, 31, 5, cold=True)["median"] * 1e3
        Lp.close()
        Lp, sq, wk, wd, nz, un = make(args.rho, n=16, variant="gather", weights=Wp)
        g16 = timed_chunks(Lp, sq, wd, 31, 5, cold=True)["median"] * 1e3
        Lp.close()
        Lp, sq, wk, wd, nz, un = make(args.rho, n=16, variant="auto", weights=Wp)
        a16 = timed_chunks(Lp, sq, wd, 31, 5, cold=True)["median"] * 1e3
        Lp.close()
        sw[f"{args.rho:g}_x16_streams"] = {"weight_sparse_us": s16, "column_gather_us": g16, "library_auto_us": a16,
                                           "speedup_vs_column_gather": g16 / s16, "speedup_vs_library_auto": a16 / s16}
        sw["note"] = ("one launch per 32-frame chunk, cold L2, median; library_auto = what RRM_VARIANT_AUTO runs on the pruned "
                      "matrix stored densely (column gather or the dense tensor-core chunk)")
        extra["weight_sparse_fc"] = sw
        del Wp

    # ---- the convolution configurations, compact (rank 0, one GPU): cfg1, cfg3 int8, cfg4 with the sparse product forced
    # and as the library chooses
    conv = None
    if rank == 0 and world == 1 and not args.quick:
        conv = {}
        for key, name, variant, fr_n, cpu_n in (("cfg1", "cfg1", "auto", None, 2), ("cfg3_f32", "cfg3_f32", "auto", 16, 1),
                                                ("cfg3_i8", "cfg3_i8", "auto", 16, 2), ("cfg3_i8_quiet_video", "cfg3_i8_quiet", "auto", 16, 0),
                                                ("cfg5", "cfg5", "auto", 16, 1),
                                                ("cfg4_delta_forced", "cfg4", "tensor", 8, 1), ("cfg4_auto", "cfg4", "auto", 8, 0)):
            try:
                conv[key] = compact_conv(conv_measure(name, variant, steps=30, warmup=5, frames=fr_n, cpu_frames=cpu_n,
                                                      sample_clocks=False, seq=None if name == "cfg4" else FRAMES))
            except Exception as e:  # noqa: BLE001
                conv[key] = {"error": str(e)}
        conv["note"] = ("one step = one frame of every stream through rrm_net_step, median of 30 cold-L2 steps; S / S0 / eta: "
                        "Eq. 9 and Eq. 10 from the measured per-layer densities; chunk: 32 consecutive frames per rrm_net_step_seq "
                        "call (as the library chooses; delta_forced: its density switches out of reach) / rrm_net_dense_seq call (dense), cold L2, median, per frame; cfg3_i8_quiet_video: the cfg3 "
                        "stack on a quieter video (one 24-32 px rectangle moving 1-2 px per frame), not a contract configuration; "
                        "cpu_baseline: the oracle on the host cores")

    # ---- CPU oracle on the host cores (rank 0, N = 1 only): a bounded sample of the same workload
    cpu = None
    if rank == 0 and world == 1 and not args.quick:
        r_fps, r_n, d_fps, d_n, cores = cpu_fc_baseline(spec, seq, order, budget_s=10.0, max_frames=4 * period)
        cpu = {"value": r_fps, "unit": "frames/s", "cores": cores, "kind": "oracle",
               "sample": f"{r_n} frames of the same sequence through the oracle's Algorithm-1 recurrence (delta path); "
                         f"weights promoted to int64 once, outside the timed region",
               "dense_value": d_fps, "dense_sample": f"{d_n} frames through the oracle's dense definition (Eq. 3)"}

    if rank == 0:
        line = {
            "metric": "frames_per_sec", "value": fps, "unit": "frames/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "ms_per_step_stats": tm, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "i8", "data": "synthetic",
            "config": {"workload": f"cfg2 delta-FC int8 fc6 {C_IN}->{C_OUT}, rho={args.rho:g}, 1 stream per GPU; one step = "
                                   f"one chunk of {T} consecutive frames (one rrm_step_seq call) of the {FRAMES}-frame "
                                   f"sequence walked back and forth",
                       "frames_per_step": T, "evaluation": EVAL.get(main_variant, "?"),
                       "l2": "flushed before every timed step (256 MiB write); each step timed by its own event pair; "
                             "ms_per_step is the median",
                       "measured_nnz_mean_per_frame": nnz_mean, "measured_density": nnz_mean / C_IN,
                       "distinct_columns_per_chunk": uniq_mean},
            "dense_equiv_gmacs": fps * DENSE_MACS / 1e9,
            "clocks": clocks,
            "e2e": {"value": world * T * 1e3 / e2e_ms, "unit": "frames/s", "h2d_bytes_per_step": T * C_IN,
                    "d2h_bytes_per_step": T * 4 * C_OUT,
                    "call": "rrm_step_seq_host_async per step, one rrm_host_sync after the last step; steps back to back "
                            "(no L2 flush between them, unlike `value`: W stays L2-resident), timed on the host clock",
                    "value_waiting_every_call": world * T * 1e3 / e2e_sync_ms},
            "gpu_launches": args.steps,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": committed_traffic(KERNEL.get(main_variant, "fc_seq_kernel"), args.rho),
                         "peak_kind": f"of {peak_kind}",
                         "kernel": KERNEL.get(main_variant, "?"), "evaluation": EVAL.get(main_variant, "?"),
                         "algorithmic_bytes_per_launch": own_bytes,
                         "note": "bytes the kernel that ran must move with a cold L2 (dense evaluation: W once for all "
                                 "frames + frames, outputs, state; column gather: every distinct column of the chunk once "
                                 "+ frames, per-frame projection deltas, outputs) / median launch duration"},
            "roofline_delta_fc": delta_fc or None,
            "cpu_baseline": cpu,
            "conv": conv,
            "last_step_stats": st,
        }
        line.update(extra)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
