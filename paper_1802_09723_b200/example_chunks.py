"""Example: an AlexNet-shaped int8 stack over a synthetic video, 32 frames per rrm_net_step_seq call.

    python -m paper_1802_09723_b200.example_chunks [--dense-switch]

Every call hands the library a chunk of consecutive frames; it returns every frame's output.  By default the
library may evaluate a chunk densely when the measured activity of the previous one is high (same results);
without --dense-switch this example keeps it on the delta path (rrm_options.chunk_dense_activity out of reach),
which is also what the profiles of the several-frames kernels were taken with."""
import argparse
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), ".."))
import paper_1802_09723_b200 as rrm  # noqa: E402
import workloads as wl  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--dense-switch", action="store_true")
    ap.add_argument("--chunks", type=int, default=3)
    args = ap.parse_args()
    T = 32
    specs = wl.alexnet_convs("i8")
    video = wl.moving_rect_video(frames=T + 1, hw=227, dtype="i8", seed=51)
    net = rrm.net_from_specs(specs, n=1)
    if not args.dense_switch:
        net.set_options(chunk_dense_activity=2.0)
    frames = torch.from_numpy(np.ascontiguousarray(video)).cuda()
    outs = net.new_output(frames=T)
    out = net.new_output()
    net.keyframe(frames[0], out)
    for k in range(args.chunks):                  # the video forwards, then backwards, ...
        net.step_seq(frames[1:T + 1] if k % 2 == 0 else frames[0:T].flip(0).contiguous(), outs, T)
    torch.cuda.synchronize()
    st = [net.stats(l) for l in range(len(specs))]
    print("last frame: non-zero delta entries per layer", [s["nnz_elems"] for s in st],
          "updated projection pixels", [s["active_out_pixels"] for s in st])
    net.close()


if __name__ == "__main__":
    main()
