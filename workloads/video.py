"""Seeded synthetic frame sequences (inputs only; no inference arithmetic).

These stand in for the real videos the paper measured on: what matters for the
method is that most of a frame is bit-identical to the previous one and that the
changed part is spatially clustered.
"""
import numpy as np


def _rng(seed):
    return np.random.Generator(np.random.Philox(seed))


def _draw(rng, shape, dtype):
    if dtype == "f32_relu":                      # max(0, N(0,1))
        return np.maximum(rng.standard_normal(shape), 0.0).astype(np.float32)
    if dtype == "f32":                           # pixels in [0,1)
        return rng.random(shape, dtype=np.float32)
    if dtype == "i8":                            # post-ReLU quantised, [0,127]
        return rng.integers(0, 128, size=shape).astype(np.int8)
    if dtype == "pm1":                           # +-1 stored as int8
        return (rng.integers(0, 2, size=shape) * 2 - 1).astype(np.int8)
    raise ValueError(dtype)


def block_redraw_sequence(frames=8, c=64, hw=56, frac=0.10, block=8, dtype="f32_relu", seed=11, n=1):
    """[frames, n, c, hw, hw].  Frame 0 is fully random; every later frame re-draws
    ceil(frac*hw*hw/block^2) randomly placed (unaligned, possibly overlapping)
    block x block spatial patches over all channels; everything else is a bit copy."""
    rng = _rng(seed)
    out = np.empty((frames, n, c, hw, hw), dtype=_draw(rng, (1,), dtype).dtype)
    out[0] = _draw(rng, (n, c, hw, hw), dtype)
    nblk = int(np.ceil(frac * hw * hw / (block * block)))
    for t in range(1, frames):
        out[t] = out[t - 1]
        for s in range(n):
            for _ in range(nblk):
                y = int(rng.integers(0, hw - block + 1))
                x = int(rng.integers(0, hw - block + 1))
                out[t, s, :, y:y + block, x:x + block] = _draw(rng, (c, block, block), dtype)
    return out


def fc_run_sequence(frames=32, c_in=9216, rho=0.05, run=32, seed=21, n=1, aligned=False):
    """[frames, n, c_in] int8 in [0,127].  Per frame round(rho*c_in/run) non-overlapping
    runs of `run` consecutive entries are re-drawn uniformly (a re-draw may repeat the
    old value, so the realised delta density is slightly below rho)."""
    rng = _rng(seed)
    out = np.empty((frames, n, c_in), dtype=np.int8)
    out[0] = _draw(rng, (n, c_in), "i8")
    nruns = int(round(rho * c_in / run))
    for t in range(1, frames):
        out[t] = out[t - 1]
        for s in range(n):
            taken = np.zeros(c_in, dtype=bool)
            placed = 0
            while placed < nruns:
                if aligned:
                    st = int(rng.integers(0, c_in // run)) * run
                else:
                    st = int(rng.integers(0, c_in - run + 1))
                if taken[st:st + run].any():
                    continue
                taken[st:st + run] = True
                out[t, s, st:st + run] = _draw(rng, (run,), "i8")
                placed += 1
    return out


def moving_rect_video(frames=64, hw=227, dtype="f32", seed=31, n=1, n_rect=3,
                      side=(32, 64), speed=(1, 4), bg_redraw=0.0):
    """[frames, n, 3, hw, hw].  Static uniform-noise background; `n_rect` rectangles
    (side 32..64 px, each carrying its own fixed noise texture) move 1..4 px per frame
    per axis and reflect at the borders.  Static pixels are exactly equal across
    frames.  `bg_redraw` > 0 additionally re-draws that fraction of background pixels
    (all 3 channels) per frame; the re-drawn values persist.  Each of the n streams is
    an independent video (its own seed offset)."""
    kind = "f32" if dtype == "f32" else "i8"
    out = None
    for s in range(n):
        rng = _rng(seed * 1000 + s)
        bg = _draw(rng, (3, hw, hw), kind)
        if out is None:
            out = np.empty((frames, n, 3, hw, hw), dtype=bg.dtype)
        rects = []
        for _ in range(n_rect):
            sh = int(rng.integers(side[0], side[1] + 1))
            sw = int(rng.integers(side[0], side[1] + 1))
            tex = _draw(rng, (3, sh, sw), kind)
            y = int(rng.integers(0, hw - sh + 1))
            x = int(rng.integers(0, hw - sw + 1))
            vy = int(rng.integers(speed[0], speed[1] + 1)) * (1 if rng.random() < 0.5 else -1)
            vx = int(rng.integers(speed[0], speed[1] + 1)) * (1 if rng.random() < 0.5 else -1)
            rects.append([tex, y, x, vy, vx, sh, sw])
        for t in range(frames):
            if t > 0:
                if bg_redraw > 0:
                    m = rng.random((hw, hw)) < bg_redraw
                    cnt = int(m.sum())
                    bg[:, m] = _draw(rng, (3, cnt), kind)
                for r in rects:
                    tex, y, x, vy, vx, sh, sw = r
                    y += vy
                    x += vx
                    if y < 0:
                        y, vy = -y, -vy
                    if y > hw - sh:
                        y, vy = 2 * (hw - sh) - y, -vy
                    if x < 0:
                        x, vx = -x, -vx
                    if x > hw - sw:
                        x, vx = 2 * (hw - sw) - x, -vx
                    r[1:5] = [y, x, vy, vx]
            f = bg.copy()
            for tex, y, x, vy, vx, sh, sw in rects:
                f[:, y:y + sh, x:x + sw] = tex
            out[t, s] = f
    return out
