"""Shared test helpers (layout conversion between the oracle's [N][C][H][W] arrays and the
library's boundary layouts, uploads).  Holds no inference arithmetic."""
import numpy as np
import torch


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def pack_bits_nhwc(pm1):
    """[N,C,H,W] array of +-1 -> uint32 [N,H,W,ceil(C/32)], bit i of word k = channel 32k+i, 1 = +1."""
    n, c, h, w = pm1.shape
    cw = (c + 31) // 32
    bits = (np.transpose(pm1, (0, 2, 3, 1)) > 0).astype(np.uint32)
    pad = np.zeros((n, h, w, cw * 32), dtype=np.uint32)
    pad[..., :c] = bits
    pad = pad.reshape(n, h, w, cw, 32)
    weights = (np.uint32(1) << np.arange(32, dtype=np.uint32))
    return (pad * weights).sum(axis=-1).astype(np.uint32)


def unpack_bits_nhwc(words, c):
    """Inverse of pack_bits_nhwc -> int64 [N,C,H,W] of +-1."""
    words = np.asarray(words).astype(np.uint32)
    n, h, w, cw = words.shape
    bits = ((words[..., None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(n, h, w, cw * 32)[..., :c]
    return np.transpose(bits.astype(np.int64) * 2 - 1, (0, 3, 1, 2))


def tensor_to_oracle(t, spec_c=None, is_bin=False):
    """GPU tensor in boundary layout -> numpy in the oracle's convention."""
    a = t.cpu().numpy()
    if is_bin:
        return unpack_bits_nhwc(a.view(np.uint32), spec_c)
    return a
