"""Layer-stack descriptions and random-init weights (no inference arithmetic here).

A network is a list of LayerSpec.  Tensor 0 is the network input; layer l produces
tensor l+1.  `src` names the tensor a layer reads, `res` (or -1) a tensor that is
added to the requantised projection before the activation (ResNet shortcut).

Nonlinear map f of a layer, in order: [per-channel affine] -> [requant by `shift`] -> [+ res] -> act -> pool,
except act == "sign", where pooling comes first and the sign is taken last.
`shift == -1` on an integer layer means "emit the raw int32 projection".
The per-channel affine (`bn_scale`, `bn_shift`, both None = absent) is an explicit, unfolded batch
normalisation at inference: fp32 layers y = scale * P + shift; int8 layers use integer multipliers and
offsets inside the requantisation, q = clamp((P * scale + shift + 2^(s-1)) >> s, -127, 127).
"""
from dataclasses import dataclass, field
import math
import numpy as np


@dataclass
class LayerSpec:
    kind: str            # "conv" | "fc"
    dtype: str           # "f32" | "i8" | "bin"  (type of the layer's input and weights)
    c_in: int
    h: int
    w: int
    c_out: int
    kh: int = 1
    kw: int = 1
    stride: int = 1
    pad: int = 0
    act: str = "none"    # "none" | "relu" | "sign"
    pool: tuple = None   # (k, s, p) max-pool or None
    shift: int = -1      # int8 requant shift (power-of-two scale); -1: raw int32 out
    theta: int = 0       # sign threshold
    src: int = -1        # input tensor index; -1 means "previous layer's output"
    res: int = -1        # residual tensor index or -1
    name: str = ""
    weight: np.ndarray = field(default=None, repr=False)   # [c_out, c_in, kh, kw]
    bias: np.ndarray = field(default=None, repr=False)     # [c_out] f32 or int32
    bn_scale: np.ndarray = field(default=None, repr=False)  # [c_out] f32 (fp32 layers) or int32 multipliers (int8 layers), or None
    bn_shift: np.ndarray = field(default=None, repr=False)  # [c_out] f32 or int32 offsets, or None


def out_hw(s: LayerSpec):
    """Spatial size of the projection and of the layer's output tensor."""
    ph = (s.h + 2 * s.pad - s.kh) // s.stride + 1
    pw = (s.w + 2 * s.pad - s.kw) // s.stride + 1
    if s.pool is None:
        return (ph, pw), (ph, pw)
    k, st, p = s.pool
    return (ph, pw), ((ph + 2 * p - k) // st + 1, (pw + 2 * p - k) // st + 1)


def tensor_shapes(layers, n=1):
    """[(n, c, h, w)] for tensor 0..L."""
    l0 = layers[0]
    shapes = [(n, l0.c_in, l0.h, l0.w)]
    for s in layers:
        _, (oh, ow) = out_hw(s)
        shapes.append((n, s.c_out, oh, ow))
    return shapes


def dense_macs(layers):
    tot = 0
    for s in layers:
        (ph, pw), _ = out_hw(s)
        tot += ph * pw * s.c_out * s.c_in * s.kh * s.kw
    return tot


def _resolve_src(layers):
    for i, s in enumerate(layers):
        if s.src < 0:
            s.src = i
    return layers


def _rng(seed):
    return np.random.Generator(np.random.Philox(seed))


def _he_f32(rng, s: LayerSpec):
    fan_in = s.c_in * s.kh * s.kw
    w = rng.standard_normal((s.c_out, s.c_in, s.kh, s.kw)).astype(np.float32)
    return (w * np.float32(math.sqrt(2.0 / fan_in))).astype(np.float32)


def _quantise_i8(w):
    m = float(np.max(np.abs(w)))
    q = np.rint(w.astype(np.float64) / m * 127.0)
    return np.clip(q, -127, 127).astype(np.int8)


def _pick_shift(s: LayerSpec, wq):
    """Power-of-two output scale from weight statistics only (no forward pass):
    projection std ~ sqrt(fan_in * E[w^2]) * rms(x); the shift maps that to the
    same rms the input is assumed to have, so activations neither die nor saturate."""
    fan_in = s.c_in * s.kh * s.kw
    e_w2 = float(np.mean(wq.astype(np.float64) ** 2))
    return max(0, int(round(math.log2(math.sqrt(fan_in * e_w2)))))


def _fill(layers, seed, bias_std=0.1):
    """Random-init weights, biases, requant shifts and sign thresholds.

    Everything is derived from weight statistics alone.  The bias of an int8 layer
    that reads the raw frame (tensor 0, pixels in [0,127]) folds in a mean-64 input
    centring, bias_c = -64 * sum(w_c), as a folded input normalisation would."""
    rng = _rng(seed)
    for s in layers:
        fan_in = s.c_in * s.kh * s.kw
        if s.dtype == "f32":
            s.weight = _he_f32(rng, s)
            s.bias = (rng.standard_normal(s.c_out) * bias_std).astype(np.float32)
            continue
        if s.dtype == "i8":
            s.weight = _quantise_i8(_he_f32(rng, s))
            x_rms = 37.0 if s.src == 0 else 32.0
        elif s.dtype == "bin":
            w = rng.standard_normal((s.c_out, s.c_in, s.kh, s.kw))
            s.weight = np.where(w >= 0, 1, -1).astype(np.int8)
            x_rms = 1.0
        else:
            raise ValueError(s.dtype)
        e_w2 = float(np.mean(s.weight.astype(np.float64) ** 2))
        sigma_p = math.sqrt(fan_in * e_w2) * x_rms          # rough std of the projection
        sh = _pick_shift(s, s.weight)
        if s.shift >= 0:
            s.shift = sh
        noise = max(1, int(sigma_p / 8))
        s.bias = rng.integers(-noise, noise + 1, size=s.c_out).astype(np.int32)
        if s.dtype == "i8" and s.src == 0:
            s.bias = (s.bias - 64 * s.weight.astype(np.int64).sum(axis=(1, 2, 3))).astype(np.int32)
        if s.act == "sign":
            # a 3x3 max-pool shifts the median of the pooled projection upwards
            s.theta = int(round(1.0 * sigma_p)) if s.pool is not None else 0
    return layers


# ---------------------------------------------------------------- config 1
def single_conv_f32(seed=1, c_in=64, c_out=64, hw=56, k=3, stride=1, pad=1):
    """One fp32 conv layer: W ~ N(0, 2/(k*k*c_in)), bias ~ N(0, 0.1)."""
    s = LayerSpec("conv", "f32", c_in, hw, hw, c_out, k, k, stride, pad, name="conv")
    return _fill(_resolve_src([s]), seed)


# ---------------------------------------------------------------- config 2
def fc6_i8(seed=2, c_in=9216, c_out=4096):
    """AlexNet-fc6-shaped int8 FC: W uniform[-127,127], int32 accumulation, raw int32 out."""
    rng = _rng(seed)
    s = LayerSpec("fc", "i8", c_in, 1, 1, c_out, name="fc6")
    s.weight = rng.integers(-127, 128, size=(c_out, c_in, 1, 1)).astype(np.int8)
    s.bias = rng.integers(-1000, 1001, size=c_out).astype(np.int32)
    return _resolve_src([s])


def fc6_i8_pruned(seed=2, c_in=9216, c_out=4096, keep=0.10):
    """The same layer after magnitude pruning: only the fraction `keep` of the weights with the largest magnitude
    stays, the rest is zero (unstructured, as deep compression leaves a layer; stands in for the compressed
    AlexNet of the paper's Table 4, whose trained weights are not available)."""
    s = fc6_i8(seed, c_in, c_out)[0]
    mag = np.abs(s.weight.astype(np.int16))
    thr = np.quantile(mag, 1.0 - keep)
    s.weight = np.where(mag > thr, s.weight, 0).astype(np.int8)
    s.name = "fc6_pruned"
    return [s]


# ---------------------------------------------------------------- config 3
def alexnet_convs(dtype="f32", seed=3, hw=227, scale=1):
    """conv1..conv5 of an AlexNet-shaped stack (groups=1, no LRN, 3x3 s2 floor pools
    after conv1/conv2/conv5).  `scale` divides channel counts (tests use small nets)."""
    c = [max(4, x // scale) for x in (96, 256, 384, 384, 256)]
    sh = 0 if dtype == "i8" else -1
    L = []
    L.append(LayerSpec("conv", dtype, 3, hw, hw, c[0], 11, 11, 4, 0, "relu", (3, 2, 0), sh, name="conv1"))
    _, (h, w) = out_hw(L[-1])
    L.append(LayerSpec("conv", dtype, c[0], h, w, c[1], 5, 5, 1, 2, "relu", (3, 2, 0), sh, name="conv2"))
    _, (h, w) = out_hw(L[-1])
    L.append(LayerSpec("conv", dtype, c[1], h, w, c[2], 3, 3, 1, 1, "relu", None, sh, name="conv3"))
    L.append(LayerSpec("conv", dtype, c[2], h, w, c[3], 3, 3, 1, 1, "relu", None, sh, name="conv4"))
    L.append(LayerSpec("conv", dtype, c[3], h, w, c[4], 3, 3, 1, 1, "relu", (3, 2, 0), sh, name="conv5"))
    return _fill(_resolve_src(L), seed)


# ---------------------------------------------------------------- config 4
def resnet18_convs(seed=4, hw=224, scale=1):
    """The 20 convs of ResNet-18 (BN folded into weight/bias), int8, with shortcuts.
    Basic block: a = relu(q(conv_a(x))); out = relu(q(conv_b(a)) + shortcut),
    shortcut = x or q(1x1-s2 downsample conv(x))."""
    ch = [max(4, x // scale) for x in (64, 128, 256, 512)]
    L = [LayerSpec("conv", "i8", 3, hw, hw, ch[0], 7, 7, 2, 3, "relu", (3, 2, 1), 0, name="conv1")]
    _, (h, w) = out_hw(L[-1])
    cur_t, cur_c = 1, ch[0]            # tensor index and channels of the block input
    for stage, c in enumerate(ch):
        for blk in range(2):
            stride = 2 if (stage > 0 and blk == 0) else 1
            nm = f"layer{stage + 1}.{blk}"
            a = LayerSpec("conv", "i8", cur_c, h, w, c, 3, 3, stride, 1, "relu", None, 0,
                          src=cur_t, name=nm + ".conv1")
            L.append(a)
            a_t = len(L)
            (h2, w2), _ = out_hw(a)
            short_t = cur_t
            if stride != 1 or cur_c != c:
                d = LayerSpec("conv", "i8", cur_c, h, w, c, 1, 1, stride, 0, "none", None, 0,
                              src=cur_t, name=nm + ".downsample")
                L.append(d)
                short_t = len(L)
            b = LayerSpec("conv", "i8", c, h2, w2, c, 3, 3, 1, 1, "relu", None, 0,
                          src=a_t, res=short_t, name=nm + ".conv2")
            L.append(b)
            cur_t, cur_c, h, w = len(L), c, h2, w2
    return _fill(_resolve_src(L), seed)


# ---------------------------------------------------------------- config 5
def xnor_alexnet_convs(seed=5, hw=227, scale=1):
    """conv1 int8 -> sign; conv2..conv5 binary (+-1 weights and inputs, zero padding,
    int32 popcount accumulation).  The last layer emits its pooled int32 projection."""
    c = [max(4, x // scale) for x in (96, 256, 384, 384, 256)]
    L = []
    L.append(LayerSpec("conv", "i8", 3, hw, hw, c[0], 11, 11, 4, 0, "sign", (3, 2, 0), -1, name="conv1"))
    _, (h, w) = out_hw(L[-1])
    L.append(LayerSpec("conv", "bin", c[0], h, w, c[1], 5, 5, 1, 2, "sign", (3, 2, 0), -1, name="conv2"))
    _, (h, w) = out_hw(L[-1])
    L.append(LayerSpec("conv", "bin", c[1], h, w, c[2], 3, 3, 1, 1, "sign", None, -1, name="conv3"))
    L.append(LayerSpec("conv", "bin", c[2], h, w, c[3], 3, 3, 1, 1, "sign", None, -1, name="conv4"))
    L.append(LayerSpec("conv", "bin", c[3], h, w, c[4], 3, 3, 1, 1, "none", (3, 2, 0), -1, name="conv5"))
    return _fill(_resolve_src(L), seed)


# ---------------------------------------------------------------- whole networks (second workloads)
def alexnet_full(dtype="i8", seed=6, hw=227, scale=1, classes=1000):
    """conv1..conv5 as in alexnet_convs plus fc6, fc7, fc8.  An FC layer after a convolution is the
    convolution whose filter covers the whole map (fc6: 6x6 over the 6x6x256 map); fc7 and fc8 are 1x1
    convolutions of a 1x1 map."""
    L = alexnet_convs(dtype, seed=seed, hw=hw, scale=scale)
    sh = 0 if dtype == "i8" else -1
    _, (h, w) = out_hw(L[-1])
    c = L[-1].c_out
    f = max(8, 4096 // scale)
    L.append(LayerSpec("conv", dtype, c, h, w, f, h, w, 1, 0, "relu", None, sh, name="fc6"))
    L.append(LayerSpec("conv", dtype, f, 1, 1, f, 1, 1, 1, 0, "relu", None, sh, name="fc7"))
    L.append(LayerSpec("conv", dtype, f, 1, 1, max(4, classes // scale), 1, 1, 1, 0, "none", None, -1 if dtype == "i8" else sh,
                       name="fc8"))
    for s in L:
        s.src = -1
    return _fill(_resolve_src(L), seed)


def vgg16_convs(dtype="i8", seed=7, hw=224, scale=1):
    """The 13 convolutions of a VGG-16-shaped stack (3x3, pad 1, ReLU; 2x2 stride-2 max-pool after
    conv 2, 4, 7, 10 and 13): the third model of the paper's Table 2."""
    plan = [(64, False), (64, True), (128, False), (128, True), (256, False), (256, False), (256, True),
            (512, False), (512, False), (512, True), (512, False), (512, False), (512, True)]
    sh = 0 if dtype == "i8" else -1
    L = []
    c_in, h, w = 3, hw, hw
    for i, (c, pool) in enumerate(plan):
        c = max(4, c // scale)
        L.append(LayerSpec("conv", dtype, c_in, h, w, c, 3, 3, 1, 1, "relu", (2, 2, 0) if pool else None, sh,
                           name=f"conv{i + 1}"))
        _, (h, w) = out_hw(L[-1])
        c_in = c
    return _fill(_resolve_src(L), seed)


# ---------------------------------------------------------------- explicit (unfolded) batch normalisation
def with_explicit_bn(layers, seed=8):
    """Gives every layer of a stack an explicit per-channel affine after its projection (batch normalisation at
    inference, not folded into the filters).  fp32 layers: scale in [0.5, 1.5], shift ~ N(0, 0.1).  int8 layers with
    a requantisation: integer multipliers in [24, 40] with the layer's shift raised by 5 (so the affine is about a
    factor one) and small integer offsets.  Layers of other kinds are left as they are.  Modifies `layers` in place."""
    rng = _rng(seed)
    for s in layers:
        if s.dtype == "f32":
            s.bn_scale = (0.5 + rng.random(s.c_out)).astype(np.float32)
            s.bn_shift = (rng.standard_normal(s.c_out) * 0.1).astype(np.float32)
        elif s.dtype == "i8" and s.shift >= 0 and s.act != "sign":
            s.bn_scale = rng.integers(24, 41, size=s.c_out).astype(np.int32)
            s.shift += 5
            s.bn_shift = rng.integers(-(1 << (s.shift - 1)), (1 << (s.shift - 1)) + 1, size=s.c_out).astype(np.int32)
    return layers


def fold_bn_f32(layers):
    """The same fp32 stack with every explicit affine folded into filters and bias (F' = scale * F,
    b' = scale * b + shift, in fp64 rounded to fp32): what a deployment that folds batch normalisation runs."""
    import copy
    out = []
    for s in layers:
        t = copy.copy(s)
        if s.dtype == "f32" and s.bn_scale is not None:
            sc = s.bn_scale.astype(np.float64)
            t.weight = (s.weight.astype(np.float64) * sc.reshape(-1, 1, 1, 1)).astype(np.float32)
            t.bias = (s.bias.astype(np.float64) * sc + s.bn_shift.astype(np.float64)).astype(np.float32)
            t.bn_scale = t.bn_shift = None
        out.append(t)
    return out
