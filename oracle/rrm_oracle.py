"""CPU oracle for the Recurrent Residual Module (RRM) hot path.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path imports this module; it is
used by tests/, by the smoke check and by the bench's CPU-baseline leg.  It shares no
code with the CUDA library: the arithmetic lives in rrm_oracle.c (plain loops) and in
the numpy expressions below.

Two independent evaluations of a layer stack are provided:

* `dense_forward`  - the plain definition (Eq. 1-2): every frame is pushed through
  the ordinary dense network on its own.  This is what RRM claims to reproduce exactly.
* `Recurrence`     - Algorithm 1 taken literally: per linear layer keep the previous
  input I_{t-1,l} and projection P_{t-1,l}; form the delta, visit its non-zeros only
  (Sec. 3.5), add F*dI (no bias, Eq. 4) onto P_{t-1,l}, apply f.

Precision: fp32 layers are evaluated in fp64 on the exactly promoted fp32 data; int8
and binary layers in exact int64 arithmetic (results are asserted to fit int32).

Readings of points the paper leaves open (these bind the CUDA path too):
  - P_{0,l} = b_l, so that the first frame processed as a delta from I_0 = 0 is a
    dense pass (Algorithm 1 initialises I_0 but not P_0).
  - f is applied to the sum P_{t-1,l} + F*dI; that sum and the layer input are what
    is kept for the next frame.
  - '*' is cross-correlation with zero padding; filters are [C_out][C_in][kh][kw].
  - an element is "non-zero" iff the two frames' values differ (threshold eps = 0).
Parity unpinned by the paper (not in it; fixed here by definition and hand-checked
tiny cases): the int8 requantisation rule, the sign threshold, pooling order, the integer
form of an explicit batch normalisation.
  - int8: q = clamp((P + 2^(s-1)) >> s, -127, 127) (arithmetic shift), then + shortcut,
    then ReLU (clamp to [0,127]) or clamp to [-127,127], then max-pool.
  - binary: inputs/weights are +-1, padding is 0; sign(v) = +1 iff v >= theta, taken on
    the max-pooled int32 projection.
  - explicit batch normalisation (the non-linear layer the paper's Discussion names, Sec. 4.5):
    at inference a per-channel affine applied to the full projection P_t before anything else of
    f.  fp32: y = scale * P + shift.  int8: integer multiplier and offset inside the
    requantisation, q = clamp((P * scale + shift + 2^(s-1)) >> s, -127, 127), 64-bit exact.
"""
import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "librrm_oracle.so")
_SRC = os.path.join(_HERE, "rrm_oracle.c")
_lib = None


def build(force=False):
    """Compile rrm_oracle.c with gcc -O3 and OpenMP."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O3", "-march=native", "-fopenmp", "-shared", "-fPIC",
                               "-o", _SO, _SRC, "-lm"])
    return _SO


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_SO)
        for n in ("conv_delta", "fc_delta"):
            for t in ("f64", "i64"):
                getattr(_lib, f"rrm_oracle_{n}_{t}").restype = ctypes.c_int64
    return _lib


def threads():
    return int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _kind(spec):
    """('f64', np.float64) for fp32 layers, ('i64', np.int64) for int8/binary layers."""
    return ("f64", np.float64) if spec.dtype == "f32" else ("i64", np.int64)


def _out_dim(i, k, s, p):
    return (i + 2 * p - k) // s + 1


# --------------------------------------------------------------------- linear part
_promoted = []      # [(weight array, element type, promoted copy)], most recently used last


def _weights(spec, dt):
    """The layer's filters in the oracle's element type.  The C routines take fp64 / int64 arrays; promoting a
    large filter bank (fc6: 37.7 M int8 -> 302 MB of int64) costs far more than the recurrence's own work, so
    the promoted copy of a large, unchanged weight array is kept between calls.  Small arrays are promoted
    every time (tests edit them in place)."""
    w = spec.weight
    if w.size < (1 << 20):
        return np.ascontiguousarray(w, dtype=dt)
    for i, (src, t, F) in enumerate(_promoted):
        if src is w and t == dt:
            _promoted.append(_promoted.pop(i))
            return F
    F = np.ascontiguousarray(w, dtype=dt)
    _promoted.append((w, dt, F))
    del _promoted[:-3]
    return F


def projection(spec, I, with_bias=True):
    """Eq. 3: P = F*I + b (conv) or W I + b (FC).  I: [N,C,H,W] (FC: [N,C] or [N,C,1,1])."""
    t, dt = _kind(spec)
    I = np.ascontiguousarray(I, dtype=dt)
    F = _weights(spec, dt)
    b = np.ascontiguousarray(spec.bias, dtype=dt) if with_bias else None
    N = I.shape[0]
    if spec.kind == "fc":
        P = np.empty((N, spec.c_out), dtype=dt)
        getattr(lib(), f"rrm_oracle_fc_{t}")(_p(I), _p(F), _p(b) if b is not None else None, _p(P),
                                            N, spec.c_in, spec.c_out)
        return P.reshape(N, spec.c_out, 1, 1)
    oh = _out_dim(spec.h, spec.kh, spec.stride, spec.pad)
    ow = _out_dim(spec.w, spec.kw, spec.stride, spec.pad)
    P = np.empty((N, spec.c_out, oh, ow), dtype=dt)
    getattr(lib(), f"rrm_oracle_conv_{t}")(_p(I), _p(F), _p(b) if b is not None else None, _p(P),
                                          N, spec.c_in, spec.h, spec.w, spec.c_out,
                                          spec.kh, spec.kw, spec.stride, spec.pad)
    return P


def delta_accumulate(spec, D, P):
    """Algorithm 1, P_t = P_{t-1} + F*dI, visiting only the non-zeros of dI (Sec. 3.5).
    Updates P in place; returns the multiply-accumulates executed."""
    t, dt = _kind(spec)
    D = np.ascontiguousarray(D, dtype=dt)
    F = _weights(spec, dt)
    assert P.dtype == dt and P.flags["C_CONTIGUOUS"]
    N = D.shape[0]
    if spec.kind == "fc":
        return int(getattr(lib(), f"rrm_oracle_fc_delta_{t}")(_p(D), _p(F), _p(P), N, spec.c_in, spec.c_out))
    return int(getattr(lib(), f"rrm_oracle_conv_delta_{t}")(_p(D), _p(F), _p(P), N, spec.c_in, spec.h,
                                                           spec.w, spec.c_out, spec.kh, spec.kw,
                                                           spec.stride, spec.pad))


# ------------------------------------------------------------------ nonlinear part
def maxpool(X, k, s, p):
    t = "f64" if X.dtype == np.float64 else "i64"
    X = np.ascontiguousarray(X)
    N, C, H, W = X.shape
    Y = np.empty((N, C, _out_dim(H, k, s, p), _out_dim(W, k, s, p)), dtype=X.dtype)
    getattr(lib(), f"rrm_oracle_maxpool_{t}")(_p(X), _p(Y), N, C, H, W, k, s, p)
    return Y


def requant(P, shift):
    """q = clamp((P + 2^(s-1)) >> s, -127, 127), arithmetic shift (round half up)."""
    P = P.astype(np.int64)
    if shift > 0:
        P = (P + (1 << (shift - 1))) >> shift
    return np.clip(P, -127, 127)


def nonlinearity(spec, P, res=None):
    """The map f of Eq. 1 for one layer: I_{t,l+1} = f(P_tl)."""
    bn = getattr(spec, "bn_scale", None) is not None
    if spec.dtype == "f32":
        if bn:                                           # explicit batch normalisation: per-channel affine first
            P = (np.asarray(spec.bn_scale, dtype=np.float64).reshape(1, -1, 1, 1) * P
                 + np.asarray(spec.bn_shift, dtype=np.float64).reshape(1, -1, 1, 1))
        v = P if res is None else P + res
        if spec.act == "relu":
            v = np.maximum(v, 0.0)
        elif spec.act == "leaky":                       # leaky ReLU with the slope 0.1 (as an fp32 constant)
            v = np.where(v > 0.0, v, float(np.float32(0.1)) * v)
        elif spec.act != "none":
            raise ValueError(spec.act)
        return maxpool(v, *spec.pool) if spec.pool is not None else v
    # integer projections
    assert np.all(np.abs(P) < 2 ** 31), "projection does not fit int32"
    if spec.act == "sign":
        v = maxpool(P, *spec.pool) if spec.pool is not None else P
        return np.where(v >= spec.theta, 1, -1).astype(np.int64)
    assert not bn or (spec.shift >= 0 and spec.act != "sign"), "integer affine is defined inside the requantisation only"
    if spec.shift < 0:
        assert res is None and spec.act == "none"
        return maxpool(P, *spec.pool) if spec.pool is not None else P
    if bn:                                               # integer multiplier and offset, exact in int64
        P = (P.astype(np.int64) * np.asarray(spec.bn_scale, dtype=np.int64).reshape(1, -1, 1, 1)
             + np.asarray(spec.bn_shift, dtype=np.int64).reshape(1, -1, 1, 1))
        assert np.all(np.abs(P) < 2 ** 62)
    v = requant(P, spec.shift)
    if res is not None:
        v = v + res
    v = np.clip(v, 0, 127) if spec.act == "relu" else np.clip(v, -127, 127)
    return maxpool(v, *spec.pool) if spec.pool is not None else v


# ---------------------------------------------------------------- dense definition
def dense_forward(layers, frame):
    """Ordinary dense inference of one frame.  Returns (tensors, projections):
    tensors[0] is the frame, tensors[l+1] = f(P_l)."""
    _, dt = _kind(layers[0])
    tensors = [np.asarray(frame).astype(dt)]
    if layers[0].kind == "fc":
        tensors[0] = tensors[0].reshape(tensors[0].shape[0], -1, 1, 1)
    projs = []
    for s in layers:
        P = projection(s, tensors[s.src])
        projs.append(P)
        tensors.append(nonlinearity(s, P, tensors[s.res] if s.res >= 0 else None))
    return tensors, projs


# ------------------------------------------------------------- Algorithm 1, literal
class Recurrence:
    """Algorithm 1.  State per linear layer: I_prev (zeros at start) and P_prev (= bias).

    eps > 0 (fp32 layers) is the sparsity enhancement of Sec. 3.4: delta entries with |d| < eps are
    truncated to zero before the sparse product.  Reading: the snapshot still becomes I_t, so the
    truncated part u is lost and the error accumulates; the decision |d| < eps is taken on the delta
    computed in fp32 (the kernel's precision).  trunc_l2[l] is l2(u) of the last step for layer l
    (over all streams of the batch) and e_t the running sum of Eq. 7 since the last reset."""

    def __init__(self, layers, n=1, eps=0.0):
        self.layers = layers
        self.eps = float(eps)
        self.trunc_l2 = [0.0] * len(layers)
        self.e_t = 0.0
        self.I_prev, self.P_prev = [], []
        for s in layers:
            _, dt = _kind(s)
            oh = _out_dim(s.h, s.kh, s.stride, s.pad)
            ow = _out_dim(s.w, s.kw, s.stride, s.pad)
            self.I_prev.append(np.zeros((n, s.c_in, s.h, s.w), dtype=dt))
            P0 = np.empty((n, s.c_out, oh, ow), dtype=dt)
            P0[:] = np.asarray(s.bias, dtype=dt).reshape(1, -1, 1, 1)
            self.P_prev.append(P0)
        self.nnz = [0] * len(layers)      # non-zero delta elements, last step
        self.macs = [0] * len(layers)     # multiply-accumulates executed, last step

    def step(self, frame):
        layers = self.layers
        _, dt = _kind(layers[0])
        tensors = [np.asarray(frame).astype(dt)]
        if layers[0].kind == "fc":
            tensors[0] = tensors[0].reshape(tensors[0].shape[0], -1, 1, 1)
        for l, s in enumerate(layers):
            I = tensors[s.src]
            D = I - self.I_prev[l]                              # Alg. 1: delta of the layer input
            self.trunc_l2[l] = 0.0
            if self.eps > 0.0 and s.dtype == "f32":            # Sec. 3.4: truncate small delta entries
                d32 = I.astype(np.float32) - self.I_prev[l].astype(np.float32)
                keep = np.abs(d32) >= np.float32(self.eps)
                u = np.where(keep, 0.0, D)
                D = np.where(keep, D, 0.0)
                self.trunc_l2[l] = float(np.sqrt(np.sum(u * u)))
                self.e_t += self.trunc_l2[l]                   # Eq. 7
            self.nnz[l] = int(np.count_nonzero(D))
            self.macs[l] = delta_accumulate(s, D, self.P_prev[l])   # P_t = P_{t-1} + F*dI
            self.I_prev[l] = I.copy()                           # snapshot the input
            tensors.append(nonlinearity(s, self.P_prev[l], tensors[s.res] if s.res >= 0 else None))
        return tensors, [p.copy() for p in self.P_prev]

    def reset_to(self, frame):
        """A precise (dense) inference of `frame` replaces the state and clears the accumulated
        truncated value (Sec. 3.4, last sentence)."""
        tensors, projs = dense_forward(self.layers, frame)
        for l, s in enumerate(self.layers):
            self.I_prev[l] = tensors[s.src].copy()
            self.P_prev[l] = projs[l].copy()
        self.e_t = 0.0
        self.trunc_l2 = [0.0] * len(self.layers)
        return tensors, projs

    def density(self):
        """Per-layer element density rho of the last step's input delta (Table 1)."""
        return [self.nnz[l] / self.I_prev[l].size for l in range(len(self.layers))]


def aecs_predict(mu, e_t):
    """Eq. 8 with H a fourth-order polynomial: e_c = mu[0] + mu[1] e_t + ... + mu[4] e_t^4."""
    assert len(mu) == 5
    return float(sum(float(m) * float(e_t) ** k for k, m in enumerate(mu)))


# ------------------------------------------------------------- evaluation formulas
def layer_macs(s):
    oh = _out_dim(s.h, s.kh, s.stride, s.pad)
    ow = _out_dim(s.w, s.kw, s.stride, s.pad)
    return oh * ow * s.c_in * s.c_out * s.kh * s.kw


def overall_sparsity(sparsities, macs):
    """Eq. 9: MAC-weighted mean of the per-layer input sparsities."""
    return float(np.dot(sparsities, macs) / np.sum(macs))


def speedup_ratio(rho, rho_hat, macs):
    """Eq. 10: eta = sum(rho * MACs) / sum(rho_hat * MACs)."""
    return float(np.dot(rho, macs) / np.dot(rho_hat, macs))
