"""ctypes binding of include/rrm.h.  Argument marshalling only: device pointers come from
torch tensors (`.data_ptr()`), streams from `torch.cuda.current_stream().cuda_stream`."""
import ctypes
import os

import numpy as np
import torch

from . import build as _build

KIND = {"conv": 0, "fc": 1}
DTYPE = {"f32": 0, "i8": 1, "bin": 2}
ACT = {"none": 0, "relu": 1, "sign": 2, "leaky": 3}
VARIANT = {"auto": 0, "gather": 1, "tensor": 2, "dense": 3, "sparse_w": 4}


class RRMError(RuntimeError):
    pass


class LayerDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "kind", "dtype", "n", "c_in", "h", "w", "c_out", "kh", "kw", "stride", "pad", "act",
        "pool_k", "pool_s", "pool_p", "shift", "theta", "src", "res", "variant")]


class Stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in (
        "in_elems", "nnz_elems", "in_pixels", "active_in_pixels", "out_pixels", "active_out_pixels",
        "active_macs", "dense_macs")] + [("variant", ctypes.c_int32), ("error_word", ctypes.c_int32)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class Options(ctypes.Structure):
    _fields_ = [("wait_limit", ctypes.c_uint32), ("layer_dense_activity", ctypes.c_float),
                ("layer_delta_activity", ctypes.c_float), ("stack_dense_activity", ctypes.c_float),
                ("stack_reprobe", ctypes.c_int32), ("fc_dense_rows", ctypes.c_float), ("fc_dense_density", ctypes.c_float),
                ("chunk_dense_activity", ctypes.c_float)]


_lib = None
_P = ctypes.c_void_p


def lib():
    """Loads librrm_b200.so (building it with nvcc if absent or older than its sources).  Raises if
    that fails: there is no fallback implementation and a stale library is never loaded."""
    global _lib
    if _lib is not None:
        return _lib
    so = _build.SO
    if _build.needs_build():
        # never load a library that is older than its sources: a failed rebuild is an error, not a fallback
        try:
            _build.build()
        except Exception as e:  # noqa: BLE001
            state = "out of date" if os.path.exists(so) else "missing"
            raise RRMError(f"librrm_b200.so is {state} and could not be built: {e}") from e
    L = ctypes.CDLL(so)
    sig = {
        "rrm_layer_create": [ctypes.POINTER(_P), ctypes.POINTER(LayerDesc), _P, _P],
        "rrm_layer_destroy": [_P],
        "rrm_keyframe": [_P, _P, _P, _P],
        "rrm_step": [_P, _P, _P, _P],
        "rrm_dense": [_P, _P, _P, _P],
        "rrm_step_host": [_P, _P, _P, _P],
        "rrm_get_stats": [_P, ctypes.POINTER(Stats)],
        "rrm_layer_projection": [_P, _P, _P],
        "rrm_net_create": [ctypes.POINTER(_P), ctypes.POINTER(LayerDesc), ctypes.c_int, ctypes.POINTER(_P),
                           ctypes.POINTER(_P)],
        "rrm_net_destroy": [_P],
        "rrm_net_keyframe": [_P, _P, _P, _P],
        "rrm_net_step": [_P, _P, _P, _P],
        "rrm_net_dense": [_P, _P, _P, _P],
        "rrm_net_step_host": [_P, _P, _P, _P],
        "rrm_step_seq": [_P, _P, _P, ctypes.c_int, _P],
        "rrm_dense_seq": [_P, _P, _P, ctypes.c_int, _P],
        "rrm_step_seq_host": [_P, _P, _P, ctypes.c_int, _P],
        "rrm_net_step_seq": [_P, _P, _P, ctypes.c_int, _P],
        "rrm_net_dense_seq": [_P, _P, _P, ctypes.c_int, _P],
        "rrm_net_step_seq_host": [_P, _P, _P, ctypes.c_int, _P],
        "rrm_step_seq_host_async": [_P, _P, _P, ctypes.c_int, _P],
        "rrm_net_step_seq_host_async": [_P, _P, _P, ctypes.c_int, _P],
        "rrm_host_sync": [_P],
        "rrm_net_host_sync": [_P],
        "rrm_net_get_stats": [_P, ctypes.c_int, ctypes.POINTER(Stats)],
        "rrm_net_projection": [_P, ctypes.c_int, _P, _P],
        "rrm_net_tensor": [_P, ctypes.c_int, _P, _P],
        "rrm_net_set_affine": [_P, ctypes.c_int, _P, _P],
        "rrm_clear_errors": [_P],
        "rrm_net_clear_errors": [_P],
        "rrm_get_options": [_P, ctypes.POINTER(Options)],
        "rrm_set_options": [_P, ctypes.POINTER(Options)],
        "rrm_net_get_options": [_P, ctypes.POINTER(Options)],
        "rrm_net_set_options": [_P, ctypes.POINTER(Options)],
    }
    for name, args in sig.items():
        f = getattr(L, name)
        f.argtypes = args
        f.restype = ctypes.c_int
    L.rrm_fc_step_noalloc.argtypes = [_P, _P, _P, _P, _P] + [ctypes.c_int] * 5 + [_P]
    L.rrm_fc_step_noalloc.restype = ctypes.c_int
    L.rrm_net_set_epsilon.argtypes = [_P, ctypes.c_float]
    L.rrm_net_set_epsilon.restype = ctypes.c_int
    L.rrm_net_truncation.argtypes = [_P, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    L.rrm_net_truncation.restype = ctypes.c_int
    L.rrm_aecs_predict.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.c_double]
    L.rrm_aecs_predict.restype = ctypes.c_double
    L.rrm_net_tensor_bytes.argtypes = [_P, ctypes.c_int]
    L.rrm_net_tensor_bytes.restype = ctypes.c_int64
    L.rrm_measure_alu_peak.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_double)]
    L.rrm_measure_alu_peak.restype = ctypes.c_int
    L.rrm_strerror.argtypes = [ctypes.c_int]
    L.rrm_strerror.restype = ctypes.c_char_p
    _lib = L
    return L


def _check(status, what):
    if status != 0:
        raise RRMError(f"{what}: {lib().rrm_strerror(status).decode()} ({status})")


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t)


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def desc_from_spec(s, n=1, variant="auto"):
    """rrm_layer_desc from any object with the LayerSpec attributes."""
    d = LayerDesc()
    d.kind, d.dtype, d.n = KIND[s.kind], DTYPE[s.dtype], n
    d.c_in, d.h, d.w, d.c_out = s.c_in, s.h, s.w, s.c_out
    d.kh, d.kw, d.stride, d.pad = s.kh, s.kw, s.stride, s.pad
    d.act = ACT[s.act]
    d.pool_k, d.pool_s, d.pool_p = s.pool if s.pool is not None else (0, 0, 0)
    d.shift, d.theta = s.shift, s.theta
    d.src, d.res = max(s.src, 0), s.res
    d.variant = VARIANT[variant]
    return d


class Net:
    """Owner of an rrm_net*.  Methods mirror the C entry points one to one."""

    def __init__(self, descs, weights, biases):
        self._h = _P()
        self.descs = list(descs)
        L = len(self.descs)
        arr = (LayerDesc * L)(*self.descs)
        self._keep = (weights, biases)
        W = (_P * L)(*[_ptr(w) for w in weights])
        B = (_P * L)(*[_ptr(b) for b in biases])
        _check(lib().rrm_net_create(ctypes.byref(self._h), arr, L, W, B), "rrm_net_create")
        self.n_layers = L

    def close(self):
        if self._h:
            lib().rrm_net_destroy(self._h)
            self._h = _P()

    def __del__(self):
        try:
            self.close()
        except Exception:  # noqa: BLE001
            pass

    def keyframe(self, frame, out=None, stream=None):
        _check(lib().rrm_net_keyframe(self._h, _ptr(frame), _ptr(out), _stream(stream)), "rrm_net_keyframe")

    def step(self, frame, out=None, stream=None):
        _check(lib().rrm_net_step(self._h, _ptr(frame), _ptr(out), _stream(stream)), "rrm_net_step")

    def dense(self, frame, out=None, stream=None):
        _check(lib().rrm_net_dense(self._h, _ptr(frame), _ptr(out), _stream(stream)), "rrm_net_dense")

    def step_host(self, frame_host, out_host=None, stream=None):
        _check(lib().rrm_net_step_host(self._h, _ptr(frame_host), _ptr(out_host), _stream(stream)),
               "rrm_net_step_host")

    def step_seq(self, frames, outs=None, T=None, stream=None):
        T = frames.shape[0] if T is None else T
        _check(lib().rrm_net_step_seq(self._h, _ptr(frames), _ptr(outs), T, _stream(stream)), "rrm_net_step_seq")

    def dense_seq(self, frames, outs=None, T=None, stream=None):
        T = frames.shape[0] if T is None else T
        _check(lib().rrm_net_dense_seq(self._h, _ptr(frames), _ptr(outs), T, _stream(stream)), "rrm_net_dense_seq")

    def step_seq_host(self, frames_host, outs_host=None, T=None, stream=None):
        T = frames_host.shape[0] if T is None else T
        _check(lib().rrm_net_step_seq_host(self._h, _ptr(frames_host), _ptr(outs_host), T, _stream(stream)),
               "rrm_net_step_seq_host")

    def step_seq_host_async(self, frames_host, outs_host=None, T=None, stream=None):
        T = frames_host.shape[0] if T is None else T
        _check(lib().rrm_net_step_seq_host_async(self._h, _ptr(frames_host), _ptr(outs_host), T, _stream(stream)),
               "rrm_net_step_seq_host_async")

    def host_sync(self):
        _check(lib().rrm_net_host_sync(self._h), "rrm_net_host_sync")

    def set_epsilon(self, eps):
        _check(lib().rrm_net_set_epsilon(self._h, float(eps)), "rrm_net_set_epsilon")

    def set_affine(self, layer, scale, shift):
        """rrm_net_set_affine: explicit per-channel affine (unfolded batch normalisation) as the first step of f."""
        _check(lib().rrm_net_set_affine(self._h, layer, _ptr(scale), _ptr(shift)), "rrm_net_set_affine")

    def truncation(self):
        """(e_t of Eq. 7 since the last keyframe, [per-layer l2 of the last frame])."""
        e = ctypes.c_double()
        per = (ctypes.c_double * self.n_layers)()
        _check(lib().rrm_net_truncation(self._h, ctypes.byref(e), per), "rrm_net_truncation")
        return e.value, list(per)

    def stats(self, layer=0, check=True):
        """rrm_net_get_stats.  A device-side error since the last clear_errors() (a bounded wait that ran out, an
        int8 delta outside a byte) comes back as the call's status: raised, or with check=False returned beside the
        counters under the key "status"."""
        s = Stats()
        status = lib().rrm_net_get_stats(self._h, layer, ctypes.byref(s))
        if check or status not in (0, -5, -6):
            _check(status, "rrm_net_get_stats")
        d = s.as_dict()
        d["status"] = status
        return d

    def clear_errors(self):
        _check(lib().rrm_net_clear_errors(self._h), "rrm_net_clear_errors")

    def options(self):
        o = Options()
        _check(lib().rrm_net_get_options(self._h, ctypes.byref(o)), "rrm_net_get_options")
        return {n: getattr(o, n) for n, _ in o._fields_}

    def set_options(self, **kw):
        """rrm_net_set_options with the named fields replaced (the others keep their current values)."""
        o = Options()
        _check(lib().rrm_net_get_options(self._h, ctypes.byref(o)), "rrm_net_get_options")
        for k, v in kw.items():
            if k not in dict(o._fields_):
                raise KeyError(k)
            setattr(o, k, v)
        _check(lib().rrm_net_set_options(self._h, ctypes.byref(o)), "rrm_net_set_options")

    def tensor_bytes(self, t):
        b = lib().rrm_net_tensor_bytes(self._h, t)
        if b < 0:
            _check(int(b), "rrm_net_tensor_bytes")
        return int(b)

    def _tensor_meta(self, t):
        """(torch dtype, shape) of tensor t in the boundary layout."""
        d0 = self.descs[0]
        if t == 0:
            code, c, h, w = d0.dtype, d0.c_in, d0.h, d0.w
            kind = {0: "f32", 1: "i8", 2: "bin"}[code]
        else:
            d = self.descs[t - 1]
            oh = (d.h + 2 * d.pad - d.kh) // d.stride + 1
            ow = (d.w + 2 * d.pad - d.kw) // d.stride + 1
            if d.pool_k:
                oh = (oh + 2 * d.pool_p - d.pool_k) // d.pool_s + 1
                ow = (ow + 2 * d.pool_p - d.pool_k) // d.pool_s + 1
            c, h, w = d.c_out, oh, ow
            kind = "f32" if d.dtype == 0 else ("bin" if d.act == 2 else ("i8" if d.shift >= 0 else "i32"))
        n = d0.n
        if kind == "bin":
            return torch.int32, (n, h, w, (c + 31) // 32)
        return {"f32": torch.float32, "i8": torch.int8, "i32": torch.int32}[kind], (n, c, h, w)

    def new_output(self, t=None, frames=None):
        dt, shape = self._tensor_meta(self.n_layers if t is None else t)
        if frames is not None:
            shape = (frames,) + tuple(shape)
        return torch.empty(shape, dtype=dt, device="cuda")

    def tensor(self, t, stream=None):
        out = self.new_output(t)
        _check(lib().rrm_net_tensor(self._h, t, out.data_ptr(), _stream(stream)), "rrm_net_tensor")
        return out

    def projection(self, layer, stream=None):
        d = self.descs[layer]
        oh = (d.h + 2 * d.pad - d.kh) // d.stride + 1
        ow = (d.w + 2 * d.pad - d.kw) // d.stride + 1
        out = torch.empty((d.n, d.c_out, oh, ow), dtype=torch.float32 if d.dtype == 0 else torch.int32, device="cuda")
        _check(lib().rrm_net_projection(self._h, layer, out.data_ptr(), _stream(stream)), "rrm_net_projection")
        return out


Layer = Net   # a single layer is a stack of one


def fc_step_noalloc(Wt, Xt, Xprev, P, Y, n, c_in, c_out, shift=-1, act="none", stream=None):
    """rrm_fc_step_noalloc: one int8 delta-FC frame on caller-owned state, for callers that may
    not allocate device memory.  Returns the status code instead of raising, so that a caller
    can test the documented limits."""
    return lib().rrm_fc_step_noalloc(_ptr(Wt), _ptr(Xt), _ptr(Xprev), _ptr(P), _ptr(Y), n, c_in, c_out, shift,
                                     ACT[act], _stream(stream))


def measure_alu_peak(kind):
    """rrm_measure_alu_peak: measured multiply-accumulates per second of "ffma", "dp4a" or "popc" on the current device."""
    v = ctypes.c_double()
    _check(lib().rrm_measure_alu_peak({"ffma": 0, "dp4a": 1, "popc": 2}[kind], ctypes.byref(v)), "rrm_measure_alu_peak")
    return v.value


def aecs_predict(mu, e_t):
    """rrm_aecs_predict: the fourth-order polynomial error estimate of Eq. 8."""
    arr = (ctypes.c_double * 5)(*[float(m) for m in mu])
    return lib().rrm_aecs_predict(arr, float(e_t))


def net_from_specs(specs, n=1, variant="auto", device="cuda"):
    """Uploads weights/biases of a list of LayerSpec-like objects and creates the stack."""
    descs = [desc_from_spec(s, n, variant) for s in specs]
    Ws = [torch.from_numpy(np.ascontiguousarray(s.weight)).to(device) for s in specs]
    Bs = [torch.from_numpy(np.ascontiguousarray(s.bias)).to(device) for s in specs]
    torch.cuda.synchronize()
    net = Net(descs, Ws, Bs)
    for l, s in enumerate(specs):
        if getattr(s, "bn_scale", None) is not None:
            net.set_affine(l, torch.from_numpy(np.ascontiguousarray(s.bn_scale)).to(device),
                           torch.from_numpy(np.ascontiguousarray(s.bn_shift)).to(device))
    return net


def layer_from_spec(spec, n=1, variant="auto", device="cuda"):
    return net_from_specs([spec], n, variant, device)
