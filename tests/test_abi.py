"""Host-side checks that need no GPU: the shared library builds, loads, and exports every
symbol the public header declares; the Python structs mirror the C structs."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "rrm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rrm_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import paper_1802_09723_b200 as rrm
    L = rrm.lib()
    names = _declared_symbols()
    assert "rrm_step" in names and "rrm_net_step" in names and "rrm_layer_create" in names
    for n in names:
        assert hasattr(L, n), n


def test_strerror_and_struct_sizes():
    import paper_1802_09723_b200 as rrm
    L = rrm.lib()
    assert L.rrm_strerror(0) == b"ok"
    assert L.rrm_strerror(-2) == b"shape mismatch"
    assert ctypes.sizeof(rrm.LayerDesc) == 20 * 4
    assert ctypes.sizeof(rrm.Stats) == 8 * 8 + 2 * 4


def test_null_arguments_are_rejected_without_a_device():
    import paper_1802_09723_b200 as rrm
    L = rrm.lib()
    assert L.rrm_layer_create(None, None, None, None) == -1
    assert L.rrm_net_step(None, None, None, None) == -1
    assert L.rrm_net_tensor_bytes(None, 0) == -1
    assert L.rrm_net_get_options(None, None) == -1 and L.rrm_net_set_options(None, None) == -1
    assert L.rrm_net_clear_errors(None) == -1
    assert ctypes.sizeof(rrm.Options) == 8 * 4


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_1802_09723_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f


def _desc(**kw):
    import paper_1802_09723_b200 as rrm
    d = rrm.LayerDesc()
    base = dict(kind=0, dtype=0, n=1, c_in=4, h=8, w=8, c_out=4, kh=3, kw=3, stride=1, pad=1, act=0, pool_k=0, pool_s=0,
                pool_p=0, shift=-1, theta=0, src=0, res=-1, variant=0)
    base.update(kw)
    for k, v in base.items():
        setattr(d, k, v)
    return d


def test_invalid_descriptions_are_rejected_before_any_device_work():
    """Validation comes first in rrm_layer_create, so these calls return their error codes on a machine
    without a GPU too (the weight pointer is a dummy that is never dereferenced)."""
    import paper_1802_09723_b200 as rrm
    L = rrm.lib()
    INVALID, SHAPE, DTYPE, UNSUPPORTED = -1, -2, -3, -8
    dummy = ctypes.c_void_p(16)
    cases = [
        (_desc(kind=7), INVALID), (_desc(dtype=9), DTYPE), (_desc(n=0), SHAPE), (_desc(c_out=0), SHAPE),
        (_desc(stride=0), SHAPE), (_desc(pad=3), SHAPE), (_desc(kh=11, kw=11, h=4, w=4, pad=0), SHAPE),
        (_desc(kind=1, h=2), SHAPE), (_desc(act=5), INVALID), (_desc(act=2), UNSUPPORTED), (_desc(act=3, dtype=1, shift=4), UNSUPPORTED),
        (_desc(pool_k=3, pool_s=0), SHAPE), (_desc(pool_k=5, pool_s=2), UNSUPPORTED), (_desc(shift=40, dtype=1), INVALID),
        (_desc(variant=9), INVALID), (_desc(dtype=1, shift=-1, act=1), UNSUPPORTED),
    ]
    for d, want in cases:
        h = ctypes.c_void_p()
        got = L.rrm_layer_create(ctypes.byref(h), ctypes.byref(d), dummy, None)
        assert got == want, ({n: getattr(d, n) for n, _ in d._fields_}, got, want)
        assert not h.value
    # a stack whose second layer reads a tensor that does not exist yet, or whose shapes do not chain
    two = (rrm.LayerDesc * 2)(_desc(), _desc(src=2))
    W = (ctypes.c_void_p * 2)(16, 16)
    h = ctypes.c_void_p()
    assert L.rrm_net_create(ctypes.byref(h), two, 2, W, None) == INVALID
    two = (rrm.LayerDesc * 2)(_desc(), _desc(src=1, c_in=5))
    assert L.rrm_net_create(ctypes.byref(h), two, 2, W, None) == SHAPE
    assert L.rrm_net_set_epsilon(None, ctypes.c_float(0.1)) == INVALID
    assert L.rrm_step_seq(None, None, None, 4, None) == INVALID


def test_error_strings_cover_every_status():
    import paper_1802_09723_b200 as rrm
    L = rrm.lib()
    seen = {L.rrm_strerror(s) for s in range(0, -9, -1)}
    assert len(seen) == 9 and b"unknown status" not in seen
    assert L.rrm_strerror(-99) == b"unknown status"
