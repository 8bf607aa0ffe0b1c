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


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_1802_09723_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f
