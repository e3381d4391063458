"""The C-ABI library loads without a GPU, exports every entry point that include/mcce.h declares, and
its host-side argument checks work (no kernel is launched here)."""
import ctypes as C
import os
import re

import pytest

from paper_2412_00099_b200 import build as mbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    path = mbuild.build()
    return C.CDLL(path)


def declared_names():
    text = open(os.path.join(ROOT, "include", "mcce.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mcce_[a-z_]+)\s*\(", text)))


def test_every_declared_entry_point_is_exported(lib):
    names = declared_names()
    assert len(names) >= 17
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_entry_points():
    src = open(os.path.join(ROOT, "paper_2412_00099_b200", "binding.py")).read()
    for n in declared_names():
        assert '"%s"' % n in src, n


def test_host_side_validation(lib):
    from paper_2412_00099_b200.binding import Config
    lib.mcce_workspace_bytes.restype = C.c_size_t
    lib.mcce_strerror.restype = C.c_char_p
    ok = Config(24, 60, 4, 2, 4, 2048, 1408, 30, 256, 0.5, 0, 1, 1, 1, 0, 0)
    n = lib.mcce_workspace_bytes(C.byref(ok))
    assert 250e6 < n < 1e9                      # gathered activations + intermediates for 6144 pairs
    for field, bad in [("n_experts", 257), ("top_k", 17), ("top_j", 5), ("d_model", 2050), ("cache_capacity", 0),
                       ("lam", -0.1), ("weight_dtype", 0), ("delta_mode", 2), ("n_streams", 0)]:
        cfg = Config(24, 60, 4, 2, 4, 2048, 1408, 30, 256, 0.5, 0, 1, 1, 1, 0, 0)
        setattr(cfg, field, bad)
        assert lib.mcce_workspace_bytes(C.byref(cfg)) == 0, field
    out = C.c_void_p()
    assert lib.mcce_create(C.byref(ok), None, 0, C.byref(out)) == -1          # null workspace
    assert lib.mcce_create(C.byref(ok), C.c_void_p(256), 1024, C.byref(out)) == -2   # too small
    assert b"workspace" in lib.mcce_strerror(-2)
    assert lib.mcce_destroy(None) == -1
