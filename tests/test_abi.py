"""The C-ABI library loads and exports every symbol that include/sgc.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sgc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sgc_[a-z_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2502_00311_b200 import build, binding
    path = build.build()
    L = ctypes.CDLL(path)
    names = declared_functions()
    assert "sgc_create" in names and "sgc_step" in names and "sgc_destroy" in names
    for n in names:
        assert hasattr(L, n), "missing export %s" % n
    assert sorted(binding.EXPORTS) == names
    assert binding.version() >= 100
    assert binding.strerror(0) == "success" and "NULL" in binding.strerror(-1)


def test_argument_errors_without_touching_the_gpu():
    from paper_2502_00311_b200 import binding
    L = binding.lib()
    h = ctypes.c_void_p()
    assert L.sgc_create(None, 10, 4, 2, 0, 1e-3, 0.9, 0.999, 1e-8) == -1
    for (d, k, s) in [(0, 4, 1), (10, 0, 1), (10, 4, 0), (10, 4, 5), (3, 8, 4), (1 << 32, 8, 4), (10 ** 6, 70000, 4),
                      (10 ** 6, 4096, 2000)]:
        assert L.sgc_create(ctypes.byref(h), d, k, s, 0, 1e-3, 0.9, 0.999, 1e-8) == -2 and not h.value
    for (b1, b2, eps) in [(1.0, 0.9, 1e-8), (-0.1, 0.9, 1e-8), (0.9, 1.5, 1e-8), (0.9, 0.9, 0.0)]:
        assert L.sgc_create(ctypes.byref(h), 100, 8, 2, 0, 1e-3, b1, b2, eps) == -3
    assert L.sgc_step(None, None, None, None) == -1
    assert L.sgc_destroy(None) == 0
    assert L.sgc_set_alpha(None, 1.0) == -1
    assert L.sgc_get(None, 0, None, 0) == -1
    assert L.sgc_step_group(None, None, None, 1, None) == -1
    assert L.sgc_z_block(0, 0, 1, 0, 1, None, None) == -1


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2502_00311_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                for needle in ("import oracle", "from oracle", "sgc_oracle", "orc_", "oracle/", "oracle."):
                    assert needle not in text, (f, needle)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".cpp")):
            assert "paper_2502_00311_b200" not in open(os.path.join(ROOT, "oracle", f)).read(), f
