"""The C ABI library builds for sm_100a, loads without a GPU, and exports every symbol
that include/gnnco.h declares; the binding refuses to run without it."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "gnnco.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gnnco_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import paper_2511_09261_b200 as gnnco
    lib = gnnco.load_library()
    names = _declared()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(gnnco.EXPORTS) == names


def test_status_strings_and_argument_checks_need_no_gpu():
    import paper_2511_09261_b200 as gnnco
    lib = gnnco.load_library()
    assert gnnco.status_string(0) == "ok"
    assert "range" in gnnco.status_string(gnnco.OUT_OF_RANGE)
    p, s = ctypes.c_size_t(0), ctypes.c_size_t(0)
    assert lib.gnnco_partition_workspace_bytes(0, 0, 1, ctypes.byref(p), ctypes.byref(s)) == gnnco.INVALID_ARGUMENT
    assert lib.gnnco_partition_workspace_bytes(10, 5, 11, ctypes.byref(p), ctypes.byref(s)) == gnnco.INVALID_ARGUMENT
    assert lib.gnnco_partition_workspace_bytes(1000, 5000, 8, ctypes.byref(p), ctypes.byref(s)) == gnnco.OK
    assert p.value > 0 and s.value > 0 and p.value % 256 == 0
    assert lib.gnnco_partition_load(None, None, 0, None, 0, None, None) == gnnco.INVALID_ARGUMENT
    assert lib.gnnco_train_step(None, None, None, None, None, None, 0, None, 0, None) == gnnco.INVALID_ARGUMENT
    assert lib.gnnco_decode_boundary(None, None, 0.5, None, None, None, None, None) == gnnco.INVALID_ARGUMENT
    assert lib.gnnco_launch_count(None) == 0


def test_binding_fails_loudly_without_the_library(monkeypatch):
    import paper_2511_09261_b200 as gnnco
    from paper_2511_09261_b200 import _build
    monkeypatch.setattr(gnnco, "_lib", None)
    monkeypatch.setattr(_build, "LIB_PATH", os.path.join(ROOT, "does_not_exist", "libgnnco.so"))
    monkeypatch.setattr(_build, "needs_build", lambda: False)
    with pytest.raises(RuntimeError):
        gnnco.load_library()


def test_product_code_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2511_09261_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "gnnco_oracle" not in text and "from oracle" not in text, f
