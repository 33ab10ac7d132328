"""The C-ABI library builds, loads without a GPU and exports every declared entry point."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2509_24248_b200 import build, binding
    build.build()
    return binding.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "specexit.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sx_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "sx_spec_exit_iter" in names and "sx_draft_step" in names and "sx_verify" in names
    assert "sx_exit_update" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/specexit.h but not exported"
    from paper_2509_24248_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_strerror_and_null_checks_without_a_device(lib):
    assert lib.sx_strerror(0) == b"ok"
    assert b"workspace" in lib.sx_strerror(-4)
    out = ctypes.c_void_p()
    assert lib.sx_create(None, None, 1, None, 0, ctypes.byref(out)) == -1
    assert lib.sx_workspace_bytes(None) == 0


def test_struct_layouts_match_header():
    from paper_2509_24248_b200 import binding as b
    assert ctypes.sizeof(b.ModelCfg) == 4 * 16
    assert ctypes.sizeof(b.Weights) == 8 * 13
    assert ctypes.sizeof(b.DraftCfg) == 20
    assert ctypes.sizeof(b.IterOut) == 8 * 18
    assert b.ExitCfg.split_bitmap_d.offset % 8 == 0


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2509_24248_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.replace("no CPU fallback", ""), f
