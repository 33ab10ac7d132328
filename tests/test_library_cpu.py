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


def test_every_entry_point_refuses_null_and_oversized_arguments_before_touching_a_device(lib):
    """Host-detectable problems return a negative status and launch nothing (no device is needed to see that)."""
    from paper_2509_24248_b200 import binding as b
    kv, cfg, st, io = b.KV(), b.ExitCfg(), b.ExitState(), b.IterOut()
    kvp, cfgp, stp, iop = ctypes.byref(kv), ctypes.byref(cfg), ctypes.byref(st), ctypes.byref(io)
    INVALID = -1
    assert lib.sx_draft_step(None, kvp, 1, 1, None, None, None, None, None, None, None, None, 0, None, None) == INVALID
    assert lib.sx_verify(None, 1, 2, None, None, None, None, None, None, 2, None, None, 0, None, None) == INVALID
    assert lib.sx_exit_update(None, 1, 2, cfgp, stp, None, None, None, 2, None, None, None, None, None, None, None,
                              None) == INVALID
    assert lib.sx_spec_exit_iter(None, kvp, cfgp, stp, None, None, None, iop, None, 0, None, None) == INVALID
    assert lib.sx_spec_exit_iter_host(None, kvp, cfgp, stp, None, None, None, None, None, None, iop, None, None, None,
                                      None, None, 0, None, None) == INVALID
    assert lib.sx_commit(None, kvp, 2, None, None, None, 2, None, None, None, None, None, 0, None, None) == INVALID
    assert lib.sx_set_sampling(None, 1.0, 0, 0) == INVALID
    assert lib.sx_profile_begin(None) == INVALID
    assert lib.sx_profile_end(None, None, None) == INVALID
    assert lib.sx_tile_weight(None, 128, 64, None, None) == INVALID
    assert lib.sx_tiled_weight_bytes(0, 64) == 0 and lib.sx_tiled_weight_bytes(129, 65) == 2 * 2 * 128 * 64 * 2
    assert lib.sx_selftest_bounded_wait(100, 1, None, None, None) == INVALID
    assert lib.sx_launch_count(None) == 0
    lib.sx_destroy(None)
    # the no-allocation entry point: NULL, misaligned and oversized requests
    fake = 4096                                                # a non-NULL, 16-byte aligned stand-in; never dereferenced
    assert lib.sx_verify_noalloc(None, 64, 64, 1, 2, fake, fake, None, fake, fake, fake, 2, fake, fake, None) == INVALID
    assert lib.sx_verify_noalloc(fake + 2, 64, 64, 1, 2, fake, fake, None, fake, fake, fake, 2, fake, fake, None) == INVALID
    assert lib.sx_verify_noalloc(fake, 64, 60, 1, 2, fake, fake, None, fake, fake, fake, 2, fake, fake, None) == INVALID
    assert lib.sx_verify_noalloc(fake, 64, 64, 13, 5, fake, fake, None, fake, fake, fake, 5, fake, fake, None) == -7
    assert lib.sx_verify_noalloc(fake, 64, 64, 1, 65, fake, fake, fake, fake, fake, fake, 5, fake, fake, None) == -2
    # sx_create: shapes the kernels do not cover are refused before any device query
    m = b.ModelCfg(60, 4, 2, 16, 96, 200, 3, 1e-6, 1e6, 16, (ctypes.c_int32 * 3)(0, 0, 0), 0, 0, 0)
    w = b.Weights(*([fake] * 11), None, None)
    dc = b.DraftCfg(0, 3, 1, 0, 0)
    out = ctypes.c_void_p()
    assert lib.sx_create(ctypes.byref(m), ctypes.byref(w), 1, ctypes.byref(dc), 0, ctypes.byref(out)) == -2   # H % 8
    m.H = 64
    m.n_q_heads = 3
    assert lib.sx_create(ctypes.byref(m), ctypes.byref(w), 1, ctypes.byref(dc), 0, ctypes.byref(out)) == -2   # group size
    m.n_q_heads = 4
    w.fc_d = fake + 4
    assert lib.sx_create(ctypes.byref(m), ctypes.byref(w), 1, ctypes.byref(dc), 0, ctypes.byref(out)) == INVALID
    w.fc_d = fake
    dc.K = 0
    assert lib.sx_create(ctypes.byref(m), ctypes.byref(w), 1, ctypes.byref(dc), 0, ctypes.byref(out)) == INVALID
    assert out.value is None


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
