"""The C-ABI library builds, loads and exports every symbol the header declares;
argument errors are reported on the host before any launch (no GPU needed)."""
import ctypes
import os
import re
import shutil

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "dpclip.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2009_03106_b200 import build as b
    if not os.path.exists(b.LIB) and shutil.which("nvcc") is None and not os.path.exists("/usr/local/cuda/bin/nvcc"):
        pytest.skip("no nvcc and no prebuilt library")
    if os.path.exists("/usr/local/cuda/bin/nvcc") or shutil.which("nvcc"):
        b.build()
    from paper_2009_03106_b200 import binding
    return binding.load_library()


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dpclip_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_four_required_entry_points():
    syms = declared_symbols()
    for name in ("dpclip_layer_sqnorms", "dpclip_factors", "dpclip_clipped_grad", "dpclip_add_noise"):
        assert name in syms


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_binding_has_the_same_names():
    import paper_2009_03106_b200 as pkg
    for name in declared_symbols():
        if name == "dpclip_step_host_arena_bytes":
            continue          # used inside HostStep only
        assert hasattr(pkg, name), name


def test_status_strings_and_version(lib):
    assert lib.dpclip_version() >= 100
    assert lib.dpclip_status_string(0) == b"ok"
    assert b"invalid" in lib.dpclip_status_string(-1)
    assert b"unknown" in lib.dpclip_status_string(-99)


def test_argument_errors_are_caught_before_any_launch(lib):
    fake = ctypes.c_void_p(0x1000)          # never dereferenced: every call below fails validation first
    ws = ctypes.c_void_p(0x2000)
    INVALID, UNSUPPORTED, MISALIGNED, WORKSPACE = -1, -2, -3, -4
    f = lib.dpclip_layer_sqnorms
    assert f(None, 4, fake, 4, 2, 1, 4, 4, 0, 1, 0, fake, ws, 256, None) == INVALID
    assert f(fake, 4, fake, 4, 0, 1, 4, 4, 0, 1, 0, fake, ws, 256, None) == INVALID      # B = 0
    assert f(fake, 4, fake, 4, 2, 0, 4, 4, 0, 1, 0, fake, ws, 256, None) == INVALID      # T = 0
    assert f(fake, 3, fake, 4, 2, 1, 4, 4, 0, 1, 0, fake, ws, 256, None) == INVALID      # lda < d_in
    assert f(fake, 4, fake, 4, 2, 1, 4, 4, 7, 1, 0, fake, ws, 256, None) == INVALID      # dtype
    assert f(ctypes.c_void_p(0x1002), 4, fake, 4, 2, 1, 4, 4, 0, 1, 0, fake, ws, 256, None) == MISALIGNED
    assert f(fake, 4, fake, 4, 2, 1, 4, 4, 0, 1, 0, fake, None, 0, None) == WORKSPACE
    assert f(fake, 4, fake, 4, 2, 3, 4, 4, 0, 1, 1, fake, ws, 1 << 20, None) == UNSUPPORTED   # T1 with T > 1
    assert f(fake, 4, fake, 4, 2, 3, 4, 4, 0, 1, 2, fake, ws, 1 << 30, None) == UNSUPPORTED   # GRAM with fp32
    g = lib.dpclip_factors
    assert g(None, 1, 4, 4, 1.0, fake, None, None, None) == INVALID
    assert g(fake, 1, 4, 4, 0.0, fake, None, None, None) == INVALID                      # C must be > 0
    assert g(fake, 1, 2, 4, 1.0, fake, None, None, None) == INVALID                      # ld_sq < B
    h = lib.dpclip_clipped_grad
    assert h(fake, 4, fake, 4, 2, 1, 4, 4, 0, None, None, 4, None, ws, 256, None) == INVALID
    assert h(fake, 4, fake, 4, 2, 1, 4, 4, 0, None, fake, 3, None, ws, 256, None) == INVALID   # ldg < d_in
    n = lib.dpclip_add_noise
    assert n(None, 0, 1.0, 1.0, 0, 0, None) == 0                                          # n = 0 is a no-op
    assert n(None, 8, 1.0, 1.0, 0, 0, None) == INVALID
    assert n(fake, 8, -1.0, 1.0, 0, 0, None) == INVALID
    assert lib.dpclip_workspace_bytes(128, 256, 512, 512, 1, 0) >= 256
    assert lib.dpclip_pick_method(128, 1, 784, 256, 784, 256, 0) == 1
