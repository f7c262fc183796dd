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


def test_streams_step_argument_errors(lib):
    """dpclip_step_streams checks its stream and workspace arrays on the host before anything is enqueued."""
    fake = ctypes.c_void_p(0x1000)
    INVALID = -1
    from paper_2009_03106_b200 import binding
    own = ctypes.CDLL(binding.library_path())      # a handle of its own: the prototypes set here stay out of the binding's
    f = own.dpclip_step_streams
    f.restype = ctypes.c_int
    vp = ctypes.c_void_p

    class Layer(ctypes.Structure):
        _fields_ = [("A", vp), ("lda", ctypes.c_long), ("Zbar", vp), ("ldz", ctypes.c_long), ("T", ctypes.c_int),
                    ("d_in", ctypes.c_int), ("d_out", ctypes.c_int), ("has_bias", ctypes.c_int), ("method", ctypes.c_int),
                    ("gW", vp), ("ldg", ctypes.c_long), ("gb", vp)]
    f.argtypes = [ctypes.POINTER(Layer), ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_float, ctypes.c_float,
                  ctypes.c_ulonglong, ctypes.c_ulonglong, vp, vp, vp, ctypes.c_int, ctypes.POINTER(vp), ctypes.POINTER(vp),
                  ctypes.c_size_t]
    layers = (Layer * 1)(Layer(0x1000, 8, 0x2000, 8, 4, 8, 8, 0, 0, 0x3000, 8, None))
    st2 = (vp * 2)(0x10, 0x20); ws2 = (vp * 2)(0x4000, 0x5000)
    same_st = (vp * 2)(0x10, 0x10); same_ws = (vp * 2)(0x4000, 0x4000)
    call = lambda n, st, ws: f(layers, 1, 2, 0, 1.0, 0.0, 0, 0, fake, fake, None, n, st, ws, 1 << 20)   # noqa: E731
    assert call(0, st2, ws2) == INVALID
    assert call(9, st2, ws2) == INVALID
    assert call(2, None, ws2) == INVALID
    assert call(2, st2, None) == INVALID
    assert call(2, same_st, ws2) == INVALID
    assert call(2, st2, same_ws) == INVALID
    assert f(layers, 1, 2, 0, 0.0, 0.0, 0, 0, fake, fake, None, 2, st2, ws2, 1 << 20) == INVALID     # C must be > 0


def test_workspace_queries_without_a_gpu(lib):
    """The workspace queries are host arithmetic: the fixed scratch for ordinary layers, room for one partial
    tile per row slice for long bf16 layers whose 64 tiles leave SMs idle in one wave, and the copies of the
    fp32 feature-map convolution routes."""
    from paper_2009_03106_b200 import binding
    lib = ctypes.CDLL(binding.library_path())      # own handle, own prototypes
    lib.dpclip_workspace_bytes.restype = ctypes.c_size_t
    lib.dpclip_workspace_bytes.argtypes = [ctypes.c_int] * 6
    floor = lib.dpclip_workspace_bytes(1, 1, 1, 1, 1, 0)
    assert lib.dpclip_workspace_bytes(128, 256, 512, 128, 1, 0) == floor            # narrow d_out: one partial tile per SM
    # d_out wide enough for the CTA-pair kernel: one 512 x 256 segment (+ 512 bias sums) per tile (+ 16 for part-empty super-layers) and one per pair
    seg = 512 * 256 * 4 + 512 * 4
    assert lib.dpclip_workspace_bytes(128, 256, 512, 2048, 1, 0) == 256 + (8 + 16 + 74) * seg
    assert lib.dpclip_workspace_bytes(256, 128, 1024, 4096, 1, 0) == 256 + (32 + 16 + 74) * seg
    # 64 tiles of 256 x 256 and long rows: the single-CTA kernel's preferred cut (9 slices per tile) is larger still
    long64 = lib.dpclip_workspace_bytes(256, 2048, 1024, 4096, 1, 0)
    assert long64 == 256 + 64 * 9 * (256 * 256 * 4 + 256 * 4)
    assert lib.dpclip_workspace_bytes(32, 1, 784, 256, 0, 0) == 256                 # small fp32 layer: header only

    class Conv(ctypes.Structure):
        _fields_ = [(n, ctypes.c_int) for n in ("C", "H", "W", "kh", "kw", "stride", "pad")]
    lib.dpclip_conv_workspace_bytes.restype = ctypes.c_size_t
    lib.dpclip_conv_workspace_bytes.argtypes = [ctypes.c_int, ctypes.POINTER(Conv), ctypes.c_int, ctypes.c_int, ctypes.c_int]
    g = Conv(32, 16, 16, 3, 3, 1, 1)
    rows = lib.dpclip_conv_workspace_bytes(128, ctypes.byref(g), 64, 0, 0)
    cm = lib.dpclip_conv_workspace_bytes(128, ctypes.byref(g), 64, 0, 1)
    assert cm == rows + 128 * 256 * 64 * 4                                          # the [B][T][d_out] copy
    assert lib.dpclip_conv_workspace_bytes(128, ctypes.byref(g), 64, 1, 1) == floor  # bf16 reads either layout
    g1 = Conv(3, 32, 32, 3, 3, 1, 1)
    first = lib.dpclip_conv_workspace_bytes(128, ctypes.byref(g1), 32, 0, 0)
    assert first == rows + 128 * 1024 * 32 * 4 + 128 * 1024 * 27 * 4                # dL/dZ rows + the patch matrix
