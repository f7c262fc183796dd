"""ctypes binding of libdpclip.so: same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's kernels.  torch is used for
device memory and for the current CUDA stream.  There is no CPU fallback: if
the shared library is missing or does not load, the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# DPCLIP_LIBRARY selects another build of the same library (the range-checked libdpclip_debug.so)
_LIB_PATH = os.environ.get("DPCLIP_LIBRARY") or os.path.join(_HERE, "libdpclip.so")
_lib = None

DPCLIP_F32, DPCLIP_BF16 = 0, 1
DPCLIP_AUTO, DPCLIP_T1, DPCLIP_GRAM, DPCLIP_MATERIALIZE, DPCLIP_SIMT = 0, 1, 2, 3, 4

_vp, _i, _l, _f = ctypes.c_void_p, ctypes.c_int, ctypes.c_long, ctypes.c_float
_sz, _u64 = ctypes.c_size_t, ctypes.c_ulonglong


class DpclipError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {status} ({dpclip_status_string(status)})")


class _CConv(ctypes.Structure):
    _fields_ = [("C", ctypes.c_int), ("H", ctypes.c_int), ("W", ctypes.c_int), ("kh", ctypes.c_int),
                ("kw", ctypes.c_int), ("stride", ctypes.c_int), ("pad", ctypes.c_int)]


class _CLayer(ctypes.Structure):
    _fields_ = [("A", _vp), ("lda", _l), ("Zbar", _vp), ("ldz", _l),
                ("T", _i), ("d_in", _i), ("d_out", _i), ("has_bias", _i), ("method", _i),
                ("gW", _vp), ("ldg", _l), ("gb", _vp)]


class _CModelLayer(ctypes.Structure):
    _fields_ = [("kind", _i), ("layer", _CLayer), ("conv", _CConv), ("z_channel_major", _i)]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libdpclip.so (built in-tree by paper_2009_03106_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with "
                          "`python -m paper_2009_03106_b200.build` (there is no fallback path)")
    L = ctypes.CDLL(_LIB_PATH)
    L.dpclip_layer_sqnorms.argtypes = [_vp, _l, _vp, _l, _i, _i, _i, _i, _i, _i, _i, _vp, _vp, _sz, _vp]
    L.dpclip_factors.argtypes = [_vp, _i, _l, _i, _f, _vp, _vp, _vp, _vp]
    L.dpclip_clipped_grad.argtypes = [_vp, _l, _vp, _l, _i, _i, _i, _i, _i, _vp, _vp, _l, _vp, _vp, _sz, _vp]
    L.dpclip_clipped_grad_noalloc.argtypes = [_vp, _l, _vp, _l, _i, _i, _i, _i, _i, _vp, _vp, _l, _vp, _vp]
    L.dpclip_clipped_grad_noalloc.restype = _i
    L.dpclip_noalloc_max_output_bytes.argtypes = []
    L.dpclip_noalloc_max_output_bytes.restype = _sz
    L.dpclip_clipped_grad_noise.argtypes = [_vp, _l, _vp, _l, _i, _i, _i, _i, _i, _vp, _vp, _vp, _f, _f, _u64, _u64,
                                            _u64, _vp, _sz, _vp]
    L.dpclip_clipped_grad_noise.restype = _i
    L.dpclip_add_noise.argtypes = [_vp, _sz, _f, _f, _u64, _u64, _vp]
    L.dpclip_conv_sqnorms.argtypes = [_vp, _vp, _i, _i, ctypes.POINTER(_CConv), _i, _i, _i, _vp, _vp, _sz, _vp]
    L.dpclip_conv_sqnorms.restype = _i
    L.dpclip_conv_clipped_grad.argtypes = [_vp, _vp, _i, _i, ctypes.POINTER(_CConv), _i, _i, _vp, _vp, _l, _vp, _vp, _sz, _vp]
    L.dpclip_conv_clipped_grad.restype = _i
    L.dpclip_conv_workspace_bytes.argtypes = [_i, ctypes.POINTER(_CConv), _i, _i, _i]
    L.dpclip_conv_workspace_bytes.restype = _sz
    L.dpclip_dp_sgd_step.argtypes = [_vp, _vp, _sz, _f, _f, _f, _u64, _u64, _f, _vp]
    L.dpclip_dp_sgd_step.restype = _i
    L.dpclip_dp_adam_step.argtypes = [_vp, _vp, _vp, _vp, _sz, _f, _f, _f, _u64, _u64, _f, _f, _f, _f, _i, _vp]
    L.dpclip_dp_adam_step.restype = _i
    L.dpclip_step_noise.argtypes = [ctypes.POINTER(_CLayer), _i, _f, _f, _u64, _u64, _vp]
    L.dpclip_step_noise.restype = _i
    L.dpclip_t1_layers_supported.argtypes = [ctypes.POINTER(_CLayer), _i, _i, _i]
    L.dpclip_t1_layers_supported.restype = _i
    L.dpclip_t1_layers_sqnorms.argtypes = [ctypes.POINTER(_CLayer), _i, _i, _i, _vp, _vp]
    L.dpclip_t1_layers_sqnorms.restype = _i
    L.dpclip_gram_layers_sqnorms.argtypes = [ctypes.POINTER(_CLayer), _i, _i, _i, _vp, ctypes.POINTER(ctypes.c_int),
                                             _vp, ctypes.c_size_t, _vp]
    L.dpclip_gram_layers_sqnorms.restype = _i
    L.dpclip_same_shape_layers_clipped_grad_noise.argtypes = [
        ctypes.POINTER(_CLayer), _i, _i, _i, _vp, ctypes.c_float, ctypes.c_float, ctypes.c_ulonglong,
        ctypes.c_ulonglong, ctypes.POINTER(ctypes.c_int), _vp, ctypes.c_size_t, _vp]
    L.dpclip_same_shape_layers_clipped_grad_noise.restype = _i
    L.dpclip_t1_layers_clipped_grad_noise.argtypes = [ctypes.POINTER(_CLayer), _i, _i, _i, _vp, _f, _f, _u64, _u64,
                                                      _vp, _sz, _vp]
    L.dpclip_t1_layers_clipped_grad_noise.restype = _i
    L.dpclip_elementwise_sqnorms.argtypes = [_vp, _l, _vp, _l, _i, _i, _i, _i, _i, _vp, _vp]
    L.dpclip_elementwise_sqnorms.restype = _i
    L.dpclip_elementwise_clipped_grad.argtypes = [_vp, _l, _vp, _l, _i, _i, _i, _i, _vp, _vp, _vp, _vp]
    L.dpclip_elementwise_clipped_grad.restype = _i
    L.dpclip_step.argtypes = [ctypes.POINTER(_CLayer), _i, _i, _i, _f, _f, _u64, _u64, _vp, _vp, _vp, _vp, _sz, _vp]
    L.dpclip_step_streams.argtypes = [ctypes.POINTER(_CLayer), _i, _i, _i, _f, _f, _u64, _u64, _vp, _vp, _vp, _i,
                                      ctypes.POINTER(_vp), ctypes.POINTER(_vp), _sz]
    L.dpclip_step_streams.restype = _i
    L.dpclip_model_step_streams.argtypes = [ctypes.POINTER(_CModelLayer), _i, _i, _i, _f, _f, _u64, _u64, _vp, _vp, _vp,
                                            _i, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _sz]
    L.dpclip_model_step_streams.restype = _i
    L.dpclip_step_host.argtypes = [ctypes.POINTER(_CLayer), _i, _i, _i, _f, _f, _u64, _u64, _vp, _vp, _vp, _sz, _vp]
    L.dpclip_step_host_arena_bytes.argtypes = [ctypes.POINTER(_CLayer), _i, _i, _i]
    L.dpclip_step_host_arena_bytes.restype = _sz
    L.dpclip_step_per_layer.argtypes = [ctypes.POINTER(_CLayer), _i, _i, _i, ctypes.POINTER(ctypes.c_float), _f, _u64, _u64,
                                        _vp, _vp, _vp, _vp, _sz, _vp]
    L.dpclip_step_per_layer.restype = _i
    L.dpclip_model_step.argtypes = [ctypes.POINTER(_CModelLayer), _i, _i, _i, _f, _f, _u64, _u64, _vp, _vp, _vp, _vp,
                                    _sz, _vp]
    L.dpclip_model_step.restype = _i
    L.dpclip_model_workspace_bytes.argtypes = [ctypes.POINTER(_CModelLayer), _i, _i, _i]
    L.dpclip_model_workspace_bytes.restype = _sz
    L.dpclip_workspace_bytes.argtypes = [_i, _i, _i, _i, _i, _i]
    L.dpclip_workspace_bytes.restype = _sz
    L.dpclip_step_workspace_bytes.argtypes = [ctypes.POINTER(_CLayer), _i, _i, _i]
    L.dpclip_step_workspace_bytes.restype = _sz
    L.dpclip_workspace_init.argtypes = [_vp, _sz, _vp]
    L.dpclip_read_status.argtypes = [_vp, ctypes.POINTER(_i), _vp]
    L.dpclip_pick_method.argtypes = [_i, _i, _i, _i, _l, _l, _i]
    L.dpclip_status_string.argtypes = [_i]
    L.dpclip_status_string.restype = ctypes.c_char_p
    L.dpclip_version.argtypes = []
    L.dpclip_debug_build.argtypes = []
    L.dpclip_launch_count.argtypes = []
    L.dpclip_launch_count.restype = _u64
    L.dpclip_null_launch.argtypes = [_i, _i, _vp]
    L.dpclip_null_launch.restype = _i
    L.dpclip_reload_path_switches.argtypes = []
    L.dpclip_reload_path_switches.restype = None
    for name in ("dpclip_layer_sqnorms", "dpclip_factors", "dpclip_clipped_grad", "dpclip_add_noise",
                 "dpclip_step", "dpclip_step_host", "dpclip_workspace_init", "dpclip_read_status",
                 "dpclip_pick_method", "dpclip_version"):
        getattr(L, name).restype = _i
    _lib = L
    return L


# ----------------------------------------------------------------------------
# marshalling helpers
# ----------------------------------------------------------------------------
def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DPCLIP_F32
    if t.dtype == torch.bfloat16:
        return DPCLIP_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _check(fn: str, rc: int):
    if rc != 0:
        raise DpclipError(fn, rc)


def _rows(t: torch.Tensor):
    """(B, T, d) tensor with contiguous features -> (B, T, d, row stride in elements)."""
    if t.dim() == 2:
        t = t.unsqueeze(1)
    B, T, d = t.shape
    if t.stride(2) != 1 and d > 1:
        raise ValueError("feature dimension must be contiguous")
    ld = t.stride(1) if T > 1 else (t.stride(0) if B > 1 else d)
    if T > 1 and B > 1 and t.stride(0) != T * ld:
        raise ValueError("rows of consecutive examples must be equally spaced")
    return B, T, d, ld


# ----------------------------------------------------------------------------
# the C ABI, one function per entry point
# ----------------------------------------------------------------------------
def dpclip_version() -> int:
    return load_library().dpclip_version()


def dpclip_debug_build() -> bool:
    return bool(load_library().dpclip_debug_build())


def dpclip_launch_count() -> int:
    return load_library().dpclip_launch_count()


def dpclip_null_launch(cooperative: bool, grid: int = 128, stream=None) -> None:
    """One empty kernel with the launch shape of the one-launch T = 1 step (launch-floor measurements)."""
    _check("dpclip_null_launch", load_library().dpclip_null_launch(int(cooperative), grid, _stream(stream)))


def dpclip_reload_path_switches() -> None:
    """Re-read the DPCLIP_* test/measurement switches from the environment (they are read once otherwise)."""
    load_library().dpclip_reload_path_switches()


def dpclip_status_string(status: int) -> str:
    try:
        return load_library().dpclip_status_string(status).decode()
    except ImportError:
        return "library not loaded"


def dpclip_workspace_bytes(B, T, d_in, d_out, dtype=DPCLIP_F32, method=DPCLIP_AUTO) -> int:
    return load_library().dpclip_workspace_bytes(B, T, d_in, d_out, dtype, method)


def dpclip_workspace_init(workspace: torch.Tensor, stream=None) -> None:
    _check("dpclip_workspace_init",
           load_library().dpclip_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                                _stream(stream)))


def dpclip_read_status(workspace: torch.Tensor, stream=None) -> int:
    out = _i(0)
    _check("dpclip_read_status", load_library().dpclip_read_status(_ptr(workspace), ctypes.byref(out),
                                                                   _stream(stream)))
    return out.value


def dpclip_pick_method(B, T, d_in, d_out, lda=None, ldz=None, dtype=DPCLIP_F32) -> int:
    return load_library().dpclip_pick_method(B, T, d_in, d_out, lda or d_in, ldz or d_out, dtype)


def dpclip_layer_sqnorms(A: torch.Tensor, Zbar: torch.Tensor, has_bias: bool, sq_layer: torch.Tensor,
                         workspace: torch.Tensor, method: int = DPCLIP_AUTO, stream=None) -> None:
    B, T, d_in, lda = _rows(A)
    B2, T2, d_out, ldz = _rows(Zbar)
    assert (B, T) == (B2, T2) and A.dtype == Zbar.dtype
    assert sq_layer.dtype == torch.float32 and sq_layer.numel() >= B and sq_layer.is_contiguous()
    _check("dpclip_layer_sqnorms", load_library().dpclip_layer_sqnorms(
        _ptr(A), lda, _ptr(Zbar), ldz, B, T, d_in, d_out, _dtype_code(A), int(has_bias), method,
        _ptr(sq_layer), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


def dpclip_factors(sq_layers: torch.Tensor, C: float, clip: torch.Tensor, norms: Optional[torch.Tensor] = None,
                   n_clipped: Optional[torch.Tensor] = None, stream=None) -> None:
    L, B = sq_layers.shape
    assert sq_layers.dtype == torch.float32 and sq_layers.stride(1) == 1
    _check("dpclip_factors", load_library().dpclip_factors(
        _ptr(sq_layers), L, sq_layers.stride(0) if L > 1 else B, B, C, _ptr(clip), _ptr(norms),
        _ptr(n_clipped), _stream(stream)))


def dpclip_clipped_grad(A: torch.Tensor, Zbar: torch.Tensor, clip: Optional[torch.Tensor], gW: torch.Tensor,
                        gb: Optional[torch.Tensor], workspace: torch.Tensor, stream=None) -> None:
    B, T, d_in, lda = _rows(A)
    _, _, d_out, ldz = _rows(Zbar)
    assert gW.dtype == torch.float32 and gW.shape == (d_out, d_in) and gW.stride(1) == 1
    _check("dpclip_clipped_grad", load_library().dpclip_clipped_grad(
        _ptr(A), lda, _ptr(Zbar), ldz, B, T, d_in, d_out, _dtype_code(A), _ptr(clip), _ptr(gW),
        gW.stride(0) if d_out > 1 else d_in, _ptr(gb), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream(stream)))


def dpclip_clipped_grad_noise(A: torch.Tensor, Zbar: torch.Tensor, clip: Optional[torch.Tensor], gW: torch.Tensor,
                              gb: Optional[torch.Tensor], sigma: float, C: float, seed: int, stream_id_w: int,
                              stream_id_b: int, workspace: torch.Tensor, stream=None) -> None:
    B, T, d_in, lda = _rows(A)
    _, _, d_out, ldz = _rows(Zbar)
    assert gW.dtype == torch.float32 and gW.shape == (d_out, d_in) and gW.is_contiguous()
    _check("dpclip_clipped_grad_noise", load_library().dpclip_clipped_grad_noise(
        _ptr(A), lda, _ptr(Zbar), ldz, B, T, d_in, d_out, _dtype_code(A), _ptr(clip), _ptr(gW), _ptr(gb),
        sigma, C, seed, stream_id_w, stream_id_b, _ptr(workspace), workspace.numel() * workspace.element_size(),
        _stream(stream)))


def dpclip_noalloc_max_output_bytes() -> int:
    return load_library().dpclip_noalloc_max_output_bytes()


def dpclip_clipped_grad_noalloc(A: torch.Tensor, Zbar: torch.Tensor, clip: Optional[torch.Tensor],
                                gW: torch.Tensor, gb: Optional[torch.Tensor], stream=None) -> None:
    """dpclip_clipped_grad without a workspace argument: for callers that cannot hand the library
    device memory.  The scratch is a fixed array inside the library; see the header for its limits."""
    B, T, d_in, lda = _rows(A)
    _, _, d_out, ldz = _rows(Zbar)
    assert gW.dtype == torch.float32 and gW.shape == (d_out, d_in) and gW.stride(1) == 1
    _check("dpclip_clipped_grad_noalloc", load_library().dpclip_clipped_grad_noalloc(
        _ptr(A), lda, _ptr(Zbar), ldz, B, T, d_in, d_out, _dtype_code(A), _ptr(clip), _ptr(gW),
        gW.stride(0) if d_out > 1 else d_in, _ptr(gb), _stream(stream)))


def dpclip_add_noise(g: torch.Tensor, sigma: float, C: float, seed: int, stream_id: int, stream=None) -> None:
    assert g.dtype == torch.float32 and g.is_contiguous()
    _check("dpclip_add_noise", load_library().dpclip_add_noise(_ptr(g), g.numel(), sigma, C, seed, stream_id,
                                                               _stream(stream)))


def dpclip_elementwise_sqnorms(Hbar: torch.Tensor, Zbar: torch.Tensor, has_shift: bool, sq_layer: torch.Tensor,
                               stream=None) -> None:
    B, T, d, ldh = _rows(Hbar)
    B2, T2, d2, ldz = _rows(Zbar)
    assert (B, T, d) == (B2, T2, d2) and Hbar.dtype == Zbar.dtype
    assert sq_layer.dtype == torch.float32 and sq_layer.numel() >= B and sq_layer.is_contiguous()
    _check("dpclip_elementwise_sqnorms", load_library().dpclip_elementwise_sqnorms(
        _ptr(Hbar), ldh, _ptr(Zbar), ldz, B, T, d, _dtype_code(Hbar), int(has_shift), _ptr(sq_layer), _stream(stream)))


def dpclip_elementwise_clipped_grad(Hbar: torch.Tensor, Zbar: torch.Tensor, clip: Optional[torch.Tensor],
                                    g_scale: torch.Tensor, g_shift: Optional[torch.Tensor], stream=None) -> None:
    B, T, d, ldh = _rows(Hbar)
    B2, T2, d2, ldz = _rows(Zbar)
    assert (B, T, d) == (B2, T2, d2) and Hbar.dtype == Zbar.dtype
    assert g_scale.dtype == torch.float32 and g_scale.numel() == d and g_scale.is_contiguous()
    assert g_shift is None or (g_shift.dtype == torch.float32 and g_shift.numel() == d and g_shift.is_contiguous())
    assert clip is None or (clip.dtype == torch.float32 and clip.numel() >= B and clip.is_contiguous())
    _check("dpclip_elementwise_clipped_grad", load_library().dpclip_elementwise_clipped_grad(
        _ptr(Hbar), ldh, _ptr(Zbar), ldz, B, T, d, _dtype_code(Hbar), _ptr(clip) if clip is not None else None,
        _ptr(g_scale), _ptr(g_shift) if g_shift is not None else None, _stream(stream)))


# ----------------------------------------------------------------------------
# whole step
# ----------------------------------------------------------------------------
@dataclass
class Layer:
    A: torch.Tensor            # (B, T, d_in)
    Zbar: torch.Tensor         # (B, T, d_out)
    has_bias: bool = True
    method: int = DPCLIP_AUTO


class StepPlan:
    """Buffers and the C descriptor array for repeated whole-step calls on one
    set of layer shapes.  Holds no arithmetic: `run` is one dpclip_step call."""

    def __init__(self, layers: Sequence[Layer], device=None):
        self.layers = list(layers)
        self.L = len(self.layers)
        dev = device or self.layers[0].A.device
        self.B = self.layers[0].A.shape[0]
        self.dtype_code = _dtype_code(self.layers[0].A)
        self.gW: List[torch.Tensor] = []
        self.gb: List[Optional[torch.Tensor]] = []
        self._c = (_CLayer * self.L)()
        # all outputs live in one flat fp32 buffer (each tensor starts on a 256-byte boundary), so a
        # data-parallel caller can all-reduce the whole gradient with one collective
        offs, total = [], 0
        for y in self.layers:
            d_in, d_out = y.A.shape[-1], y.Zbar.shape[-1]
            ow = total; total += -(-d_out * d_in // 64) * 64
            ob = total; total += (-(-d_out // 64) * 64) if y.has_bias else 0
            offs.append((ow, ob))
        self.flat = torch.zeros((total,), dtype=torch.float32, device=dev)
        for l, y in enumerate(self.layers):
            B, T, d_in, lda = _rows(y.A)
            _, _, d_out, ldz = _rows(y.Zbar)
            assert B == self.B and _dtype_code(y.A) == self.dtype_code
            ow, ob = offs[l]
            gW = self.flat[ow:ow + d_out * d_in].view(d_out, d_in)
            gb = self.flat[ob:ob + d_out] if y.has_bias else None
            self.gW.append(gW); self.gb.append(gb)
            self._c[l] = _CLayer(_ptr(y.A), lda, _ptr(y.Zbar), ldz, T, d_in, d_out, int(y.has_bias),
                                 y.method, _ptr(gW), d_in, _ptr(gb))
        ws = dpclip_step_workspace_bytes(self)
        self.sq_layers = torch.empty((self.L, self.B), dtype=torch.float32, device=dev)
        self.clip = torch.empty((self.B,), dtype=torch.float32, device=dev)
        self.norms = torch.empty((self.B,), dtype=torch.float32, device=dev)
        self.workspace = torch.empty((ws,), dtype=torch.uint8, device=dev)
        dpclip_workspace_init(self.workspace)

    def run(self, C: float, sigma: float, seed: int, stream_id0: int = 0, stream=None) -> None:
        dpclip_step(self, C, sigma, seed, stream_id0, stream)

    def _branches(self, branches: int):
        """Side streams and their workspaces for the several-streams entry points (allocated once)."""
        if len(getattr(self, "_branch_ws", [])) < branches:
            self._branch_ws = [self.workspace] + [torch.empty_like(self.workspace) for _ in range(branches - 1)]
            for w in self._branch_ws[1:]:
                dpclip_workspace_init(w)
            self._streams = [torch.cuda.Stream() for _ in range(branches - 1)]
            torch.cuda.synchronize()
        return self._streams[:branches - 1], self._branch_ws[:branches]

    def run_streams(self, C: float, sigma: float, seed: int, stream_id0: int = 0, branches: int = 4) -> None:
        """One dpclip_step_streams call: the library spreads the launches of a stage over `branches` streams,
        starting from and joining back into the current stream."""
        side, ws = self._branches(branches)
        dpclip_step_streams(self, C, sigma, seed, stream_id0, [torch.cuda.current_stream()] + side, ws)

    def workspaces(self) -> List[torch.Tensor]:
        """Every workspace the plan has used (their status words are checked separately)."""
        return list(getattr(self, "_branch_ws", [self.workspace]))

    def capture(self, C: float, sigma: float, seed: int, stream_id0: int = 0, branches: int = 1):
        """Record one step into a CUDA graph (the launch-bound small workloads spend most of a step
        in launch gaps).  Returns the graph; `graph.replay()` re-runs the same kernels on the same
        buffers with the same (C, sigma, seed, stream ids).  The graph holds exactly ONE library call:
        dpclip_step (branches = 1) or dpclip_step_streams (the fork/join over `branches` streams happens
        inside the library and becomes the graph's parallel branches)."""
        step = self.run if branches <= 1 else (lambda *a: self.run_streams(*a, branches=branches))
        step(C, sigma, seed, stream_id0)               # warm-up outside capture (function attributes, maps)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step(C, sigma, seed, stream_id0)
        return graph


def _conv_args(X: torch.Tensor, Zbar: torch.Tensor, kh: int, kw: int, stride: int, pad: int, z_channel_major: bool):
    assert X.dim() == 4 and X.is_contiguous() and Zbar.is_contiguous() and X.dtype == Zbar.dtype
    B, C, H, W = X.shape
    Ho, Wo = (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1
    if z_channel_major:
        d_out = Zbar.shape[1]
        assert Zbar.numel() == B * d_out * Ho * Wo
    else:
        d_out = Zbar.shape[-1]
        assert Zbar.numel() == B * Ho * Wo * d_out
    return B, d_out, _CConv(C, H, W, kh, kw, stride, pad)


def dpclip_conv_workspace_bytes(X: torch.Tensor, Zbar: torch.Tensor, kh: int, kw: int, stride: int, pad: int,
                                z_channel_major: bool = False) -> int:
    B, d_out, geom = _conv_args(X, Zbar, kh, kw, stride, pad, z_channel_major)
    return load_library().dpclip_conv_workspace_bytes(B, ctypes.byref(geom), d_out, _dtype_code(X), int(z_channel_major))


def dpclip_conv_sqnorms(X: torch.Tensor, Zbar: torch.Tensor, kh: int, kw: int, stride: int, pad: int, has_bias: bool,
                        sq_layer: torch.Tensor, z_channel_major: bool = False,
                        workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    B, d_out, geom = _conv_args(X, Zbar, kh, kw, stride, pad, z_channel_major)
    assert sq_layer.dtype == torch.float32 and sq_layer.numel() >= B and sq_layer.is_contiguous()
    _check("dpclip_conv_sqnorms", load_library().dpclip_conv_sqnorms(
        _ptr(X), _ptr(Zbar), int(z_channel_major), B, ctypes.byref(geom), d_out, _dtype_code(X), int(has_bias),
        _ptr(sq_layer), _ptr(workspace) if workspace is not None else None,
        workspace.numel() if workspace is not None else 0, _stream(stream)))


def dpclip_conv_clipped_grad(X: torch.Tensor, Zbar: torch.Tensor, kh: int, kw: int, stride: int, pad: int,
                             clip: Optional[torch.Tensor], gW: torch.Tensor, gb: Optional[torch.Tensor],
                             z_channel_major: bool = False, workspace: Optional[torch.Tensor] = None,
                             stream=None) -> None:
    B, d_out, geom = _conv_args(X, Zbar, kh, kw, stride, pad, z_channel_major)
    d_in = X.shape[1] * kh * kw
    assert gW.dtype == torch.float32 and gW.shape == (d_out, d_in) and gW.stride(1) == 1
    assert gb is None or (gb.dtype == torch.float32 and gb.numel() == d_out and gb.is_contiguous())
    _check("dpclip_conv_clipped_grad", load_library().dpclip_conv_clipped_grad(
        _ptr(X), _ptr(Zbar), int(z_channel_major), B, ctypes.byref(geom), d_out, _dtype_code(X),
        _ptr(clip) if clip is not None else None, _ptr(gW), gW.stride(0), _ptr(gb) if gb is not None else None,
        _ptr(workspace) if workspace is not None else None, workspace.numel() if workspace is not None else 0,
        _stream(stream)))


def dpclip_dp_sgd_step(theta: torch.Tensor, gsum: torch.Tensor, inv_tau: float, C: float, sigma: float, seed: int,
                       stream_id: int, lr: float, stream=None) -> None:
    assert theta.dtype == gsum.dtype == torch.float32 and theta.is_contiguous() and gsum.is_contiguous()
    assert theta.numel() == gsum.numel()
    _check("dpclip_dp_sgd_step", load_library().dpclip_dp_sgd_step(
        _ptr(theta), _ptr(gsum), theta.numel(), inv_tau, C, sigma, seed, stream_id, lr, _stream(stream)))


def dpclip_dp_adam_step(theta: torch.Tensor, m: torch.Tensor, v: torch.Tensor, gsum: torch.Tensor, inv_tau: float,
                        C: float, sigma: float, seed: int, stream_id: int, lr: float, beta1: float, beta2: float,
                        eps: float, step: int, stream=None) -> None:
    for t in (theta, m, v, gsum):
        assert t.dtype == torch.float32 and t.is_contiguous() and t.numel() == theta.numel()
    _check("dpclip_dp_adam_step", load_library().dpclip_dp_adam_step(
        _ptr(theta), _ptr(m), _ptr(v), _ptr(gsum), theta.numel(), inv_tau, C, sigma, seed, stream_id, lr, beta1, beta2,
        eps, step, _stream(stream)))


def dpclip_step_noise(plan: StepPlan, C: float, sigma: float, seed: int, stream_id0: int = 0, stream=None) -> None:
    _check("dpclip_step_noise", load_library().dpclip_step_noise(plan._c, plan.L, C, sigma, seed, stream_id0,
                                                                 _stream(stream)))


def dpclip_t1_layers_sqnorms(plan: StepPlan, stream=None) -> None:
    _check("dpclip_t1_layers_sqnorms", load_library().dpclip_t1_layers_sqnorms(
        plan._c, plan.L, plan.B, plan.dtype_code, _ptr(plan.sq_layers), _stream(stream)))


def dpclip_t1_layers_clipped_grad_noise(plan: StepPlan, C: float, sigma: float, seed: int, stream_id0: int = 0,
                                        workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    ws = plan.workspace if workspace is None else workspace
    _check("dpclip_t1_layers_clipped_grad_noise", load_library().dpclip_t1_layers_clipped_grad_noise(
        plan._c, plan.L, plan.B, plan.dtype_code, _ptr(plan.clip), C, sigma, seed, stream_id0, _ptr(ws), ws.numel(),
        _stream(stream)))


def dpclip_gram_layers_sqnorms(plan: StepPlan, workspace: Optional[torch.Tensor] = None, stream=None) -> List[bool]:
    """Norms of the plan's Gram-method layers in one launch; returns which layers were taken."""
    ws = plan.workspace if workspace is None else workspace
    taken = (ctypes.c_int * plan.L)()
    _check("dpclip_gram_layers_sqnorms", load_library().dpclip_gram_layers_sqnorms(
        plan._c, plan.L, plan.B, plan.dtype_code, _ptr(plan.sq_layers), taken, _ptr(ws), ws.numel(), _stream(stream)))
    return [bool(t) for t in taken]


def dpclip_same_shape_layers_clipped_grad_noise(plan: StepPlan, C: float, sigma: float, seed: int, stream_id0: int = 0,
                                                workspace: Optional[torch.Tensor] = None, stream=None) -> List[bool]:
    """Clipped sums + noise of the plan's same-shape layer groups, one launch per group; returns which
    layers were taken."""
    ws = plan.workspace if workspace is None else workspace
    taken = (ctypes.c_int * plan.L)()
    _check("dpclip_same_shape_layers_clipped_grad_noise", load_library().dpclip_same_shape_layers_clipped_grad_noise(
        plan._c, plan.L, plan.B, plan.dtype_code, _ptr(plan.clip), C, sigma, seed, stream_id0, taken, _ptr(ws),
        ws.numel(), _stream(stream)))
    return [bool(t) for t in taken]


def dpclip_t1_layers_supported(plan: StepPlan) -> bool:
    """Whether the library takes the plan's T = 1 layers together (nothing is launched)."""
    return bool(load_library().dpclip_t1_layers_supported(plan._c, plan.L, plan.B, plan.dtype_code))


def dpclip_step_workspace_bytes(plan) -> int:
    """Workspace for whole-step calls over the plan's layers (per-layer needs and shared launches)."""
    return load_library().dpclip_step_workspace_bytes(plan._c, plan.L, plan.B, plan.dtype_code)


def dpclip_step(plan: StepPlan, C: float, sigma: float, seed: int, stream_id0: int = 0, stream=None) -> None:
    _check("dpclip_step", load_library().dpclip_step(
        plan._c, plan.L, plan.B, plan.dtype_code, C, sigma, seed, stream_id0, _ptr(plan.sq_layers),
        _ptr(plan.clip), _ptr(plan.norms), _ptr(plan.workspace), plan.workspace.numel(), _stream(stream)))


def _stream_args(streams, workspaces):
    n = len(streams)
    assert n == len(workspaces) and all(w.numel() == workspaces[0].numel() for w in workspaces)
    st = (_vp * n)(*[s.cuda_stream for s in streams])
    ws = (_vp * n)(*[w.data_ptr() for w in workspaces])
    return n, st, ws, workspaces[0].numel()


def dpclip_step_streams(plan: StepPlan, C: float, sigma: float, seed: int, stream_id0: int, streams, workspaces) -> None:
    """dpclip_step with the library forking over `streams` (torch streams; streams[0] = the caller's)."""
    n, st, ws, nbytes = _stream_args(streams, workspaces)
    _check("dpclip_step_streams", load_library().dpclip_step_streams(
        plan._c, plan.L, plan.B, plan.dtype_code, C, sigma, seed, stream_id0, _ptr(plan.sq_layers), _ptr(plan.clip),
        _ptr(plan.norms), n, st, ws, nbytes))


def dpclip_model_step_streams(plan, C: float, sigma: float, seed: int, stream_id0: int, streams, workspaces) -> None:
    n, st, ws, nbytes = _stream_args(streams, workspaces)
    _check("dpclip_model_step_streams", load_library().dpclip_model_step_streams(
        plan._c, plan.L, plan.B, plan.dtype_code, C, sigma, seed, stream_id0, _ptr(plan.sq_layers), _ptr(plan.clip),
        _ptr(plan.norms), n, st, ws, nbytes))


DPCLIP_KIND_DENSE, DPCLIP_KIND_ELEMENTWISE, DPCLIP_KIND_CONV = 0, 1, 2


@dataclass
class ModelLayer:
    """One layer of a model for dpclip_model_step.
    dense:        A (B, T, d_in), Zbar (B, T, d_out)
    element-wise: A = hbar (B, T, d), Zbar (B, T, d); has_bias = the layer has a shift
    conv:         A = X (B, C, H, W), Zbar (B, Ho*Wo, d_out) or, z_channel_major, (B, d_out, Ho*Wo);
                  conv = (kh, kw, stride, pad)"""
    kind: int
    A: torch.Tensor
    Zbar: torch.Tensor
    has_bias: bool = True
    method: int = DPCLIP_AUTO
    conv: Optional[tuple] = None
    z_channel_major: bool = False


class ModelPlan(StepPlan):
    """Buffers and the C descriptor array of a model with dense, element-wise and convolution layers.
    Holds no arithmetic: `run` is one dpclip_model_step call, `run_streams` one dpclip_model_step_streams call
    (which `capture` with several branches records).  gW[l] is (d_out, d_in)
    for dense and convolution layers (d_in = C*kh*kw) and (d,) for element-wise layers; all live in `flat`."""

    def __init__(self, layers: Sequence[ModelLayer], device=None):
        self.layers = list(layers)
        self.L = len(self.layers)
        dev = device or self.layers[0].A.device
        self.B = self.layers[0].A.shape[0]
        self.dtype_code = _dtype_code(self.layers[0].A)
        self._c = (_CModelLayer * self.L)()
        shapes, total = [], 0
        for y in self.layers:
            assert y.A.shape[0] == self.B and _dtype_code(y.A) == self.dtype_code and y.A.dtype == y.Zbar.dtype
            if y.kind == DPCLIP_KIND_DENSE:
                w_shape, nb = (y.Zbar.shape[-1], y.A.shape[-1]), y.Zbar.shape[-1]
            elif y.kind == DPCLIP_KIND_ELEMENTWISE:
                assert y.A.shape == y.Zbar.shape
                w_shape, nb = (y.A.shape[-1],), y.A.shape[-1]
            elif y.kind == DPCLIP_KIND_CONV:
                kh, kw, stride, pad = y.conv
                _, d_out, _ = _conv_args(y.A, y.Zbar, kh, kw, stride, pad, y.z_channel_major)
                w_shape, nb = (d_out, y.A.shape[1] * kh * kw), d_out
            else:
                raise ValueError(f"unknown layer kind {y.kind}")
            nw = 1
            for v in w_shape:
                nw *= v
            ow = total; total += -(-nw // 64) * 64
            ob = total; total += (-(-nb // 64) * 64) if y.has_bias else 0
            shapes.append((w_shape, nw, ow, nb, ob))
        self.flat = torch.zeros((total,), dtype=torch.float32, device=dev)
        self.gW: List[torch.Tensor] = []
        self.gb: List[Optional[torch.Tensor]] = []
        for l, (y, (w_shape, nw, ow, nb, ob)) in enumerate(zip(self.layers, shapes)):
            gW = self.flat[ow:ow + nw].view(*w_shape)
            gb = self.flat[ob:ob + nb] if y.has_bias else None
            self.gW.append(gW); self.gb.append(gb)
            c = self._c[l]
            c.kind = y.kind
            if y.kind == DPCLIP_KIND_CONV:
                kh, kw, stride, pad = y.conv
                _, d_out, geom = _conv_args(y.A, y.Zbar, kh, kw, stride, pad, y.z_channel_major)
                c.conv = geom
                c.z_channel_major = int(y.z_channel_major)
                c.layer = _CLayer(_ptr(y.A), 0, _ptr(y.Zbar), 0, 0, w_shape[1], d_out, int(y.has_bias), y.method,
                                  _ptr(gW), w_shape[1], _ptr(gb))
            else:
                B, T, d_in, lda = _rows(y.A)
                _, _, d_out, ldz = _rows(y.Zbar)
                c.layer = _CLayer(_ptr(y.A), lda, _ptr(y.Zbar), ldz, T, d_in, d_out, int(y.has_bias), y.method,
                                  _ptr(gW), d_in, _ptr(gb))
        self.sq_layers = torch.empty((self.L, self.B), dtype=torch.float32, device=dev)
        self.clip = torch.empty((self.B,), dtype=torch.float32, device=dev)
        self.norms = torch.empty((self.B,), dtype=torch.float32, device=dev)
        ws = dpclip_model_workspace_bytes(self)
        self.workspace = torch.empty((ws,), dtype=torch.uint8, device=dev)
        dpclip_workspace_init(self.workspace)

    def run(self, C: float, sigma: float, seed: int, stream_id0: int = 0, stream=None) -> None:
        dpclip_model_step(self, C, sigma, seed, stream_id0, stream)

    def run_streams(self, C: float, sigma: float, seed: int, stream_id0: int = 0, branches: int = 4) -> None:
        side, ws = self._branches(branches)
        dpclip_model_step_streams(self, C, sigma, seed, stream_id0, [torch.cuda.current_stream()] + side, ws)


def dpclip_step_per_layer(plan: StepPlan, C_layer: Sequence[float], sigma: float, seed: int, stream_id0: int = 0,
                          clip_layers: Optional[torch.Tensor] = None, norms_layers: Optional[torch.Tensor] = None,
                          stream=None) -> torch.Tensor:
    """Per-layer clipping over the plan's (dense) layers; returns the (L, B) factors."""
    assert len(C_layer) == plan.L
    if clip_layers is None:
        clip_layers = torch.empty((plan.L, plan.B), dtype=torch.float32, device=plan.sq_layers.device)
    assert clip_layers.dtype == torch.float32 and clip_layers.shape == (plan.L, plan.B) and clip_layers.is_contiguous()
    assert norms_layers is None or (norms_layers.dtype == torch.float32 and norms_layers.shape == (plan.L, plan.B)
                                    and norms_layers.is_contiguous())
    c = (ctypes.c_float * plan.L)(*[float(v) for v in C_layer])
    _check("dpclip_step_per_layer", load_library().dpclip_step_per_layer(
        plan._c, plan.L, plan.B, plan.dtype_code, c, sigma, seed, stream_id0, _ptr(plan.sq_layers), _ptr(clip_layers),
        _ptr(norms_layers) if norms_layers is not None else None, _ptr(plan.workspace), plan.workspace.numel(),
        _stream(stream)))
    return clip_layers


def dpclip_model_workspace_bytes(plan: ModelPlan) -> int:
    return load_library().dpclip_model_workspace_bytes(plan._c, plan.L, plan.B, plan.dtype_code)


def dpclip_model_step(plan: ModelPlan, C: float, sigma: float, seed: int, stream_id0: int = 0, stream=None) -> None:
    _check("dpclip_model_step", load_library().dpclip_model_step(
        plan._c, plan.L, plan.B, plan.dtype_code, C, sigma, seed, stream_id0, _ptr(plan.sq_layers),
        _ptr(plan.clip), _ptr(plan.norms), _ptr(plan.workspace), plan.workspace.numel(), _stream(stream)))


class HostStep:
    """Whole step for tensors that live in (pinned) host memory: inputs are
    copied to the device, the path runs, outputs are copied back, all inside
    one dpclip_step_host call enqueued on the current stream."""

    def __init__(self, host_layers: Sequence[Layer], device="cuda", pack_inputs: bool = False):
        """Results always live in one pinned buffer carved up in the library's arena order, so they come
        back in one copy.  pack_inputs=True also copies the given host tensors, once, into one pinned
        buffer in arena order (`self.layers` then holds views of it for the caller to refill every step),
        so the inputs go up in one copy too."""
        self.layers = list(host_layers)
        self.L = len(self.layers)
        self.B = self.layers[0].A.shape[0]
        self.dtype_code = _dtype_code(self.layers[0].A)
        self._c = (_CLayer * self.L)()
        self.gW, self.gb = [], []
        self.h2d_bytes = 0
        self.d2h_bytes = 0
        up = lambda n: (n + 255) // 256 * 256                                   # noqa: E731
        shapes = []
        for y in self.layers:
            assert not y.A.is_cuda and y.A.is_contiguous() and y.Zbar.is_contiguous()
            B, T, d_in, _ = _rows(y.A)
            _, _, d_out, _ = _rows(y.Zbar)
            shapes.append((T, d_in, d_out))
        es = self.layers[0].A.element_size()
        if pack_inputs:
            total = sum(up(self.B * T * d_in * es) + up(self.B * T * d_out * es) for T, d_in, d_out in shapes)
            self._in_flat = torch.empty((total,), dtype=torch.uint8).pin_memory()
            off, packed = 0, []
            for y, (T, d_in, d_out) in zip(self.layers, shapes):
                na, nz = self.B * T * d_in * es, self.B * T * d_out * es
                a = self._in_flat[off:off + na].view(y.A.dtype).view(y.A.shape); off += up(na)
                z = self._in_flat[off:off + nz].view(y.Zbar.dtype).view(y.Zbar.shape); off += up(nz)
                a.copy_(y.A); z.copy_(y.Zbar)
                packed.append(Layer(a, z, y.has_bias, y.method))
            self.layers = packed
        total = sum(up(d_out * d_in * 4) + up(d_out * 4) for _, d_in, d_out in shapes) + 2 * up(self.B * 4)
        self._out_flat = torch.empty((total,), dtype=torch.uint8).pin_memory()
        off = 0
        for l, (y, (T, d_in, d_out)) in enumerate(zip(self.layers, shapes)):
            gW = self._out_flat[off:off + d_out * d_in * 4].view(torch.float32).view(d_out, d_in); off += up(d_out * d_in * 4)
            gb = self._out_flat[off:off + d_out * 4].view(torch.float32) if y.has_bias else None; off += up(d_out * 4)
            self.gW.append(gW); self.gb.append(gb)
            self._c[l] = _CLayer(_ptr(y.A), d_in, _ptr(y.Zbar), d_out, T, d_in, d_out, int(y.has_bias),
                                 y.method, _ptr(gW), d_in, _ptr(gb))
            self.h2d_bytes += y.A.numel() * y.A.element_size() + y.Zbar.numel() * y.Zbar.element_size()
            self.d2h_bytes += gW.numel() * 4 + (gb.numel() * 4 if gb is not None else 0)
        self.clip = self._out_flat[off:off + self.B * 4].view(torch.float32); off += up(self.B * 4)
        self.norms = self._out_flat[off:off + self.B * 4].view(torch.float32)
        # the merged device-to-host copy ends with the last float of `norms`: what lies behind it is not the
        # library's to write (the bytes up to the 256-byte boundary are kept as a guard band for the tests)
        self._out_end = off + self.B * 4
        self._out_flat[self._out_end:].fill_(0xA5)
        self.d2h_bytes += 8 * self.B
        nbytes = load_library().dpclip_step_host_arena_bytes(self._c, self.L, self.B, self.dtype_code)
        self.arena = torch.empty((nbytes,), dtype=torch.uint8, device=device)

    def run(self, C: float, sigma: float, seed: int, stream_id0: int = 0, stream=None) -> None:
        dpclip_step_host(self, C, sigma, seed, stream_id0, stream)


def dpclip_step_host(hs: HostStep, C: float, sigma: float, seed: int, stream_id0: int = 0, stream=None) -> None:
    _check("dpclip_step_host", load_library().dpclip_step_host(
        hs._c, hs.L, hs.B, hs.dtype_code, C, sigma, seed, stream_id0, _ptr(hs.clip), _ptr(hs.norms),
        _ptr(hs.arena), hs.arena.numel(), _stream(stream)))
