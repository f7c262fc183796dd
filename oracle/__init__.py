"""TEST INFRASTRUCTURE ONLY: ctypes access to the fp64 CPU oracle.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It builds `dpclip_oracle.c` with gcc on first use (into
`oracle/_build/`) and exposes thin numpy wrappers; there is no arithmetic of
the method in this file, only argument marshalling.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dpclip_oracle.c")
_BUILD = os.path.join(_HERE, "_build")
_SO = os.path.join(_BUILD, "libdpclip_oracle.so")
_lock = threading.Lock()
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the oracle (plain C, no CUDA).  Returns the library path."""
    os.makedirs(_BUILD, exist_ok=True)
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
                               _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            L.oracle_example_grad.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_int, _dp, _dp]
            L.oracle_example_grad.restype = None
            L.oracle_layer_sqnorms.argtypes = [_dp, _dp] + [ctypes.c_int] * 5 + [_dp]
            L.oracle_layer_sqnorms.restype = ctypes.c_int
            L.oracle_factors.argtypes = [_dp, ctypes.c_int, ctypes.c_int, ctypes.c_double, _dp, _dp]
            L.oracle_factors.restype = None
            L.oracle_clipped_grad.argtypes = [_dp, _dp] + [ctypes.c_int] * 4 + [_dp, _dp, _dp]
            L.oracle_clipped_grad.restype = ctypes.c_int
            u32p = ctypes.POINTER(ctypes.c_uint32)
            L.oracle_elementwise_example_grad.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, _dp, _dp]
            L.oracle_elementwise_example_grad.restype = None
            L.oracle_elementwise_sqnorms.argtypes = [_dp, _dp] + [ctypes.c_int] * 4 + [_dp]
            L.oracle_elementwise_sqnorms.restype = ctypes.c_int
            L.oracle_elementwise_clipped_grad.argtypes = [_dp, _dp] + [ctypes.c_int] * 3 + [_dp, _dp, _dp]
            L.oracle_elementwise_clipped_grad.restype = ctypes.c_int
            L.oracle_dp_sgd_step.argtypes = [_dp, _dp, ctypes.c_size_t, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                             ctypes.c_uint64, ctypes.c_uint64, ctypes.c_double]
            L.oracle_dp_sgd_step.restype = ctypes.c_int
            L.oracle_dp_adam_step.argtypes = [_dp, _dp, _dp, _dp, ctypes.c_size_t] + [ctypes.c_double] * 3 + \
                                             [ctypes.c_uint64, ctypes.c_uint64] + [ctypes.c_double] * 4 + [ctypes.c_int]
            L.oracle_dp_adam_step.restype = ctypes.c_int
            L.oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
            L.oracle_philox4x32_10.restype = None
            L.oracle_normals.argtypes = [ctypes.c_size_t, ctypes.c_uint64, ctypes.c_uint64, _dp]
            L.oracle_normals.restype = None
            L.oracle_add_noise.argtypes = [_dp, ctypes.c_size_t, ctypes.c_double, ctypes.c_double,
                                           ctypes.c_uint64, ctypes.c_uint64]
            L.oracle_add_noise.restype = ctypes.c_int
            _lib = L
    return _lib


def _f64(x) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.float64)


def _p(x: np.ndarray):
    return x.ctypes.data_as(_dp)


def example_grad(A_i, Z_i) -> Tuple[np.ndarray, np.ndarray]:
    """A_i: (T, d_in), Z_i: (T, d_out) -> (G_i (d_out, d_in), gb_i (d_out,))."""
    A_i, Z_i = _f64(A_i), _f64(Z_i)
    T, d_in = A_i.shape
    d_out = Z_i.shape[1]
    assert Z_i.shape[0] == T
    G = np.empty((d_out, d_in)); gb = np.empty(d_out)
    lib().oracle_example_grad(_p(A_i), _p(Z_i), T, d_in, d_out, _p(G), _p(gb))
    return G, gb


def layer_sqnorms(A, Z, has_bias: bool) -> np.ndarray:
    """A: (B, T, d_in), Z: (B, T, d_out) -> squared per-example norms (B,)."""
    A, Z = _f64(A), _f64(Z)
    B, T, d_in = A.shape
    d_out = Z.shape[2]
    assert Z.shape[:2] == (B, T)
    sq = np.empty(B)
    if lib().oracle_layer_sqnorms(_p(A), _p(Z), B, T, d_in, d_out, int(has_bias), _p(sq)):
        raise MemoryError
    return sq


def factors(sq_layers, C: float) -> Tuple[np.ndarray, np.ndarray]:
    """sq_layers: (L, B) -> (norms (B,), clip (B,))."""
    sq_layers = _f64(sq_layers)
    L, B = sq_layers.shape
    norms = np.empty(B); clip = np.empty(B)
    lib().oracle_factors(_p(sq_layers), L, B, float(C), _p(norms), _p(clip))
    return norms, clip


def clipped_grad(A, Z, clip: Optional[np.ndarray]) -> Tuple[np.ndarray, np.ndarray]:
    """-> (gW (d_out, d_in), gb (d_out,)), the clipped sums before noise."""
    A, Z = _f64(A), _f64(Z)
    B, T, d_in = A.shape
    d_out = Z.shape[2]
    gW = np.empty((d_out, d_in)); gb = np.empty(d_out)
    cp = None
    if clip is not None:
        clip = _f64(clip); assert clip.shape == (B,)
        cp = _p(clip)
    if lib().oracle_clipped_grad(_p(A), _p(Z), B, T, d_in, d_out, cp, _p(gW), _p(gb)):
        raise MemoryError
    return gW, gb


def elementwise_example_grad(H_i, Z_i) -> Tuple[np.ndarray, np.ndarray]:
    """H_i, Z_i: (T, d) -> (ggamma_i (d,), gbeta_i (d,)) of a LayerNorm-style gain/shift pair."""
    H_i, Z_i = _f64(H_i), _f64(Z_i)
    T, d = H_i.shape
    assert Z_i.shape == (T, d)
    gg = np.empty(d); gs = np.empty(d)
    lib().oracle_elementwise_example_grad(_p(H_i), _p(Z_i), T, d, _p(gg), _p(gs))
    return gg, gs


def elementwise_sqnorms(H, Z, has_shift: bool) -> np.ndarray:
    """H, Z: (B, T, d) -> squared per-example norms (B,) of the gain (and shift) gradients."""
    H, Z = _f64(H), _f64(Z)
    B, T, d = H.shape
    assert Z.shape == (B, T, d)
    sq = np.empty(B)
    if lib().oracle_elementwise_sqnorms(_p(H), _p(Z), B, T, d, int(has_shift), _p(sq)):
        raise MemoryError
    return sq


def elementwise_clipped_grad(H, Z, clip: Optional[np.ndarray]) -> Tuple[np.ndarray, np.ndarray]:
    """-> (g_scale (d,), g_shift (d,)), the clipped sums before noise."""
    H, Z = _f64(H), _f64(Z)
    B, T, d = H.shape
    g_scale = np.empty(d); g_shift = np.empty(d)
    cp = None
    if clip is not None:
        clip = _f64(clip); assert clip.shape == (B,)
        cp = _p(clip)
    if lib().oracle_elementwise_clipped_grad(_p(H), _p(Z), B, T, d, cp, _p(g_scale), _p(g_shift)):
        raise MemoryError
    return g_scale, g_shift


def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> List[int]:
    c = (ctypes.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    o = (ctypes.c_uint32 * 4)()
    lib().oracle_philox4x32_10(c, k, o)
    return list(o)


def normals(n: int, seed: int, stream_id: int) -> np.ndarray:
    xi = np.empty(max(n, 1))
    lib().oracle_normals(n, seed, stream_id, _p(xi))
    return xi[:n]


def add_noise(g, sigma: float, C: float, seed: int, stream_id: int) -> np.ndarray:
    out = _f64(g).copy()
    flat = out.reshape(-1)
    if lib().oracle_add_noise(_p(flat), flat.size, float(sigma), float(C), seed, stream_id):
        raise MemoryError
    return out


def dp_sgd_step(theta, gsum, inv_tau: float, C: float, sigma: float, seed: int, stream_id: int, lr: float) -> np.ndarray:
    """theta - lr * (gsum + sigma C xi) / tau (Algorithm 1's update); returns the new parameters."""
    th = _f64(theta).copy().reshape(-1); g = _f64(gsum).reshape(-1)
    if lib().oracle_dp_sgd_step(_p(th), _p(g), th.size, inv_tau, C, sigma, seed, stream_id, lr):
        raise MemoryError
    return th.reshape(np.shape(theta))


def dp_adam_step(theta, m, v, gsum, inv_tau: float, C: float, sigma: float, seed: int, stream_id: int, lr: float,
                 beta1: float, beta2: float, eps: float, t: int):
    """One step of the private Adam; returns (theta, m, v) after the step."""
    th = _f64(theta).copy().reshape(-1); mm = _f64(m).copy().reshape(-1); vv = _f64(v).copy().reshape(-1)
    g = _f64(gsum).reshape(-1)
    if lib().oracle_dp_adam_step(_p(th), _p(mm), _p(vv), _p(g), th.size, inv_tau, C, sigma, seed, stream_id, lr,
                                 beta1, beta2, eps, t):
        raise MemoryError
    sh = np.shape(theta)
    return th.reshape(sh), mm.reshape(sh), vv.reshape(sh)


def step(layers, has_bias: Sequence[bool], C: float, sigma: float, seed: int, stream_id0: int = 0):
    """Whole path over [(A_l, Z_l)].  Noise stream ids: stream_id0 + 2l for
    layer l's weights, + 2l + 1 for its bias.  Returns a dict of
    sq_layers, norms, clip, gW, gb (pre-noise), outW, outb (noised)."""
    sq = np.stack([layer_sqnorms(A, Z, hb) for (A, Z), hb in zip(layers, has_bias)])
    norms, clip = factors(sq, C)
    gW, gb, outW, outb = [], [], [], []
    for l, ((A, Z), hb) in enumerate(zip(layers, has_bias)):
        w, b = clipped_grad(A, Z, clip)
        gW.append(w); gb.append(b)
        outW.append(add_noise(w, sigma, C, seed, stream_id0 + 2 * l))
        outb.append(add_noise(b, sigma, C, seed, stream_id0 + 2 * l + 1) if hb else None)
    return dict(sq_layers=sq, norms=norms, clip=clip, gW=gW, gb=gb, outW=outW, outb=outb)
