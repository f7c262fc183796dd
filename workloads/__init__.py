"""Seeded synthetic inputs for the per-example-clipping hot path.

This module is the only code shared by the CPU oracle's tests and the CUDA
path's tests/benchmark.  It holds NONE of the method's arithmetic: it only
describes layer shapes and draws (A_l, Zbar_l) tensors with the value
distributions of the paper's workloads (dense MLPs, an im2col'd CNN,
sequence-model projections) from a seeded numpy generator.

Conventions
-----------
* A_l has shape (B, T, d_in), Zbar_l has shape (B, T, d_out); T = 1 for a
  dense layer, T = H'*W' for an im2col'd convolution, T = sequence length
  for recurrent / attention projections.
* "N(0, v)" is read as mean 0, VARIANCE v.
* For dtype "bf16" values are rounded to bfloat16 (round-to-nearest-even)
  here, so that both consumers start from identical numbers; arrays are
  returned as float32 holding exactly-representable bf16 values, and
  `to_bf16_bits` gives the uint16 payload for the device.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np


# --------------------------------------------------------------------------
# shapes
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class LayerSpec:
    name: str
    T: int
    d_in: int
    d_out: int
    has_bias: bool = True
    a_dist: str = "normal"          # "normal" | "relu" | "im2col"
    # im2col only: feature map (c_in, H, W), square kernel k, zero padding p
    conv: Optional[Tuple[int, int, int, int, int]] = None

    @property
    def n_params(self) -> int:
        return self.d_in * self.d_out + (self.d_out if self.has_bias else 0)


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    dtype: str                      # "f32" | "bf16"
    layers: Tuple[LayerSpec, ...]
    C: float
    sigma: float
    zbar_var: float                 # variance of every Zbar entry
    note: str = ""

    @property
    def n_params(self) -> int:
        return sum(l.n_params for l in self.layers)

    def input_bytes(self) -> int:
        es = 4 if self.dtype == "f32" else 2
        return sum(self.B * l.T * (l.d_in + l.d_out) * es for l in self.layers)


def _dense(name, d_in, d_out, a_dist, bias=True):
    return LayerSpec(name, 1, d_in, d_out, bias, a_dist)


def mlp_small(dtype="f32") -> Workload:
    """MLP 784->256->10, B=32 (two dense layers + biases)."""
    B = 32
    return Workload("mlp_784_256_10_b32" + ("" if dtype == "f32" else "_" + dtype), B, dtype,
                    (_dense("fc1", 784, 256, "normal"), _dense("fc2", 256, 10, "relu")),
                    C=1.0, sigma=1.1, zbar_var=1.0 / B)


def mlp_large(dtype="f32", C=1.0) -> Workload:
    """MLP 784->1000->1000->10, B=128 (three dense layers + biases)."""
    B = 128
    return Workload("mlp_784_1000_1000_10_b128" + ("" if dtype == "f32" else "_" + dtype), B, dtype,
                    (_dense("fc1", 784, 1000, "normal"), _dense("fc2", 1000, 1000, "relu"),
                     _dense("fc3", 1000, 10, "relu")),
                    C=C, sigma=1.1, zbar_var=1.0 / B)


def cnn(dtype="f32", B=128) -> Workload:
    """CNN on 32x32x3 inputs: three 3x3 pad-1 convolutions given as im2col
    patch matrices (2x2 pooling between them is implied by the map sizes),
    then dense 8192->256->10."""
    layers = (
        LayerSpec("conv1", 32 * 32, 3 * 9, 32, True, "im2col", (3, 32, 32, 3, 1)),
        LayerSpec("conv2", 16 * 16, 32 * 9, 64, True, "im2col", (32, 16, 16, 3, 1)),
        LayerSpec("conv3", 8 * 8, 64 * 9, 128, True, "im2col", (64, 8, 8, 3, 1)),
        _dense("fc1", 8192, 256, "relu"),
        _dense("fc2", 256, 10, "relu"),
    )
    return Workload(f"cnn_32x32x3_b{B}_{dtype}", B, dtype, layers, C=1.0, sigma=1.0,
                    zbar_var=1.0 / B)


def seq(dtype="bf16", B=128, T=256, d=512, d_ff=2048) -> Workload:
    """Sequence-model layers: four d->d attention projections (bias-free),
    d->d_ff and d_ff->d FFN layers, and an LSTM gate layer d->4d applied
    across all T steps (one bias vector)."""
    layers = (
        LayerSpec("attn_q", T, d, d, False, "normal"),
        LayerSpec("attn_k", T, d, d, False, "normal"),
        LayerSpec("attn_v", T, d, d, False, "normal"),
        LayerSpec("attn_o", T, d, d, False, "normal"),
        LayerSpec("ffn_in", T, d, d_ff, True, "normal"),
        LayerSpec("ffn_out", T, d_ff, d, True, "relu"),
        LayerSpec("lstm_gates", T, d, 4 * d, True, "normal"),
    )
    return Workload(f"seq_b{B}_t{T}_d{d}_{dtype}", B, dtype, layers, C=1.0, sigma=0.8,
                    zbar_var=1.0 / (B * T))


def sweep_point(B, T, d_in, d_out, dtype="bf16") -> Workload:
    """One point of the Gram-vs-materialise crossover sweep: one dense layer
    applied at T positions, bias on."""
    layers = (LayerSpec("dense", T, d_in, d_out, True, "normal"),)
    return Workload(f"sweep_b{B}_t{T}_{d_in}x{d_out}_{dtype}", B, dtype, layers, C=1.0,
                    sigma=1.0, zbar_var=1.0 / (B * T))


SWEEP_B = (256, 1024)
SWEEP_T = (16, 128, 512, 2048)
SWEEP_D = ((1024, 1024), (1024, 4096), (4096, 1024))


def by_name(name: str) -> Workload:
    """The named benchmark workloads ("cfg1" .. "cfg4", with dtype suffix
    where two precisions exist)."""
    table = {
        "cfg1": lambda: mlp_small("f32"),
        "cfg2": lambda: mlp_large("f32", 1.0),
        "cfg2_bf16": lambda: mlp_large("bf16", 1.0),
        "cfg3_f32": lambda: cnn("f32"),
        "cfg3_bf16": lambda: cnn("bf16"),
        "cfg4": lambda: seq("bf16"),
    }
    return table[name]()


# --------------------------------------------------------------------------
# bf16 helpers (representation only)
# --------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest bfloat16 (ties to even), returned as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 array of bf16-representable values -> uint16 payload."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


# --------------------------------------------------------------------------
# generators
# --------------------------------------------------------------------------
def im2col(fmap: np.ndarray, k, pad: int, stride: int = 1) -> np.ndarray:
    """(B, C, H, W) -> (B, H'*W', C*kh*kw) patch matrix of a kh x kw convolution (k = int or (kh, kw)) with
    zero padding `pad` and stride `stride`; H' = (H + 2 pad - kh) / stride + 1.  Column order is
    (c, ky, kx) with c slowest, matching a convolution weight flattened from [c_out, c_in, kh, kw]."""
    kh, kw = (k, k) if isinstance(k, int) else k
    B, C, H, W = fmap.shape
    Ho, Wo = (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1
    padded = np.zeros((B, C, H + 2 * pad, W + 2 * pad), dtype=fmap.dtype)
    padded[:, :, pad:pad + H, pad:pad + W] = fmap
    out = np.empty((B, Ho * Wo, C * kh * kw), dtype=fmap.dtype)
    col = 0
    for c in range(C):
        for ky in range(kh):
            for kx in range(kw):
                out[:, :, col] = padded[:, c, ky:ky + (Ho - 1) * stride + 1:stride,
                                        kx:kx + (Wo - 1) * stride + 1:stride].reshape(B, Ho * Wo)
                col += 1
    return out


def conv_inputs(rng_seed: int, B: int, C: int, H: int, W: int, k, pad: int, stride: int, d_out: int,
                dtype: str = "f32", var_z: float = 1.0) -> Tuple[np.ndarray, np.ndarray]:
    """Inputs of a convolution layer as back-propagation has them: the feature map X (B, C, H, W), ReLU of
    N(0,1), and Zbar (B, T, d_out) ~ N(0, var_z), T = H' W'."""
    kh, kw = (k, k) if isinstance(k, int) else k
    rng = np.random.default_rng([rng_seed, B, C, H, W, kh, kw, pad, stride, d_out])
    X = np.maximum(rng.standard_normal((B, C, H, W), dtype=np.float32), 0.0)
    Ho, Wo = (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1
    Z = rng.standard_normal((B, Ho * Wo, d_out), dtype=np.float32) * np.float32(np.sqrt(var_z))
    if dtype == "bf16":
        X, Z = round_to_bf16(X), round_to_bf16(Z)
    return np.ascontiguousarray(X), np.ascontiguousarray(Z)


def _draw_A(rng: np.random.Generator, B: int, spec: LayerSpec) -> np.ndarray:
    if spec.a_dist == "normal":
        return rng.standard_normal((B, spec.T, spec.d_in), dtype=np.float32)
    if spec.a_dist == "relu":
        return np.maximum(rng.standard_normal((B, spec.T, spec.d_in), dtype=np.float32), 0.0)
    if spec.a_dist == "im2col":
        c, H, W, k, p = spec.conv
        fmap = np.maximum(rng.standard_normal((B, c, H, W), dtype=np.float32), 0.0)
        A = im2col(fmap, k, p)
        assert A.shape == (B, spec.T, spec.d_in), (A.shape, spec)
        return A
    raise ValueError(spec.a_dist)


def generate(w: Workload, seed: int = 0, examples: Optional[int] = None
             ) -> List[Tuple[np.ndarray, np.ndarray]]:
    """Draw [(A_l, Zbar_l)] for every layer of `w`.

    Arrays are float32; for w.dtype == "bf16" every value is already rounded
    to bfloat16.  `examples` limits the batch to its first rows-worth of
    draws (a smaller B with the same per-example distribution)."""
    B = w.B if examples is None else examples
    out = []
    for li, spec in enumerate(w.layers):
        rng = np.random.default_rng([seed, li, 0xD9C11F])
        A = _draw_A(rng, B, spec)
        Z = rng.standard_normal((B, spec.T, spec.d_out), dtype=np.float32)
        Z *= np.float32(np.sqrt(w.zbar_var))
        if w.dtype == "bf16":
            A, Z = round_to_bf16(A), round_to_bf16(Z)
        out.append((np.ascontiguousarray(A), np.ascontiguousarray(Z)))
    return out


def spread_factors(B: int, seed: int = 0, lo: float = 1.0 / 8, hi: float = 8.0) -> np.ndarray:
    """Per-example positive multipliers, log-uniform on [lo, hi].  Tests use
    them to spread per-example norms around the clip threshold (the stated
    distributions alone put every norm far above C)."""
    rng = np.random.default_rng([seed, 0x5CA1E])
    return np.exp(rng.uniform(np.log(lo), np.log(hi), size=B))


def random_layer(rng_seed: int, B: int, T: int, d_in: int, d_out: int, dtype: str = "f32",
                 scale_z: float = 1.0) -> Tuple[np.ndarray, np.ndarray]:
    """One (A, Zbar) pair with N(0,1) / N(0, scale_z^2) entries for ad-hoc
    shape tests."""
    rng = np.random.default_rng([rng_seed, B, T, d_in, d_out])
    A = rng.standard_normal((B, T, d_in), dtype=np.float32)
    Z = rng.standard_normal((B, T, d_out), dtype=np.float32) * np.float32(scale_z)
    if dtype == "bf16":
        A, Z = round_to_bf16(A), round_to_bf16(Z)
    return A, Z


def layernorm_pair(rng_seed: int, B: int, T: int, d: int, dtype: str = "f32", var_z: float = 1.0
                   ) -> Tuple[np.ndarray, np.ndarray]:
    """Inputs of an element-wise gain/shift layer: Hbar (B, T, d) with every row normalised to zero mean
    and unit variance (what a LayerNorm hands to its gain), Zbar ~ N(0, var_z)."""
    rng = np.random.default_rng([rng_seed, B, T, d, 0x1A7E2])
    X = rng.standard_normal((B, T, d), dtype=np.float32)
    X -= X.mean(axis=-1, keepdims=True)
    X /= np.sqrt((X * X).mean(axis=-1, keepdims=True) + np.float32(1e-5))
    Z = rng.standard_normal((B, T, d), dtype=np.float32) * np.float32(np.sqrt(var_z))
    if dtype == "bf16":
        X, Z = round_to_bf16(X), round_to_bf16(Z)
    return np.ascontiguousarray(X), np.ascontiguousarray(Z)
