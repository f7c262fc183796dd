"""Helpers shared by the GPU parity tests (marshalling and error measures only)."""
import numpy as np
import torch

import workloads

TOL = {
    # fp32 inputs: per-example norms and gradient (relative Frobenius) within 1e-5
    "f32": dict(norm=1e-5, grad=1e-5),
    # bf16 inputs, fp32 accumulation: 5e-3 per norm, 1e-2 relative Frobenius
    "bf16": dict(norm=5e-3, grad=1e-2),
}
SAT_BAND = 1e-4      # clip decisions may differ only within this relative distance of C


def to_device(x: np.ndarray, dtype: str) -> torch.Tensor:
    """float32 numpy array (already rounded for bf16) -> CUDA tensor of the path's input dtype."""
    if dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    bits = workloads.to_bf16_bits(x).view(np.int16)
    return torch.from_numpy(bits).cuda().view(torch.bfloat16)


def rel_fro(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref.ravel())
    num = np.linalg.norm((got - ref).ravel())
    return float(num / den) if den > 0 else float(num)


def max_rel(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    den = np.where(ref != 0, np.abs(ref), 1.0)
    return float(np.max(np.abs(got - ref) / den))


def check_saturation(clip_gpu, norms_ref, clip_ref, C):
    """Clip decisions identical except within SAT_BAND of the threshold."""
    clip_gpu = np.asarray(clip_gpu, dtype=np.float64)
    sat_gpu, sat_ref = clip_gpu < 1.0, clip_ref < 1.0
    differ = sat_gpu != sat_ref
    near = np.abs(norms_ref / C - 1.0) <= SAT_BAND
    assert not np.any(differ & ~near), np.nonzero(differ & ~near)
    assert np.all(clip_gpu[~sat_gpu] == 1.0)


class Guarded:
    """An fp32 output tensor carved out of a larger allocation with 256-byte guard bands before and after it,
    filled with a bit pattern no kernel writes: stands in for a memory checker on the outputs.  `t` is the
    tensor to hand to the library; `check()` fails if a band was touched."""
    PATTERN = 0x7FA5A5A5          # a NaN payload

    def __init__(self, *shape, fill=9.0):
        n = int(np.prod(shape))
        band = 64                                       # 64 floats = 256 bytes
        pad = (-n) % 64                                 # the output keeps the 256-byte alignment of the allocation
        self.raw = torch.full((band + n + pad + band,), 0, dtype=torch.int32, device="cuda")
        self.raw.fill_(self.PATTERN)
        self.t = self.raw[band:band + n].view(torch.float32).view(*shape)
        self.t.fill_(fill)
        self._n, self._band = n, band

    def check(self):
        lo = self.raw[:self._band]; hi = self.raw[self._band + self._n:]
        assert bool((lo == self.PATTERN).all()) and bool((hi == self.PATTERN).all()), "guard band overwritten"
