"""Seeded synthetic inputs shaped like DiG activations.

Serves both the CUDA path and the test oracle; holds no arithmetic of the method itself
(the gate transform, the scan orders and the operators live elsewhere).  The recipe:
``numpy.random.default_rng(seed)``, float64 ``standard_normal`` drawn in the fixed order
q, k, v, gate logits, dO, conv weight, conv input; cast to float32; for bf16 workloads every
tensor except the temperatures is then rounded to the nearest bf16 value (ties to even) and
kept in float32 storage, so both consumers see exactly the same numbers.

Token tensors are ``[B, L, H, d]`` with ``L = grid_h * grid_w`` in row-major grid order, the
layout a projection GEMM over a ``(B, T, D)`` token sequence produces (Algorithm 1).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    grid_h: int
    grid_w: int
    d_k: int
    d_v: int
    chunk: int = 64
    dtype: str = "bf16"              # "f32" or "bf16": storage type of q, k, v, out and grads
    backward: bool = True
    directions: tuple = (0,)
    tau: tuple = (16.0,)             # cycled over heads
    conv: bool = False
    seed: int = 0
    note: str = field(default="", compare=False)

    @property
    def L(self) -> int:
        return self.grid_h * self.grid_w

    def tau_per_head(self) -> np.ndarray:
        return np.array([self.tau[h % len(self.tau)] for h in range(self.H)], dtype=np.float32)

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark workloads: latent-patch grids of 256^2 ... 2048^2 images (patch 2 on an
# 8x-downsampled latent gives L = (res/16)^2) and the hidden sizes of the S / B / XL models.
CONFIGS = {
    "C1": Workload("C1", B=1, H=6, grid_h=16, grid_w=16, d_k=64, d_v=64, chunk=64, dtype="f32",
                   backward=False, directions=(0,), note="256^2 image, S-size heads, fp32 forward"),
    "C2": Workload("C2", B=8, H=6, grid_h=32, grid_w=32, d_k=64, d_v=64, chunk=64,
                   directions=(0, 1, 2, 3), conv=True, note="512^2 image, S size, all directions + conv"),
    "C3": Workload("C3", B=4, H=12, grid_h=64, grid_w=64, d_k=64, d_v=64, chunk=64,
                   directions=(0,), tau=(16.0, 4.0), note="1024^2 image, B size, mixed gate temperature"),
    "C4": Workload("C4", B=1, H=6, grid_h=112, grid_w=112, d_k=64, d_v=64, chunk=64,
                   directions=(0,), note="1792^2 image, S size, chunk sweep"),
    "C5": Workload("C5", B=1, H=16, grid_h=128, grid_w=128, d_k=72, d_v=72, chunk=64,
                   directions=(0, 1, 2, 3), conv=True, note="2048^2 image, XL size (hidden 1152)"),
}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float32 values to bf16, returned as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    out = (r & 0xFFFFFFFF).astype(np.uint32).view(np.float32)
    nan = np.isnan(x)
    if nan.any():
        out = np.where(nan, x, out)
    return out.reshape(x.shape)


def make_inputs(wl: Workload, *, gla: bool = True, conv: bool | None = None) -> dict:
    """Returns float32 numpy arrays: q, k, v, g (gate logits), dO, tau [H]; and, for workloads
    with a conv, conv_w [3,3,D], conv_x [B,L,D] with D = H*d_v."""
    rng = np.random.default_rng(wl.seed)
    B, L, H = wl.B, wl.L, wl.H
    conv = wl.conv if conv is None else conv
    out = {}

    def draw(shape, scale=1.0):
        a = (rng.standard_normal(shape) * scale).astype(np.float32)
        return round_to_bf16(a) if wl.dtype == "bf16" else a

    # fixed draw order, also when a tensor is not requested, so that seeds stay comparable
    for name, d in (("q", wl.d_k), ("k", wl.d_k), ("v", wl.d_v), ("g", wl.d_k), ("dO", wl.d_v)):
        t = draw((B, L, H, d))
        if gla:
            out[name] = t
    out["tau"] = wl.tau_per_head()
    if conv:
        D = H * wl.d_v
        out["conv_w"] = draw((3, 3, D), scale=1.0 / 3.0)      # variance 1/9
        out["conv_x"] = draw((B, L, D))
    return out
