"""Seeded synthetic activation maps shaped like the paper's CNN workloads.

This module holds NO arithmetic of the compression method; it only makes inputs, for the
CUDA library, for its tests and for the CPU checker alike.  The paper measures on
activation maps of ResNet / WideResNet / DenseNet models trained on CIFAR and ImageNet
(Sec. 5); those models and datasets are not available here, so these tensors stand in for
them: same shapes, post-ReLU sparsity (about half the values exactly zero), a spatially
smooth component a few pixels wide (so that the block mean carries real signal) and pixel
noise on top.

Recipe (sample n of a tensor draws from numpy.random.Generator(PCG64([data_seed, n])), fp32):
  eps  iid N(0,1) per element
  g    smooth field: iid N(0,1) on a (ceil(H/4)+1) x (ceil(W/4)+1) lattice per (n,c) plane,
       bilinearly interpolated to H x W (4-pixel correlation length)
  m    iid Bernoulli(0.5) per element
  post-ReLU:  x = m * |g + 0.1*eps|          post-BN:  x = eps + g
data_seed = 1000*config + tensor_index.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

CORRELATION_PX = 4


@dataclass(frozen=True)
class TensorSpec:
    config: int
    index: int
    n: int
    c: int
    h: int
    w: int
    kind: str            # "relu" or "bn"
    x_dtype: str         # "f32" or "bf16"
    lfc_dtype: str
    block: int
    qbits: int

    @property
    def shape(self):
        return (self.n, self.c, self.h, self.w)

    @property
    def data_seed(self):
        return 1000 * self.config + self.index

    @property
    def numel(self):
        return self.n * self.c * self.h * self.w

    def label(self):
        return (f"cfg{self.config}[{self.index}] {self.n}x{self.c}x{self.h}x{self.w} {self.x_dtype} "
                f"{self.kind} B{self.block} Q{self.qbits} lfc-{self.lfc_dtype}")


def _interp_matrix(out_len: int, lattice_len: int) -> np.ndarray:
    """Linear interpolation weights from a lattice with spacing CORRELATION_PX to out_len pixels."""
    pos = np.arange(out_len, dtype=np.float64) / CORRELATION_PX
    i0 = np.minimum(np.floor(pos).astype(np.int64), lattice_len - 2)
    frac = pos - i0
    m = np.zeros((out_len, lattice_len), dtype=np.float32)
    m[np.arange(out_len), i0] = (1.0 - frac).astype(np.float32)
    m[np.arange(out_len), i0 + 1] = frac.astype(np.float32)
    return m


def smooth_field(rng: np.random.Generator, c: int, h: int, w: int) -> np.ndarray:
    hl = -(-h // CORRELATION_PX) + 1
    wl = -(-w // CORRELATION_PX) + 1
    lattice = rng.standard_normal((c, hl, wl), dtype=np.float32)
    mh = _interp_matrix(h, hl)
    mw = _interp_matrix(w, wl)
    return np.matmul(np.matmul(mh[None], lattice), mw.T[None])


def sample_map(c: int, h: int, w: int, kind: str, data_seed: int, n: int) -> np.ndarray:
    """Sample `n` (shape C x H x W, fp32) of the tensor with this data_seed; samples are seeded one by one."""
    rng = np.random.Generator(np.random.PCG64([int(data_seed), int(n)]))
    g = smooth_field(rng, c, h, w)
    eps = rng.standard_normal((c, h, w), dtype=np.float32)
    if kind == "bn":
        return (eps + g).astype(np.float32)
    if kind == "relu":
        m = rng.integers(0, 2, size=(c, h, w), dtype=np.uint8).astype(np.float32)
        return (m * np.abs(g + np.float32(0.1) * eps)).astype(np.float32)
    raise ValueError(f"unknown kind {kind!r}")


def activation_map(n: int, c: int, h: int, w: int, kind: str, data_seed: int) -> np.ndarray:
    """One fp32 N x C x H x W activation map of the given kind ("relu" or "bn")."""
    out = np.empty((n, c, h, w), dtype=np.float32)
    for i in range(n):
        out[i] = sample_map(c, h, w, kind, data_seed, i)
    return out


def to_bf16_bits(x32: np.ndarray) -> np.ndarray:
    """Input-side cast of a generated fp32 map to bfloat16 bit patterns (nearest even)."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32).astype(np.uint64)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def make_input(spec: TensorSpec) -> np.ndarray:
    """The tensor of `spec`: float32 array, or uint16 bfloat16 bit patterns for bf16 specs."""
    x = activation_map(spec.n, spec.c, spec.h, spec.w, spec.kind, spec.data_seed)
    return to_bf16_bits(x) if spec.x_dtype == "bf16" else x


def make_sample(spec: TensorSpec, n: int) -> np.ndarray:
    """Sample `n` of the tensor of `spec` with a leading axis of 1 (same bits as make_input(spec)[n:n+1])."""
    x = sample_map(spec.c, spec.h, spec.w, spec.kind, spec.data_seed, n)[None]
    return to_bf16_bits(x) if spec.x_dtype == "bf16" else x


# ----------------------------------------------------------------------------------------
# the five workload configurations
# ----------------------------------------------------------------------------------------
def config0():
    return [TensorSpec(0, 0, 8, 64, 32, 32, "relu", "f32", "f32", 8, 2)]


def config1():
    out = []
    idx = 0
    for (c, s) in [(64, 32), (128, 16), (256, 8), (512, 4)]:
        for kind in ("bn", "relu"):
            out.append(TensorSpec(1, idx, 128, c, s, s, kind, "f32", "f32", 8, 2))
            idx += 1
    return out


def config2():
    shapes = [(64, 112), (256, 56), (512, 28), (1024, 14), (2048, 7)]
    return [TensorSpec(2, i, 64, c, s, s, "relu", "f32", "f32", 8, 2) for i, (c, s) in enumerate(shapes)]


def config3():
    out = []
    idx = 0
    for (c, s) in [(160, 32), (320, 16), (640, 8)]:
        for block in (4, 8):
            for q in (2, 4):
                out.append(TensorSpec(3, idx, 128, c, s, s, "relu", "bf16", "bf16", block, q))
                idx += 1
    return out


DENSENET_CHANNELS = {56: (64, 256), 28: (128, 512), 14: (256, 1024), 7: (512, 1024)}


def config4():
    """Concatenated feature maps of a growth-32 DenseNet-121 at each resolution (62 tensors)."""
    out = []
    idx = 0
    for s, (c_lo, c_hi) in DENSENET_CHANNELS.items():
        for c in range(c_lo, c_hi + 1, 32):
            out.append(TensorSpec(4, idx, 64, c, s, s, "relu", "f32", "f32", 8, 2))
            idx += 1
    return out


CONFIGS = {0: config0, 1: config1, 2: config2, 3: config3, 4: config4}


def config_specs(config: int):
    return CONFIGS[config]()
