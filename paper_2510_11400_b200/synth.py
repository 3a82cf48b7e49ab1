"""Seeded synthetic activation tensors.

This module only draws random numbers and shapes them into tensors; it holds none of the
codec's arithmetic.  Both the CPU oracle's tests and the CUDA path's tests/bench use it so
that they see identical bytes.

Recipe: values are drawn in chunks of 2**24 elements, chunk ``j`` of a tensor with seed ``s``
from ``numpy.random.default_rng([s, j])``, always as float32.  bf16 tensors are the float32
draws rounded to bfloat16 with round-half-to-even and returned as ``uint16`` bit patterns.

The distributions stand in for the saved activations of the CNNs the paper trains
(Section 5, Fig. 18a tensor shapes): post-ReLU maps (about half exact zeros), pre-activation
maps (Gaussian), heavy-tailed maps with channel-clustered outliers (Section 4.4.1), and a
sparse-spiky recipe that drives planes through the block-wise path.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import numpy as np

CHUNK = 1 << 24

F32 = 0
BF16 = 1


def _chunks(total: int):
    j = 0
    off = 0
    while off < total:
        n = min(CHUNK, total - off)
        yield j, off, n
        off += n
        j += 1


def normal(total: int, seed: int) -> np.ndarray:
    """z ~ N(0,1), float32, flat."""
    out = np.empty(total, dtype=np.float32)
    for j, off, n in _chunks(total):
        out[off:off + n] = np.random.default_rng([seed, j]).standard_normal(n, dtype=np.float32)
    return out


def relu_normal(total: int, seed: int) -> np.ndarray:
    """max(z, 0), z ~ N(0,1): about 50 % exact zeros."""
    out = normal(total, seed)
    np.maximum(out, 0.0, out=out)
    return out


def laplace(total: int, seed: int) -> np.ndarray:
    """Laplace(0,1), float32, flat."""
    out = np.empty(total, dtype=np.float32)
    for j, off, n in _chunks(total):
        out[off:off + n] = np.random.default_rng([seed, j]).laplace(0.0, 1.0, n).astype(np.float32)
    return out


def laplace_channel_outliers(shape: Tuple[int, int, int, int], seed: int,
                             every: int = 8, prob: float = 0.08, mag: float = 50.0) -> np.ndarray:
    """Laplace(0,1); in channels with c % every == 0 each element becomes +-mag with probability
    prob (fair sign).  Outliers are clustered channel-wise."""
    n, c, h, w = shape
    total = n * c * h * w
    out = laplace(total, seed)
    for j, off, cnt in _chunks(total):
        rng = np.random.default_rng([seed, 1000 + j])
        u = rng.random(cnt, dtype=np.float32)
        sgn = rng.random(cnt, dtype=np.float32) < 0.5
        idx = np.arange(off, off + cnt, dtype=np.int64)
        ch = (idx // (h * w)) % c
        hit = (ch % every == 0) & (u < prob)
        vals = np.where(sgn, np.float32(mag), np.float32(-mag))
        seg = out[off:off + cnt]
        seg[hit] = vals[hit]
    return out


def laplace_iid_outliers(total: int, seed: int, prob: float = 0.01, mag: float = 50.0) -> np.ndarray:
    """Laplace(0,1) with prob of all elements replaced by +-mag, i.i.d. everywhere."""
    out = laplace(total, seed)
    for j, off, cnt in _chunks(total):
        rng = np.random.default_rng([seed, 2000 + j])
        u = rng.random(cnt, dtype=np.float32)
        sgn = rng.random(cnt, dtype=np.float32) < 0.5
        hit = u < prob
        vals = np.where(sgn, np.float32(mag), np.float32(-mag))
        seg = out[off:off + cnt]
        seg[hit] = vals[hit]
    return out


def sparse_spiky(shape: Tuple[int, int, int, int], seed: int, every: int = 16,
                 base: str = "relu") -> np.ndarray:
    """Base tensor (relu or normal) whose planes with c % every == 0 are replaced by a
    sparse-spiky pattern: columns j < max(1, W//4) hold max(z,0); elsewhere the value is
    6+|z'| with probability 0.06, else 0.  Those planes carry about 4.5 % three-sigma outliers
    and a mix of dense and sparse 8x8 blocks."""
    n, c, h, w = shape
    total = n * c * h * w
    out = relu_normal(total, seed) if base == "relu" else normal(total, seed)
    out = out.reshape(n, c, h, w)
    wcut = max(1, w // 4)
    for ci in range(0, c, every):
        rng = np.random.default_rng([seed, 3000 + ci])
        z = rng.standard_normal((n, h, w), dtype=np.float32)
        z2 = rng.standard_normal((n, h, w), dtype=np.float32)
        u = rng.random((n, h, w), dtype=np.float32)
        plane = np.where(u < 0.06, np.float32(6.0) + np.abs(z2), np.float32(0.0)).astype(np.float32)
        plane[:, :, :wcut] = np.maximum(z[:, :, :wcut], 0.0)
        out[:, ci] = plane
    return out.reshape(-1)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-half-to-even; finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32 (exact widening)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class TensorSpec:
    """One synthetic tensor: contiguous NCHW."""
    name: str
    shape: Tuple[int, int, int, int]
    dtype: int          # F32 or BF16
    kind: str           # "relu", "normal", "laplace_ch", "laplace_iid", "spiky_relu", "spiky_normal"
    seed: int
    compress: bool = True

    @property
    def elems(self) -> int:
        n, c, h, w = self.shape
        return n * c * h * w

    @property
    def esize(self) -> int:
        return 4 if self.dtype == F32 else 2

    @property
    def dense_bytes(self) -> int:
        return self.elems * self.esize


def make(spec: TensorSpec) -> np.ndarray:
    """Materialise a spec: float32 array for F32, uint16 bit patterns for BF16 (flat)."""
    k = spec.kind
    if k == "relu":
        x = relu_normal(spec.elems, spec.seed)
    elif k == "normal":
        x = normal(spec.elems, spec.seed)
    elif k == "laplace_ch":
        x = laplace_channel_outliers(spec.shape, spec.seed)
    elif k == "laplace_iid":
        x = laplace_iid_outliers(spec.elems, spec.seed)
    elif k == "spiky_relu":
        x = sparse_spiky(spec.shape, spec.seed, base="relu")
    elif k == "spiky_normal":
        x = sparse_spiky(spec.shape, spec.seed, base="normal")
    else:
        raise ValueError(f"unknown kind {k}")
    return x if spec.dtype == F32 else to_bf16_bits(x)


# ---------------------------------------------------------------------------------------------
# The five workloads (shapes follow the CNN activations of the paper's Fig. 18a).
# ---------------------------------------------------------------------------------------------

def config1() -> List[TensorSpec]:
    return [TensorSpec("c1", (32, 16, 32, 32), F32, "relu", 0)]


def config2(batch: int = 64) -> List[TensorSpec]:
    shapes = [(batch, 64, 112, 112)] + [(batch, 64, 56, 56)] * 4 + [(batch, 128, 28, 28)] * 4 \
        + [(batch, 256, 14, 14)] * 4 + [(batch, 512, 7, 7)] * 4
    return [TensorSpec(f"c2_{i}", s, F32, "relu" if i % 2 == 0 else "normal", 100 + i)
            for i, s in enumerate(shapes)]


def config3(batch: int = 128, stress: bool = False) -> List[TensorSpec]:
    shapes = [(batch, 96, 112, 112), (batch, 144, 56, 56), (batch, 192, 28, 28),
              (batch, 384, 14, 14), (batch, 960, 7, 7)]
    kind = "laplace_iid" if stress else "laplace_ch"
    return [TensorSpec(f"c3{'b' if stress else 'a'}_{i}", s, BF16, kind, 300 + i)
            for i, s in enumerate(shapes)]


def config4(mib: int, dtype: int, k: int = 0) -> List[TensorSpec]:
    esize = 4 if dtype == F32 else 2
    planes = mib * (1 << 20) // (1024 * esize)
    n = max(1, planes // 64)
    c = planes // n
    return [TensorSpec(f"c4_{mib}MiB_{'f32' if dtype == F32 else 'bf16'}", (n, c, 32, 32), dtype,
                       "relu", 400 + k)]


def config5(batch: int = 128) -> List[TensorSpec]:
    shapes = [(batch, 64, 32, 32)] * 5 + [(batch, 128, 16, 16)] * 5 + [(batch, 256, 8, 8)] * 5 \
        + [(batch, 512, 4, 4)] * 5
    return [TensorSpec(f"c5_{i}", s, F32, "relu", 500 + i, compress=(i % 2 == 0))
            for i, s in enumerate(shapes)]


def supplement(specs: List[TensorSpec]) -> List[TensorSpec]:
    """Same shapes, with every 16th channel replaced by the sparse-spiky recipe."""
    out = []
    for s in specs:
        kind = "spiky_relu" if s.kind == "relu" else "spiky_normal"
        out.append(TensorSpec(s.name + "_S", s.shape, s.dtype, kind, s.seed, s.compress))
    return out
