"""Seeded synthetic inputs for the adapted-quantized-linear workloads.

This module only draws numbers and shapes them; it contains none of the
method's arithmetic (no quantizer, no pooling, no matmul), so both the GPU
library's callers and the CPU checker can be fed from it.  numpy only.

Each tensor gets its own counter-based stream (Philox keyed by seed and a
stable hash of the tensor's name), so tensors are reproducible independently of
the order in which they are generated.  The fine-tuning datasets and model
weights the paper measures on are replaced by Gaussian tensors with the real
layer shapes; activations, gradients and adapter matrices are rounded to values
representable in bf16 (round-to-nearest-even), the storage type of those
tensors.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np


def _stream(seed: int, name: str) -> np.random.Generator:
    h = hashlib.sha256(name.encode()).digest()
    key = int.from_bytes(h[:8], "little") ^ (int(seed) * 0x9E3779B97F4A7C15 & (2**64 - 1))
    return np.random.Generator(np.random.Philox(key=key))


def normal(seed: int, name: str, shape, std: float = 1.0) -> np.ndarray:
    g = _stream(seed, name)
    out = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        out *= np.float32(std)
    return out


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float32 array whose values are the bf16 round-to-nearest-even of ``a`` (non-finite values keep
    their class)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    out = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))   # cannot wrap for finite values
    out &= np.uint32(0xFFFF0000)
    special = (u & np.uint32(0x7F800000)) == np.uint32(0x7F800000)
    if special.any():
        nan = special & ((u & np.uint32(0x007FFFFF)) != 0)
        out[special] = u[special] & np.uint32(0xFFFF0000)
        out[nan] |= np.uint32(0x00400000)
    return out.view(np.float32).reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of an array already representable in bf16."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def outlier_channels(seed: int, name: str, d_in: int, fraction: float) -> np.ndarray:
    """Indices of round(fraction * d_in) input channels, by seeded permutation."""
    n = int(round(fraction * d_in))
    g = _stream(seed, name + "/outliers")
    return np.sort(g.permutation(d_in)[:n])


@dataclass(frozen=True)
class Geometry:
    """Adapter geometry: pooling factor on the input, repeat factor on the output."""
    name: str
    lambda_in: int
    lambda_out: int


GEOM_A = Geometry("GA", 64, 8)   # one pooling window per 64-wide quantization group
GEOM_B = Geometry("GB", 4, 4)    # the paper's single balancing factor on both sides


@dataclass(frozen=True)
class LinearSpec:
    name: str
    d_out: int
    d_in: int


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration: a set of independent adapted linears."""
    name: str
    tokens: int
    linears: Tuple[LinearSpec, ...]
    rank: int
    w_std: float = 0.02
    ab_std: float = 0.01
    scaling: float = 1.0
    qfmt: int = 0                 # 0 = level table + absmax, 1 = min-max (zero-point) format
    block_in: int = 64
    outlier_fraction: float = 0.0
    outlier_gain: float = 20.0
    lowbit_tokens: Tuple[int, ...] = ()


WORKLOADS: Dict[str, Workload] = {
    "C1": Workload("C1", 256, (LinearSpec("lin", 1024, 1024),), rank=64),
    "C2": Workload("C2", 2048, (LinearSpec("attn_proj", 4096, 4096),), rank=256),
    "C3": Workload("C3", 4096, (LinearSpec("gate", 11008, 4096), LinearSpec("up", 11008, 4096),
                                LinearSpec("down", 4096, 11008)), rank=256,
                   outlier_fraction=0.01),
    "C4": Workload("C4", 8192, (LinearSpec("q", 5120, 5120), LinearSpec("k", 5120, 5120),
                                LinearSpec("v", 5120, 5120), LinearSpec("o", 5120, 5120),
                                LinearSpec("gate", 13824, 5120), LinearSpec("up", 13824, 5120),
                                LinearSpec("down", 5120, 13824)), rank=256),
    "C5": Workload("C5", 2048, (LinearSpec("q", 6656, 6656), LinearSpec("up", 17920, 6656),
                                LinearSpec("down", 6656, 17920)), rank=256, ab_std=0.02, qfmt=1,
                   lowbit_tokens=(1, 16, 2048)),
}


@dataclass
class LinearInputs:
    spec: LinearSpec
    W: np.ndarray                     # float32 [d_out][d_in]
    X: np.ndarray                     # float32 (bf16-representable) [T][d_in]
    dY: np.ndarray                    # float32 (bf16-representable) [T][d_out]
    A: np.ndarray                     # float32 (bf16-representable) [P][r]
    B: np.ndarray                     # float32 (bf16-representable) [r][Q]
    geometry: Geometry
    rank: int
    scaling: float
    outliers: Optional[np.ndarray] = None


def make_activations(seed: int, tag: str, tokens: int, width: int, outlier_fraction: float = 0.0,
                     outlier_gain: float = 20.0):
    X = normal(seed, tag, (tokens, width))
    idx = None
    if outlier_fraction > 0:
        idx = outlier_channels(seed, tag, width, outlier_fraction)
        X[:, idx] *= np.float32(outlier_gain)
    return round_to_bf16(X), idx


def make_linear_inputs(wl: Workload, spec: LinearSpec, geom: Geometry, seed: int = 0,
                       tokens: Optional[int] = None, want_w: bool = True) -> LinearInputs:
    T = wl.tokens if tokens is None else tokens
    tag = f"{wl.name}/{spec.name}"
    W = normal(seed, tag + "/W", (spec.d_out, spec.d_in), wl.w_std) if want_w else None
    X, idx = make_activations(seed, tag + "/X", T, spec.d_in, wl.outlier_fraction, wl.outlier_gain)
    dY = round_to_bf16(normal(seed, tag + "/dY", (T, spec.d_out)))
    P, Q = spec.d_in // geom.lambda_in, spec.d_out // geom.lambda_out
    A = round_to_bf16(normal(seed, f"{tag}/{geom.name}/A", (P, wl.rank), wl.ab_std))
    B = round_to_bf16(normal(seed, f"{tag}/{geom.name}/B", (wl.rank, Q), wl.ab_std))
    return LinearInputs(spec, W, X, dY, A, B, geom, wl.rank, wl.scaling, idx)


def small_workload(name: str, tokens: int, d_out: int, d_in: int, rank: int, **kw) -> Workload:
    """A scaled-down configuration with the same recipe, for quick checks."""
    return Workload(name, tokens, (LinearSpec("lin", d_out, d_in),), rank=rank, **kw)
