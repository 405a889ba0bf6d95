"""fp64 CPU oracle for the adapted quantized linear layer -- TEST INFRASTRUCTURE.

Thin ctypes access to ``qblora_oracle.c`` (numpy arrays in, numpy arrays out).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the GPU library neither imports it nor shares code with it.

Array conventions: weights are ``[d_out][d_in]`` row-major; ``codes`` is
``uint8 [d_out][d_in/2]`` (low nibble = even column); ``alpha``/``beta`` are
``float32 [d_out/block_out][d_in/block_in]``; activations and adapter matrices
are ``float32`` arrays whose values are exactly representable in bf16.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qblora_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

FMT_CODEBOOK_ABSMAX = 0
FMT_AFFINE_MINMAX = 1

# parameter-free operator pair around the adapter (Sec. 3.2; alternatives from the Sec. 4 ablation)
OP_AVGPOOL_REPEAT = 0       # AvgPool & repeat_interleave (the method's own)
OP_TRUNCATE_ZEROPAD = 1     # truncation & supplement_0
OP_SAMPLE_ZEROFILL = 2      # interval_sampling & interpolation (zeros between the samples)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _check(rc, what):
    if rc != 0:
        raise ValueError(f"oracle {what}: invalid geometry (rc={rc})")


def num_threads() -> int:
    return int(_L().orc_num_threads())


def default_code_table() -> np.ndarray:
    out = np.zeros(16, dtype=np.float32)
    _check(_L().orc_default_code_table(_p(out, ctypes.c_float)), "default_code_table")
    return out


@dataclass
class QWeight:
    d_out: int
    d_in: int
    block_in: int
    block_out: int
    qfmt: int
    code: Optional[np.ndarray]      # float32[16] for the code-table format
    codes: np.ndarray               # uint8 [d_out][d_in/2]
    alpha: np.ndarray               # float32 [d_out/block_out][d_in/block_in]
    beta: Optional[np.ndarray]      # same shape; None for the code-table format


@dataclass
class Adapter:
    lambda_in: int
    lambda_out: int
    rank: int
    scaling: float
    A: np.ndarray                   # [d_in/lambda_in][rank]  (or H [P][Q] when B is None)
    B: Optional[np.ndarray]         # [rank][d_out/lambda_out]
    scale_op: int = 0               # OP_AVGPOOL_REPEAT / OP_TRUNCATE_ZEROPAD / OP_SAMPLE_ZEROFILL


def quantize_blockwise(W, block_in=64, block_out=1, qfmt=FMT_CODEBOOK_ABSMAX, code=None, nbits=4) -> QWeight:
    """Eq. 1 per block.  nbits < 4 (min-max format only) restricts the grid to 2^nbits levels; the codes are
    still stored one per nibble, so everything downstream treats the result as a 4-bit weight."""
    W = _f32(W)
    d_out, d_in = W.shape
    if qfmt == FMT_CODEBOOK_ABSMAX and code is None:
        code = default_code_table()
    code = _f32(code)
    if d_in % block_in or d_out % block_out or d_in % 2:
        raise ValueError("oracle quantize: invalid geometry")
    codes = np.zeros((d_out, d_in // 2), dtype=np.uint8)
    alpha = np.zeros((d_out // block_out, d_in // block_in), dtype=np.float32)
    beta = np.zeros_like(alpha) if qfmt == FMT_AFFINE_MINMAX else None
    rc = _L().orc_quantize_blockwise(_p(W, ctypes.c_float), d_out, d_in, block_in, block_out, qfmt, int(nbits),
                                     _p(code, ctypes.c_float), _p(codes, ctypes.c_uint8),
                                     _p(alpha, ctypes.c_float), _p(beta, ctypes.c_float))
    _check(rc, "quantize_blockwise")
    return QWeight(d_out, d_in, block_in, block_out, qfmt, code, codes, alpha, beta)


def packed_row_bytes(d_in: int, nbits: int) -> int:
    return d_in * nbits // 8


def pack_codes(codes: np.ndarray, d_in: int, nbits: int) -> np.ndarray:
    """Nibble-stored codes [d_out][d_in/2] -> dense N-bit storage [d_out][d_in*N/8], N = 2 or 3."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    d_out = codes.shape[0]
    out = np.zeros((d_out, packed_row_bytes(d_in, nbits)), dtype=np.uint8)
    _check(_L().orc_pack_codes(_p(codes, ctypes.c_uint8), d_out, d_in, int(nbits), _p(out, ctypes.c_uint8)), "pack_codes")
    return out


def unpack_codes(packed: np.ndarray, d_in: int, nbits: int) -> np.ndarray:
    """Dense N-bit storage -> nibble-stored codes [d_out][d_in/2]."""
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    d_out = packed.shape[0]
    out = np.zeros((d_out, d_in // 2), dtype=np.uint8)
    _check(_L().orc_unpack_codes(_p(packed, ctypes.c_uint8), d_out, d_in, int(nbits), _p(out, ctypes.c_uint8)), "unpack_codes")
    return out


def dequantize(qw: QWeight) -> np.ndarray:
    Wt = np.zeros((qw.d_out, qw.d_in), dtype=np.float64)
    rc = _L().orc_dequantize(_p(qw.codes, ctypes.c_uint8), _p(qw.alpha, ctypes.c_float),
                             _p(qw.beta, ctypes.c_float), qw.d_out, qw.d_in, qw.block_in,
                             qw.block_out, qw.qfmt, _p(qw.code, ctypes.c_float),
                             _p(Wt, ctypes.c_double))
    _check(rc, "dequantize")
    return Wt


def _ad_args(ad: Optional[Adapter]):
    if ad is None:
        return 0, 0, 1, 1, 0, ctypes.c_double(0.0), None, None, None, None
    A = _f32(ad.A)
    B = _f32(ad.B)
    return (1, int(ad.scale_op), ad.lambda_in, ad.lambda_out, ad.rank, ctypes.c_double(float(ad.scaling)),
            _p(A, ctypes.c_float), _p(B, ctypes.c_float), A, B)


def linear_fwd(Wt: np.ndarray, ad: Optional[Adapter], X) -> np.ndarray:
    """Y = X W~^T + s * repeat(pool(X) A B); ``Wt`` is the dequantized weight (float64)."""
    X = _f32(X)
    Wt = np.ascontiguousarray(Wt, dtype=np.float64)
    T, d_in = X.shape
    d_out = Wt.shape[0]
    Y = np.zeros((T, d_out), dtype=np.float64)
    has, op, l1, l2, r, s, pA, pB, _A, _B = _ad_args(ad)
    rc = _L().orc_linear_fwd(_p(Wt, ctypes.c_double), d_out, d_in, _p(X, ctypes.c_float),
                             ctypes.c_int64(T), has, op, l1, l2, r, s, pA, pB, _p(Y, ctypes.c_double))
    _check(rc, "linear_fwd")
    return Y


def linear_bwd(Wt: Optional[np.ndarray], ad: Optional[Adapter], X, dY, d_out=None,
               want_dx=True, want_da=True, want_db=True):
    """Returns (dX, dA, dB) as float64 arrays (None where skipped)."""
    X = _f32(X)
    dY = _f32(dY)
    T, d_in = X.shape
    d_out = dY.shape[1]
    if Wt is not None:
        Wt = np.ascontiguousarray(Wt, dtype=np.float64)
    has, op, l1, l2, r, s, pA, pB, A, B = _ad_args(ad)
    dX = np.zeros((T, d_in), dtype=np.float64) if want_dx else None
    dA = dB = None
    if ad is not None:
        if want_da:
            dA = np.zeros(A.shape, dtype=np.float64)
        if want_db and B is not None:
            dB = np.zeros(B.shape, dtype=np.float64)
    rc = _L().orc_linear_bwd(_p(Wt, ctypes.c_double), d_out, d_in, _p(X, ctypes.c_float),
                             _p(dY, ctypes.c_float), ctypes.c_int64(T), has, op, l1, l2, r, s, pA, pB,
                             _p(dX, ctypes.c_double), _p(dA, ctypes.c_double), _p(dB, ctypes.c_double))
    _check(rc, "linear_bwd")
    return dX, dA, dB


def dense_delta_w(d_out: int, d_in: int, ad: Adapter) -> np.ndarray:
    A = _f32(ad.A)
    B = _f32(ad.B)
    dW = np.zeros((d_out, d_in), dtype=np.float64)
    rc = _L().orc_dense_delta_w(int(ad.scale_op), d_out, d_in, ad.lambda_in, ad.lambda_out, ad.rank,
                                _p(A, ctypes.c_float), _p(B, ctypes.c_float), _p(dW, ctypes.c_double))
    _check(rc, "dense_delta_w")
    return dW


def merge(qw: QWeight, ad: Adapter) -> QWeight:
    """QA-BLoRA merge: returns a new QWeight with beta' (codes and alpha are the same arrays)."""
    if qw.qfmt != FMT_AFFINE_MINMAX:
        raise ValueError("oracle merge: needs the min-max format")
    if ad.scale_op != OP_AVGPOOL_REPEAT:
        raise ValueError("oracle merge: the update is constant per block only for AvgPool & repeat_interleave")
    A = _f32(ad.A)
    B = _f32(ad.B)
    beta_out = np.zeros_like(qw.beta)
    rc = _L().orc_merge(_p(qw.beta, ctypes.c_float), qw.d_out, qw.d_in, qw.block_in, qw.block_out,
                        ad.lambda_in, ad.lambda_out, ad.rank, ctypes.c_double(float(ad.scaling)),
                        _p(A, ctypes.c_float), _p(B, ctypes.c_float), _p(beta_out, ctypes.c_float))
    _check(rc, "merge")
    return QWeight(qw.d_out, qw.d_in, qw.block_in, qw.block_out, qw.qfmt, qw.code, qw.codes,
                   qw.alpha, beta_out)


def lowbit_gemm(qw: QWeight, X) -> np.ndarray:
    X = _f32(X)
    T = X.shape[0]
    Y = np.zeros((T, qw.d_out), dtype=np.float64)
    rc = _L().orc_lowbit_gemm(_p(qw.codes, ctypes.c_uint8), _p(qw.alpha, ctypes.c_float),
                              _p(qw.beta, ctypes.c_float), qw.d_out, qw.d_in, qw.block_in,
                              qw.block_out, _p(X, ctypes.c_float), ctypes.c_int64(T),
                              _p(Y, ctypes.c_double))
    _check(rc, "lowbit_gemm")
    return Y
