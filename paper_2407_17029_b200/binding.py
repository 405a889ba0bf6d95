"""ctypes binding of the C-ABI library declared in ``include/qblora.h``.

Argument marshalling only: torch owns device memory and streams, every step of
the computation runs inside ``libqblora.so``.  Importing this module fails
loudly if the library has not been built (``python -m paper_2407_17029_b200.build``
or ``__graft_entry__.build()``); there is no fallback path.

Names follow the header: ``quantize_blockwise``, ``linear_fwd``, ``linear_bwd``,
``merge``, ``lowbit_gemm``.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqblora.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_TOO_LARGE = range(7)
FMT_CODEBOOK_ABSMAX, FMT_AFFINE_MINMAX = 0, 1
F32, BF16 = 0, 1
OP_QUANTIZE, OP_LINEAR_FWD, OP_LINEAR_BWD, OP_MERGE, OP_LOWBIT_GEMM, OP_MERGE_DENSE = range(6)
# qblora_scale_op: the parameter-free operator pair around the adapter (Sec. 3.2; Sec. 4 scale-operator ablation)
SCALE_AVGPOOL_REPEAT, SCALE_TRUNCATE_ZEROPAD, SCALE_SAMPLE_ZEROFILL = range(3)

EXPORTS = ["qblora_default_code_table", "qblora_workspace_bytes", "qblora_status_string",
           "qblora_device_status", "qblora_quantize_blockwise", "qblora_linear_fwd",
           "qblora_linear_bwd", "qablora_merge", "qablora_lowbit_gemm", "qblora_kernel_launches",
           "qblora_set_timing_events", "qablora_merge_noalloc", "qblora_merge_dense",
           "qblora_quantize_minmax_nbit", "qblora_debug_set_wait_limit", "qblora_debug_drop_load", "qblora_debug_hold_producer", "qblora_dense_gemm", "qblora_pack_codes", "qblora_unpack_codes"]


class _CQWeight(ctypes.Structure):
    _fields_ = [("d_in", ctypes.c_int32), ("d_out", ctypes.c_int32),
                ("block_in", ctypes.c_int32), ("block_out", ctypes.c_int32),
                ("qfmt", ctypes.c_int32), ("code", ctypes.c_float * 16),
                ("codes", ctypes.c_void_p), ("alpha", ctypes.c_void_p), ("beta", ctypes.c_void_p),
                ("code_bits", ctypes.c_int32)]


class _CAdapter(ctypes.Structure):
    _fields_ = [("lambda_in", ctypes.c_int32), ("lambda_out", ctypes.c_int32),
                ("rank", ctypes.c_int32), ("scaling", ctypes.c_float),
                ("A", ctypes.c_void_p), ("B", ctypes.c_void_p), ("scale_op", ctypes.c_int32)]


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build the CUDA library first "
                      "(python -m paper_2407_17029_b200.build); there is no CPU fallback")
_lib = ctypes.CDLL(LIB_PATH)
_lib.qblora_workspace_bytes.restype = ctypes.c_size_t
_lib.qblora_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64]
_lib.qblora_status_string.restype = ctypes.c_char_p
_lib.qblora_status_string.argtypes = [ctypes.c_int]
_lib.qblora_default_code_table.argtypes = [ctypes.c_void_p]
_lib.qblora_device_status.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
_lib.qblora_quantize_blockwise.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int32, ctypes.c_int32,
                                           ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
_lib.qblora_quantize_minmax_nbit.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int32, ctypes.c_int32,
                                             ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                             ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
_lib.qblora_linear_fwd.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                   ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t,
                                   ctypes.c_void_p]
_lib.qblora_linear_bwd.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                   ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                   ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
_lib.qablora_merge.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                               ctypes.c_size_t, ctypes.c_void_p]
_lib.qablora_lowbit_gemm.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                     ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]


_lib.qablora_merge_noalloc.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
_lib.qblora_merge_dense.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                    ctypes.c_size_t, ctypes.c_void_p]
_lib.qblora_merge_dense.restype = ctypes.c_int
_lib.qblora_kernel_launches.restype = ctypes.c_uint64
_lib.qblora_kernel_launches.argtypes = []
_lib.qblora_set_timing_events.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
_lib.qblora_dense_gemm.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                   ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
_lib.qblora_pack_codes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                   ctypes.c_size_t, ctypes.c_void_p]
_lib.qblora_unpack_codes.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
_lib.qblora_debug_set_wait_limit.argtypes = [ctypes.c_int64]
_lib.qblora_debug_drop_load.argtypes = [ctypes.c_int32]
_lib.qblora_debug_hold_producer.argtypes = [ctypes.c_int64]


def kernel_launches() -> int:
    return int(_lib.qblora_kernel_launches())


def set_timing_events(start, stop) -> None:
    """Arm (torch.cuda.Event, already recorded once or created with enable_timing) or disarm (None, None)."""
    if start is None:
        _lib.qblora_set_timing_events(None, None)
    else:
        _lib.qblora_set_timing_events(start.cuda_event, stop.cuda_event)


def debug_set_wait_limit(cycles: int) -> None:
    """Test hook: device-side waits of kernels launched from now on give up after `cycles` cycles (0 = default)."""
    _check_plain(_lib.qblora_debug_set_wait_limit(int(cycles)))


def debug_drop_load(iteration: int) -> None:
    """Test hook: the next fused-contraction launch leaves out one weight load (see the header); negative = disarm."""
    _check_plain(_lib.qblora_debug_drop_load(int(iteration)))


def debug_hold_producer(cycles: int) -> None:
    """Test hook: the producers of the next adapted fused-contraction launch idle `cycles` cycles before their
    first adapter K-block (see the header); 0 = disarm."""
    _check_plain(_lib.qblora_debug_hold_producer(int(cycles)))


def _check_plain(status: int):
    if status != OK:
        raise RuntimeError(f"status {status}")


class QbloraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {_lib.qblora_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != OK:
        raise QbloraError(status, where)


def status_string(status: int) -> str:
    return _lib.qblora_status_string(status).decode()


def default_code_table() -> List[float]:
    buf = (ctypes.c_float * 16)()
    _check(_lib.qblora_default_code_table(buf), "qblora_default_code_table")
    return list(buf)


@dataclass
class QWeight:
    """Frozen 4-bit weight: codes uint8 [d_out][d_in/2], alpha/beta fp32 [d_out/bo][d_in/bi] (device)."""
    d_out: int
    d_in: int
    block_in: int
    block_out: int
    qfmt: int
    code: List[float]
    codes: torch.Tensor
    alpha: torch.Tensor
    beta: Optional[torch.Tensor]
    code_bits: int = 4          # 4: codes one per nibble [d_out][d_in/2]; 2 / 3: dense storage [d_out][d_in*bits/8]

    def c_struct(self) -> _CQWeight:
        c = _CQWeight()
        c.d_in, c.d_out, c.block_in, c.block_out, c.qfmt = self.d_in, self.d_out, self.block_in, self.block_out, self.qfmt
        for j in range(16):
            c.code[j] = self.code[j] if self.code is not None else 0.0
        c.codes = self.codes.data_ptr()
        c.alpha = self.alpha.data_ptr()
        c.beta = self.beta.data_ptr() if self.beta is not None else None
        c.code_bits = int(self.code_bits)
        return c


@dataclass
class Adapter:
    """Balanced adapter: A bf16 [P][r], B bf16 [r][Q] (device); B None => A is the single matrix H [P][Q].
    scale_op picks the compress / restore operator pair (default: AvgPool & repeat_interleave)."""
    lambda_in: int
    lambda_out: int
    rank: int
    scaling: float
    A: torch.Tensor
    B: Optional[torch.Tensor]
    scale_op: int = SCALE_AVGPOOL_REPEAT

    def c_struct(self) -> _CAdapter:
        c = _CAdapter()
        c.lambda_in, c.lambda_out, c.rank, c.scaling = self.lambda_in, self.lambda_out, self.rank, self.scaling
        c.scale_op = int(self.scale_op)
        c.A = self.A.data_ptr()
        c.B = self.B.data_ptr() if self.B is not None else None
        return c


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _dt(torch_dtype) -> int:
    if torch_dtype == torch.float32:
        return F32
    if torch_dtype == torch.bfloat16:
        return BF16
    raise ValueError(f"unsupported dtype {torch_dtype}")


def _ref(obj):
    return ctypes.byref(obj) if obj is not None else None


def workspace_bytes(op: int, qw: QWeight, ad: Optional[Adapter], tokens: int) -> int:
    cq = qw.c_struct()
    ca = ad.c_struct() if ad is not None else None
    return int(_lib.qblora_workspace_bytes(op, ctypes.byref(cq), _ref(ca), tokens))


def alloc_workspace(op: int, qw: QWeight, ad: Optional[Adapter], tokens: int) -> torch.Tensor:
    n = max(workspace_bytes(op, qw, ad, tokens), 256)
    return torch.empty(n, dtype=torch.uint8, device=qw.codes.device)


def device_status(ws: torch.Tensor, stream=None) -> int:
    return int(_lib.qblora_device_status(ws.data_ptr(), _stream_ptr(stream)))


def quantize_blockwise(W: torch.Tensor, block_in: int = 64, block_out: int = 1,
                       qfmt: int = FMT_CODEBOOK_ABSMAX, code: Optional[List[float]] = None,
                       stream=None, out: Optional[QWeight] = None) -> QWeight:
    """Quantizes W [d_out][d_in] (fp32 or bf16).  `out`: a QWeight of the same geometry whose tensors are
    overwritten (no allocation in the call)."""
    assert W.is_cuda and W.is_contiguous() and W.dim() == 2
    d_out, d_in = W.shape
    if qfmt == FMT_CODEBOOK_ABSMAX and code is None:
        code = default_code_table()
    if out is not None:
        assert (out.d_out, out.d_in, out.block_in, out.block_out, out.qfmt) == (d_out, d_in, block_in, block_out, qfmt)
        codes, alpha, beta = out.codes, out.alpha, out.beta
    else:
        codes = torch.empty((d_out, d_in // 2), dtype=torch.uint8, device=W.device)
        alpha = torch.empty((max(d_out // block_out, 1), max(d_in // block_in, 1)), dtype=torch.float32, device=W.device)
        beta = torch.empty_like(alpha) if qfmt == FMT_AFFINE_MINMAX else None
    ctab = (ctypes.c_float * 16)(*code) if code is not None else None
    st = _lib.qblora_quantize_blockwise(W.data_ptr(), _dt(W.dtype), d_out, d_in, block_in, block_out, qfmt,
                                        ctab, codes.data_ptr(), alpha.data_ptr(),
                                        beta.data_ptr() if beta is not None else None, _stream_ptr(stream))
    _check(st, "qblora_quantize_blockwise")
    return QWeight(d_out, d_in, block_in, block_out, qfmt, list(code) if code is not None else [0.0] * 16,
                   codes, alpha, beta)


def quantize_minmax_nbit(W: torch.Tensor, bits: int, block_in: int = 64, block_out: int = 1, stream=None) -> QWeight:
    """Min-max quantization of W [d_out][d_in] (fp32 or bf16) on a 2^bits-level grid (Eq. 1 with N = bits).
    The codes stay one per nibble, so the result is an ordinary min-max QWeight for every other call."""
    assert W.is_cuda and W.is_contiguous() and W.dim() == 2
    d_out, d_in = W.shape
    codes = torch.empty((d_out, d_in // 2), dtype=torch.uint8, device=W.device)
    alpha = torch.empty((max(d_out // block_out, 1), max(d_in // block_in, 1)), dtype=torch.float32, device=W.device)
    beta = torch.empty_like(alpha)
    st = _lib.qblora_quantize_minmax_nbit(W.data_ptr(), _dt(W.dtype), d_out, d_in, block_in, block_out, int(bits),
                                          codes.data_ptr(), alpha.data_ptr(), beta.data_ptr(), _stream_ptr(stream))
    _check(st, "qblora_quantize_minmax_nbit")
    return QWeight(d_out, d_in, block_in, block_out, FMT_AFFINE_MINMAX, [0.0] * 16, codes, alpha, beta)


def linear_fwd(qw: QWeight, ad: Optional[Adapter], X: torch.Tensor, out_dtype=torch.bfloat16,
               ws: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    assert X.is_cuda and X.is_contiguous() and X.dtype == torch.bfloat16
    T = X.shape[0]
    Y = out if out is not None else torch.empty((T, qw.d_out), dtype=out_dtype, device=X.device)
    if ws is None:
        ws = alloc_workspace(OP_LINEAR_FWD, qw, ad, T)
    cq = qw.c_struct()
    ca = ad.c_struct() if ad is not None else None
    st = _lib.qblora_linear_fwd(ctypes.byref(cq), _ref(ca), X.data_ptr(), T, Y.data_ptr(), _dt(Y.dtype),
                                ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    _check(st, "qblora_linear_fwd")
    return Y


def linear_bwd(qw: QWeight, ad: Optional[Adapter], X: Optional[torch.Tensor], dY: torch.Tensor,
               dx_dtype=torch.bfloat16, need_dx: bool = True, need_da: bool = True, need_db: bool = True,
               ws: Optional[torch.Tensor] = None, outs: Optional[Tuple] = None, stream=None):
    """Returns (dX, dA, dB); entries are None where skipped."""
    assert dY.is_cuda and dY.is_contiguous() and dY.dtype == torch.bfloat16
    T = dY.shape[0]
    dev = dY.device
    if outs is not None:
        dX, dA, dB = outs
    else:
        dX = torch.empty((T, qw.d_in), dtype=dx_dtype, device=dev) if need_dx else None
        dA = dB = None
        if ad is not None:
            if need_da:
                dA = torch.empty(tuple(ad.A.shape), dtype=torch.float32, device=dev)
            if need_db and ad.B is not None:
                dB = torch.empty(tuple(ad.B.shape), dtype=torch.float32, device=dev)
    if ws is None:
        ws = alloc_workspace(OP_LINEAR_BWD, qw, ad, T)
    cq = qw.c_struct()
    ca = ad.c_struct() if ad is not None else None
    p = lambda t: t.data_ptr() if t is not None else None  # noqa: E731
    st = _lib.qblora_linear_bwd(ctypes.byref(cq), _ref(ca), p(X), dY.data_ptr(), T, p(dX),
                                _dt(dX.dtype) if dX is not None else BF16, p(dA), p(dB), ws.data_ptr(),
                                ws.numel(), _stream_ptr(stream))
    _check(st, "qblora_linear_bwd")
    return dX, dA, dB


def merge(qw: QWeight, ad: Adapter, in_place: bool = False, ws: Optional[torch.Tensor] = None,
          stream=None, beta_out: Optional[torch.Tensor] = None) -> QWeight:
    """QA-BLoRA merge: returns the weight with beta' (codes and alpha are shared, untouched).
    `beta_out`: preallocated fp32 tensor of beta's shape to receive beta'."""
    if qw.beta is None:
        raise QbloraError(ERR_INVALID_ARG, "qablora_merge")
    if beta_out is None:
        beta_out = qw.beta if in_place else torch.empty_like(qw.beta)
    if ws is None:
        ws = alloc_workspace(OP_MERGE, qw, ad, 0)
    cq = qw.c_struct()
    ca = ad.c_struct()
    st = _lib.qablora_merge(ctypes.byref(cq), ctypes.byref(ca), beta_out.data_ptr(), ws.data_ptr(),
                            ws.numel(), _stream_ptr(stream))
    _check(st, "qablora_merge")
    return QWeight(qw.d_out, qw.d_in, qw.block_in, qw.block_out, qw.qfmt, qw.code, qw.codes, qw.alpha, beta_out, qw.code_bits)


def merge_dense(qw: QWeight, ad: Optional[Adapter], out: Optional[torch.Tensor] = None,
                ws: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Dense 16-bit merge: bf16 [d_out][d_in] = dequantized weight + s * dense adapter update."""
    W = out if out is not None else torch.empty((qw.d_out, qw.d_in), dtype=torch.bfloat16, device=qw.codes.device)
    if ws is None:
        ws = alloc_workspace(OP_MERGE_DENSE, qw, ad, 0)
    cq = qw.c_struct()
    ca = ad.c_struct() if ad is not None else None
    st = _lib.qblora_merge_dense(ctypes.byref(cq), _ref(ca), W.data_ptr(), ws.data_ptr(), ws.numel(),
                                 _stream_ptr(stream))
    _check(st, "qblora_merge_dense")
    return W


def merge_noalloc(qw: QWeight, ad: Adapter, beta_out: torch.Tensor, stream=None) -> QWeight:
    """qablora_merge_noalloc: merge into the caller's ``beta_out`` using the library's built-in scratch.

    For callers that cannot allocate device memory at this point (see the header).  Nothing is
    allocated here either: ``beta_out`` (fp32, same shape as ``qw.beta``) comes from the caller.
    Raises QbloraError(ERR_TOO_LARGE) when (d_in/lambda_in)*(d_out/lambda_out) > 262144.
    """
    cq = qw.c_struct()
    ca = ad.c_struct()
    st = _lib.qablora_merge_noalloc(ctypes.byref(cq), ctypes.byref(ca), beta_out.data_ptr(), _stream_ptr(stream))
    _check(st, "qablora_merge_noalloc")
    return QWeight(qw.d_out, qw.d_in, qw.block_in, qw.block_out, qw.qfmt, qw.code, qw.codes, qw.alpha, beta_out, qw.code_bits)


def lowbit_gemm(qw: QWeight, X: torch.Tensor, out_dtype=torch.bfloat16, ws: Optional[torch.Tensor] = None,
                out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    assert X.is_cuda and X.is_contiguous() and X.dtype == torch.bfloat16
    T = X.shape[0]
    Y = out if out is not None else torch.empty((T, qw.d_out), dtype=out_dtype, device=X.device)
    if ws is None:
        ws = alloc_workspace(OP_LOWBIT_GEMM, qw, None, T)
    cq = qw.c_struct()
    st = _lib.qablora_lowbit_gemm(ctypes.byref(cq), X.data_ptr(), T, Y.data_ptr(), _dt(Y.dtype),
                                  ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    _check(st, "qablora_lowbit_gemm")
    return Y


def dense_gemm(W: torch.Tensor, X: torch.Tensor, out_dtype=torch.bfloat16, ws: Optional[torch.Tensor] = None,
               out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """qblora_dense_gemm: Y = X W^T for a dense bf16 weight [d_out][d_in] (the merged 16-bit deployment)."""
    assert W.is_cuda and W.is_contiguous() and W.dtype == torch.bfloat16 and W.dim() == 2
    assert X.is_cuda and X.is_contiguous() and X.dtype == torch.bfloat16 and X.shape[1] == W.shape[1]
    T = X.shape[0]
    d_out, d_in = W.shape
    Y = out if out is not None else torch.empty((T, d_out), dtype=out_dtype, device=X.device)
    if ws is None:
        ws = torch.empty(256, dtype=torch.uint8, device=X.device)
    st = _lib.qblora_dense_gemm(W.data_ptr(), d_out, d_in, X.data_ptr(), T, Y.data_ptr(), _dt(Y.dtype), ws.data_ptr(),
                                ws.numel(), _stream_ptr(stream))
    _check(st, "qblora_dense_gemm")
    return Y


def pack_codes(qw: QWeight, bits: int, stream=None) -> QWeight:
    """qblora_pack_codes: the same weight with its codes in dense `bits`-bit storage (bits = 2 or 3)."""
    assert qw.code_bits == 4
    packed = torch.empty((qw.d_out, qw.d_in * bits // 8), dtype=torch.uint8, device=qw.codes.device)
    ws = torch.empty(256, dtype=torch.uint8, device=qw.codes.device)
    st = _lib.qblora_pack_codes(qw.codes.data_ptr(), qw.d_out, qw.d_in, int(bits), packed.data_ptr(), ws.data_ptr(), ws.numel(),
                                _stream_ptr(stream))
    _check(st, "qblora_pack_codes")
    _check(device_status(ws, stream), "qblora_pack_codes (a code does not fit)")
    return QWeight(qw.d_out, qw.d_in, qw.block_in, qw.block_out, qw.qfmt, qw.code, packed, qw.alpha, qw.beta, int(bits))


def unpack_codes(qw: QWeight, stream=None) -> QWeight:
    """qblora_unpack_codes: dense storage back to one code per nibble."""
    assert qw.code_bits in (2, 3)
    codes = torch.empty((qw.d_out, qw.d_in // 2), dtype=torch.uint8, device=qw.codes.device)
    st = _lib.qblora_unpack_codes(qw.codes.data_ptr(), qw.d_out, qw.d_in, int(qw.code_bits), codes.data_ptr(), _stream_ptr(stream))
    _check(st, "qblora_unpack_codes")
    return QWeight(qw.d_out, qw.d_in, qw.block_in, qw.block_out, qw.qfmt, qw.code, codes, qw.alpha, qw.beta, 4)
