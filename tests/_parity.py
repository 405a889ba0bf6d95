"""Helpers shared by the GPU parity tests: numpy <-> device marshalling and the tolerance gates.

Gates (floating-point outputs; the oracle is fp64).  "The output" of the layer is the vector it
produces for one token (the paper's y = W^T x), so Y and dX are normalised by the RMS of their own
token row; the weight gradients dA and dB are single matrices and use their global RMS:
  strict  -- fp32 outputs (the accumulator before the final rounding) and fp32 gradients:
             max|gpu - ora| / rms <= 1e-2.
  bf16    -- bf16 outputs: rms(gpu - ora) / rms(ora) <= 1e-2 overall and, per element,
             |gpu - ora| <= 1e-2 * rms + 2^-7 * |ora|   (one bf16 ulp of the value itself).
Integer results (codes) and fp32 quantization parameters are compared bit for bit.
"""
import numpy as np
import torch

import oracle
from paper_2407_17029_b200 import binding as qb
from paper_2407_17029_b200 import synth

DEV = "cuda:0"
TOL = 1e-2


def to_bf16_dev(a: np.ndarray) -> torch.Tensor:
    bits = synth.bf16_bits(a).view(np.int16)
    return torch.from_numpy(bits.copy()).to(DEV).view(torch.bfloat16)


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def rms(a):
    return float(np.sqrt(np.mean(np.square(a, dtype=np.float64))))


def _scale(ora, per_row):
    """RMS the error is normalised by: per token row (column vector of shape [T,1]) or global."""
    if per_row and ora.ndim == 2:
        return np.maximum(np.sqrt(np.mean(np.square(ora, dtype=np.float64), axis=1, keepdims=True)), 1e-30)
    return max(rms(ora), 1e-30)


# Every gate call leaves a record (label, gate, worst error by the gate's own normalisation, the same maximum
# normalised by the GLOBAL rms of the reference, rms error / rms reference); conftest prints the tightest ones at
# the end of a run, so the margin to the 1e-2 bar is on show next to the pass / fail.
MARGINS = []


def _record(what, gate, worst, gpu, ora):
    g = max(rms(ora), 1e-30)
    MARGINS.append((what, gate, float(worst), float(np.abs(gpu - ora).max() / g), float(rms(gpu - ora) / g)))


def gate_strict(gpu, ora, what="", per_row=True):
    gpu = np.asarray(gpu, dtype=np.float64)
    r = _scale(ora, per_row)
    err = float((np.abs(gpu - ora) / r).max())
    _record(what, "strict/row" if per_row and np.ndim(ora) == 2 else "strict/global", err, gpu, ora)
    assert np.isfinite(gpu).all(), f"{what}: non-finite output"
    assert err <= TOL, f"{what}: max|gpu-ora|/rms = {err:.3e} > {TOL}"
    return err


def gate_bf16(gpu, ora, what="", per_row=True):
    gpu = np.asarray(gpu, dtype=np.float64)
    assert np.isfinite(gpu).all(), f"{what}: non-finite output"
    rel = rms(gpu - ora) / max(rms(ora), 1e-30)
    _record(what, "bf16", rel, gpu, ora)
    assert rel <= TOL, f"{what}: rms rel err {rel:.3e} > {TOL}"
    bound = TOL * _scale(ora, per_row) + 2.0 ** -7 * np.abs(ora)
    worst = float((np.abs(gpu - ora) / bound).max())
    assert worst <= 1.0, f"{what}: element error {worst:.3f} x bound"
    return rel


def qweight_to_dev(qw: oracle.QWeight) -> qb.QWeight:
    code = [float(x) for x in qw.code] if qw.code is not None else [0.0] * 16
    return qb.QWeight(qw.d_out, qw.d_in, qw.block_in, qw.block_out, qw.qfmt, code, to_dev(qw.codes),
                      to_dev(qw.alpha), to_dev(qw.beta) if qw.beta is not None else None)


def adapter_to_dev(ad: oracle.Adapter) -> qb.Adapter:
    return qb.Adapter(ad.lambda_in, ad.lambda_out, ad.rank, float(ad.scaling), to_bf16_dev(ad.A),
                      to_bf16_dev(ad.B) if ad.B is not None else None, int(ad.scale_op))


def visible_scaling(Wt, ad: oracle.Adapter, X) -> float:
    """Scaling s* (fp32-representable) at which the adapter term's RMS equals the base term's."""
    base = oracle.linear_fwd(Wt, None, X)
    one = oracle.Adapter(ad.lambda_in, ad.lambda_out, ad.rank, 1.0, ad.A, ad.B, ad.scale_op)
    term = oracle.linear_fwd(Wt, one, X) - base
    return float(np.float32(rms(base) / max(rms(term), 1e-30)))


def sample_rows(seed: int, T: int, n: int) -> np.ndarray:
    if n >= T:
        return np.arange(T)
    g = np.random.Generator(np.random.Philox(key=seed + 977))
    return np.sort(g.choice(T, size=n, replace=False))


# ------------------------------------------------------------------------------------------------ guard bands
# Every output and workspace buffer of a guarded call sits between two 4 KiB bands of a known byte pattern that
# are checked after the call: a store past either end of Y, dX, dA, dB, beta', the codes, the scales or the
# workspace fails the test even when all values inside the buffer are right.
GUARD_BYTES = 4096
GUARD_PATTERN = 0xA5


class Guarded:
    def __init__(self):
        self.bufs = []

    def alloc(self, shape, dtype):
        shape = tuple(int(x) for x in shape)
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        raw = torch.full((n + 2 * GUARD_BYTES,), GUARD_PATTERN, dtype=torch.uint8, device=DEV)
        self.bufs.append((raw, n))
        return raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)

    def workspace(self, op, qw, ad, tokens):
        return self.alloc((max(qb.workspace_bytes(op, qw, ad, tokens), 256),), torch.uint8)

    def check(self, what=""):
        torch.cuda.synchronize()
        for raw, n in self.bufs:
            lo, hi = raw[:GUARD_BYTES], raw[GUARD_BYTES + n:]
            assert bool((lo == GUARD_PATTERN).all()), f"{what}: bytes in front of a {n}-byte buffer were overwritten"
            assert bool((hi == GUARD_PATTERN).all()), f"{what}: bytes behind a {n}-byte buffer were overwritten"


def g_linear_fwd(dq, da, Xd, dtype):
    g = Guarded()
    Y = g.alloc((Xd.shape[0], dq.d_out), dtype)
    ws = g.workspace(qb.OP_LINEAR_FWD, dq, da, Xd.shape[0])
    qb.linear_fwd(dq, da, Xd, ws=ws, out=Y)
    g.check("linear_fwd")
    assert qb.device_status(ws) == qb.OK
    return Y


def g_linear_bwd(dq, da, Xd, dYd, dtype, need_dx=True, need_da=True, need_db=True):
    g = Guarded()
    T = dYd.shape[0]
    dX = g.alloc((T, dq.d_in), dtype) if need_dx else None
    dA = g.alloc(tuple(da.A.shape), torch.float32) if (da is not None and need_da) else None
    dB = g.alloc(tuple(da.B.shape), torch.float32) if (da is not None and da.B is not None and need_db) else None
    ws = g.workspace(qb.OP_LINEAR_BWD, dq, da, T)
    qb.linear_bwd(dq, da, Xd, dYd, ws=ws, outs=(dX, dA, dB))
    g.check("linear_bwd")
    assert qb.device_status(ws) == qb.OK
    return dX, dA, dB


def g_lowbit_gemm(dq, Xd, dtype):
    g = Guarded()
    Y = g.alloc((Xd.shape[0], dq.d_out), dtype)
    ws = g.workspace(qb.OP_LOWBIT_GEMM, dq, None, Xd.shape[0])
    qb.lowbit_gemm(dq, Xd, ws=ws, out=Y)
    g.check("lowbit_gemm")
    assert qb.device_status(ws) == qb.OK
    return Y


def g_quantize(Wd, bi, bo, qfmt, code=None):
    g = Guarded()
    d_out, d_in = Wd.shape
    codes = g.alloc((d_out, d_in // 2), torch.uint8)
    alpha = g.alloc((d_out // bo, d_in // bi), torch.float32)
    beta = g.alloc((d_out // bo, d_in // bi), torch.float32) if qfmt == qb.FMT_AFFINE_MINMAX else None
    if qfmt == qb.FMT_CODEBOOK_ABSMAX and code is None:
        code = qb.default_code_table()
    out = qb.QWeight(d_out, d_in, bi, bo, qfmt, list(code) if code is not None else [0.0] * 16, codes, alpha, beta)
    got = qb.quantize_blockwise(Wd, bi, bo, qfmt, code, out=out)
    g.check("quantize_blockwise")
    return got
