"""Pins for the oracle's forward, backward, dense-update, merge and low-bit product.

The reference computations below use numpy library routines (reshape/mean,
matmul, repeat) in the order the paper's prose gives them (Sec. 3.1-3.3), which
is independent of the oracle's index-by-index loops.
"""
import numpy as np
import pytest

import oracle
from paper_2407_17029_b200 import synth


def make(seed, T, d_out, d_in, l1, l2, r, s=0.75, qfmt=0, ab_std=0.2, single=False):
    W = synth.normal(seed, "W", (d_out, d_in), 0.02)
    X = synth.round_to_bf16(synth.normal(seed, "X", (T, d_in)))
    dY = synth.round_to_bf16(synth.normal(seed, "dY", (T, d_out)))
    P, Q = d_in // l1, d_out // l2
    if single:
        A = synth.round_to_bf16(synth.normal(seed, "H", (P, Q), ab_std))
        B = None
    else:
        A = synth.round_to_bf16(synth.normal(seed, "A", (P, r), ab_std))
        B = synth.round_to_bf16(synth.normal(seed, "B", (r, Q), ab_std))
    bi = 64 if d_in % 64 == 0 else d_in
    qw = oracle.quantize_blockwise(W, bi, 1, qfmt)
    ad = oracle.Adapter(l1, l2, r, s, A, B)
    return qw, ad, X, dY


def np_forward(Wt, ad, X):
    """Sec. 3.2 in library calls: AvgPool -> A -> B -> repeat_interleave, scaled, added."""
    T, d_in = X.shape
    Xd = X.astype(np.float64)
    xp = Xd.reshape(T, d_in // ad.lambda_in, ad.lambda_in).mean(axis=2)
    H = ad.A.astype(np.float64) @ ad.B.astype(np.float64) if ad.B is not None else ad.A.astype(np.float64)
    v = xp @ H
    return Xd @ Wt.T + ad.scaling * np.repeat(v, ad.lambda_out, axis=1)


def np_delta_w(ad):
    """Equivalent dense update in the paper's (D_in, D_out) orientation:
    repeat (A B) lambda1 times along the input axis, divide by lambda1, repeat lambda2
    times along the output axis (paragraph after Eq. 2; intent of Algorithm 1's second routine)."""
    H = ad.A.astype(np.float64) @ ad.B.astype(np.float64) if ad.B is not None else ad.A.astype(np.float64)
    return np.repeat(np.repeat(H, ad.lambda_in, axis=0) / ad.lambda_in, ad.lambda_out, axis=1)


def rel(a, b):
    return np.abs(a - b).max() / max(np.abs(b).max(), 1e-300)


@pytest.mark.parametrize("l1,l2", [(1, 1), (2, 2), (4, 4), (64, 8), (8, 2)])
def test_forward_matches_library_restatement(l1, l2):
    qw, ad, X, _ = make(11, 6, 64, 128, l1, l2, 12)
    Wt = oracle.dequantize(qw)
    Y = oracle.linear_fwd(Wt, ad, X)
    assert rel(Y, np_forward(Wt, ad, X)) < 1e-12
    # the adapter term is a visible part of the output in this test
    base = oracle.linear_fwd(Wt, None, X)
    assert np.sqrt(np.mean((Y - base) ** 2)) > 0.05 * np.sqrt(np.mean(base ** 2))


def test_lambda_one_is_textbook_lora():
    qw, ad, X, _ = make(12, 5, 64, 64, 1, 1, 8)
    Wt = oracle.dequantize(qw)
    Xd = X.astype(np.float64)
    ref = Xd @ Wt.T + ad.scaling * (Xd @ ad.A.astype(np.float64) @ ad.B.astype(np.float64))
    assert rel(oracle.linear_fwd(Wt, ad, X), ref) < 1e-12


def test_zero_B_reproduces_plain_dequantized_linear_exactly():
    qw, ad, X, _ = make(13, 7, 64, 128, 4, 4, 16)
    ad0 = oracle.Adapter(ad.lambda_in, ad.lambda_out, ad.rank, ad.scaling, ad.A, np.zeros_like(ad.B))
    Wt = oracle.dequantize(qw)
    Y0 = oracle.linear_fwd(Wt, ad0, X)
    assert np.array_equal(Y0, oracle.linear_fwd(Wt, None, X))
    assert rel(Y0, X.astype(np.float64) @ Wt.T) < 1e-12


@pytest.mark.parametrize("l1,l2,single", [(2, 2, False), (4, 8, False), (64, 8, False), (8, 8, True)])
def test_dense_equivalent_weight(l1, l2, single):
    qw, ad, X, dY = make(14, 5, 64, 128, l1, l2, 10, single=single)
    Wt = oracle.dequantize(qw)
    dW = oracle.dense_delta_w(64, 128, ad)
    assert rel(dW, np_delta_w(ad).T) < 1e-13                    # storage is the transpose
    # block-constant: D_in*D_out/(l1*l2) tiles of equal elements
    tiles = dW.reshape(64 // l2, l2, 128 // l1, l1)
    assert np.all(tiles == tiles[:, :1, :, :1])
    assert tiles[:, 0, :, 0].size == 64 * 128 // (l1 * l2)
    # forward and dX through the dense weight
    Y = oracle.linear_fwd(Wt, ad, X)
    Wm = Wt + ad.scaling * dW
    assert rel(Y, X.astype(np.float64) @ Wm.T) < 1e-12
    dX, _, _ = oracle.linear_bwd(Wt, ad, X, dY)
    assert rel(dX, dY.astype(np.float64) @ Wm) < 1e-12


def test_eq2_input_compression_condition():
    # pooling then multiplying by w_in equals the dense product when w_in = lambda1 * w (Eq. 2)
    l1, d_in, d_out = 4, 32, 5
    w_in = synth.normal(15, "win", (d_in // l1, d_out)).astype(np.float64)
    x = synth.normal(15, "x", (d_in,)).astype(np.float64)
    pooled = x.reshape(-1, l1).mean(axis=1)
    dense = np.repeat(w_in, l1, axis=0) / l1
    assert np.allclose(w_in.T @ pooled, dense.T @ x, rtol=1e-13)
    # same statement through the oracle in single-matrix mode (H = w_in, lambda2 = 1)
    Hf = synth.round_to_bf16(w_in.astype(np.float32))
    ad = oracle.Adapter(l1, 1, 0, 1.0, Hf, None)
    xb = synth.round_to_bf16(x.astype(np.float32))[None, :]
    Y = oracle.linear_fwd(np.zeros((d_out, d_in)), ad, xb)
    assert np.allclose(Y[0], (np.repeat(Hf.astype(np.float64), l1, 0) / l1).T @ xb[0].astype(np.float64), rtol=1e-13)


def test_parameter_count_is_invariant_in_lambda():
    d_in, d_out, d_rank = 4096, 4096, 64
    for lam in (1, 2, 4, 8):
        assert (d_in // lam) * (lam * d_rank) == d_in * d_rank          # A
        assert (lam * d_rank) * (d_out // lam) == d_rank * d_out        # B


@pytest.mark.parametrize("l1,l2,single", [(1, 1, False), (2, 4, False), (4, 2, False), (4, 4, True)])
def test_backward_finite_differences(l1, l2, single):
    T, d_out, d_in, r = 3, 8, 16, 5
    qw, ad, X, dY = make(16, T, d_out, d_in, l1, l2, r, s=1.3, single=single)
    Wt = oracle.dequantize(qw)
    G = dY.astype(np.float64)
    dX, dA, dB = oracle.linear_bwd(Wt, ad, X, dY)

    def loss(Xv, Av, Bv):
        a = oracle.Adapter(l1, l2, r, ad.scaling, Av, Bv)
        return float((G * np_forward(Wt, a, Xv)).sum())

    h = 1e-5
    Xd, Ad = X.astype(np.float64), ad.A.astype(np.float64)
    Bd = None if single else ad.B.astype(np.float64)

    def fd(arr, which):
        g = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            p = arr.copy(); p[idx] += h
            m = arr.copy(); m[idx] -= h
            args_p = {"X": (p, Ad, Bd), "A": (Xd, p, Bd), "B": (Xd, Ad, p)}[which]
            args_m = {"X": (m, Ad, Bd), "A": (Xd, m, Bd), "B": (Xd, Ad, m)}[which]
            g[idx] = (loss(*args_p) - loss(*args_m)) / (2 * h)
        return g

    assert rel(dX, fd(Xd, "X")) < 1e-7
    assert rel(dA, fd(Ad, "A")) < 1e-7
    if not single:
        assert rel(dB, fd(Bd, "B")) < 1e-7


def test_backward_adjoint_identity():
    # <dY, J d> == <J^T dY, d> for the map (X, A, B) -> Y linearised at the current point
    qw, ad, X, dY = make(17, 4, 16, 32, 4, 2, 6, s=0.9)
    Wt = oracle.dequantize(qw)
    dX, dA, dB = oracle.linear_bwd(Wt, ad, X, dY)
    eX = synth.normal(17, "eX", X.shape).astype(np.float64)
    eA = synth.normal(17, "eA", ad.A.shape).astype(np.float64)
    eB = synth.normal(17, "eB", ad.B.shape).astype(np.float64)
    h = 1e-6

    def f(k):
        a = oracle.Adapter(4, 2, 6, ad.scaling, ad.A + k * eA, ad.B + k * eB)
        return np_forward(Wt, a, X.astype(np.float64) + k * eX)

    Jd = (f(h) - f(-h)) / (2 * h)
    lhs = float((dY.astype(np.float64) * Jd).sum())
    rhs = float((dX * eX).sum() + (dA * eA).sum() + (dB * eB).sum())
    assert abs(lhs - rhs) < 1e-7 * max(abs(lhs), 1.0)


def test_backward_skips_and_adapter_grads_need_no_weight():
    qw, ad, X, dY = make(18, 6, 64, 128, 64, 8, 16)
    Wt = oracle.dequantize(qw)
    dX, dA, dB = oracle.linear_bwd(Wt, ad, X, dY)
    _, dA2, dB2 = oracle.linear_bwd(None, ad, X, dY, want_dx=False)
    assert np.array_equal(dA, dA2) and np.array_equal(dB, dB2)
    dX0, _, _ = oracle.linear_bwd(Wt, None, X, dY)
    assert rel(dX0, dY.astype(np.float64) @ Wt) < 1e-12


@pytest.mark.parametrize("single", [False, True])
@pytest.mark.parametrize("s", [1.0, 37.5])
def test_merge_identity(single, s):
    qw, ad, X, _ = make(19, 9, 64, 256, 64, 8, 24, s=s, qfmt=1, single=single)
    Wt = oracle.dequantize(qw)
    merged = oracle.merge(qw, ad)
    assert merged.codes is qw.codes and merged.alpha is qw.alpha        # only beta changes
    Y_unmerged = oracle.linear_fwd(Wt, ad, X)
    Y_merged = oracle.lowbit_gemm(merged, X)
    assert rel(Y_merged, Y_unmerged) < 1e-6
    # element-wise: alpha*code + beta' == w~ + s*dW, up to the single fp32 rounding of beta'
    Wm = oracle.dequantize(merged)
    target = Wt + s * oracle.dense_delta_w(64, 256, ad)
    tol = np.abs(np.repeat(merged.beta, 64, axis=1)).astype(np.float64) * 2.0 ** -24 + 1e-300
    assert np.all(np.abs(Wm - target) <= tol)
    # beta' against the library restatement of Algorithm 2's new-beta routine
    H = np_delta_w(ad).T[:, ::64][::1]                                   # [d_out][G] sample of dW
    ref = (qw.beta.astype(np.float64) + s * H).astype(np.float32)
    assert np.array_equal(merged.beta, ref)


def test_merge_zero_adapter_and_misalignment():
    qw, ad, X, _ = make(20, 3, 64, 256, 64, 8, 8, qfmt=1)
    ad0 = oracle.Adapter(64, 8, 8, 1.0, ad.A, np.zeros_like(ad.B))
    assert np.array_equal(oracle.merge(qw, ad0).beta.view(np.uint32), qw.beta.view(np.uint32))
    bad = oracle.Adapter(4, 4, 8, 1.0, np.zeros((64, 8), np.float32), np.zeros((8, 16), np.float32))
    with pytest.raises(ValueError):
        oracle.merge(qw, bad)          # a 64-wide block would straddle sixteen 4-wide tiles
    with pytest.raises(ValueError):
        oracle.merge(oracle.quantize_blockwise(np.zeros((64, 256), np.float32), 64, 1, 0), ad)


def test_merge_two_dimensional_blocks():
    # the paper's native geometry: quantization block (lambda1 x lambda2) = (8 in x 8 out)
    W = synth.normal(21, "W2d", (64, 128), 0.02)
    qw = oracle.quantize_blockwise(W, 8, 8, oracle.FMT_AFFINE_MINMAX)
    H = synth.round_to_bf16(synth.normal(21, "H2d", (16, 8), 0.05))
    ad = oracle.Adapter(8, 8, 0, 2.0, H, None)
    X = synth.round_to_bf16(synth.normal(21, "X2d", (4, 128)))
    merged = oracle.merge(qw, ad)
    assert rel(oracle.lowbit_gemm(merged, X), oracle.linear_fwd(oracle.dequantize(qw), ad, X)) < 1e-6


def test_lowbit_gemm_is_dequantized_product():
    qw, _, X, _ = make(22, 5, 64, 128, 1, 1, 4, qfmt=1)
    assert rel(oracle.lowbit_gemm(qw, X), X.astype(np.float64) @ oracle.dequantize(qw).T) < 1e-12
