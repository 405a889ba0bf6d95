"""Pins for the oracle's alternative scale operators (the Sec. 4 ablation on scale operators:
truncation & supplement_0, interval_sampling & interpolation, beside AvgPool & repeat_interleave).

The restatements below use numpy slicing and padding (``X[:, :P]``, ``X[:, ::l1]``, zero arrays
written through slices) in the order the paper's descriptions give them, which is independent
of the oracle's index-by-index loops.
"""
import numpy as np
import pytest

import oracle
from paper_2407_17029_b200 import synth

TRUNC, SAMPLE = oracle.OP_TRUNCATE_ZEROPAD, oracle.OP_SAMPLE_ZEROFILL


def make(seed, T, d_out, d_in, l1, l2, r, op, s=0.75, single=False, ab_std=0.2):
    W = synth.normal(seed, "W", (d_out, d_in), 0.02)
    X = synth.round_to_bf16(synth.normal(seed, "X", (T, d_in)))
    dY = synth.round_to_bf16(synth.normal(seed, "dY", (T, d_out)))
    P, Q = d_in // l1, d_out // l2
    if single:
        A, B = synth.round_to_bf16(synth.normal(seed, "H", (P, Q), ab_std)), None
    else:
        A = synth.round_to_bf16(synth.normal(seed, "A", (P, r), ab_std))
        B = synth.round_to_bf16(synth.normal(seed, "B", (r, Q), ab_std))
    bi = 64 if d_in % 64 == 0 else d_in
    qw = oracle.quantize_blockwise(W, bi, 1, 0)
    return qw, oracle.Adapter(l1, l2, r, s, A, B, op), X, dY


def np_forward(Wt, ad, X):
    """Compress the input, two linear maps, restore the output size, scale, add (Sec. 3.2 with
    the operator pair swapped as the ablation describes)."""
    T, d_in = X.shape
    d_out = Wt.shape[0]
    P, Q = d_in // ad.lambda_in, d_out // ad.lambda_out
    Xd = X.astype(np.float64)
    H = ad.A.astype(np.float64) @ ad.B.astype(np.float64) if ad.B is not None else ad.A.astype(np.float64)
    full = np.zeros((T, d_out))
    if ad.scale_op == TRUNC:
        full[:, :Q] = Xd[:, :P] @ H                       # keep the front part; pad with zeros
    else:
        full[:, ::ad.lambda_out] = Xd[:, ::ad.lambda_in] @ H   # every l1-th value; zeros between outputs
    return Xd @ Wt.T + ad.scaling * full


def np_delta_w_storage(ad, d_out, d_in):
    """Equivalent dense update in storage order [d_out][d_in]."""
    H = ad.A.astype(np.float64) @ ad.B.astype(np.float64) if ad.B is not None else ad.A.astype(np.float64)
    P, Q = H.shape
    dW = np.zeros((d_out, d_in))
    if ad.scale_op == TRUNC:
        dW[:Q, :P] = H.T
    else:
        dW[::ad.lambda_out, ::ad.lambda_in] = H.T
    return dW


def rel(a, b):
    return np.abs(a - b).max() / max(np.abs(b).max(), 1e-300)


@pytest.mark.parametrize("op", [TRUNC, SAMPLE])
@pytest.mark.parametrize("l1,l2,single", [(2, 2, False), (4, 8, False), (64, 8, False), (8, 2, True)])
def test_forward_matches_library_restatement(op, l1, l2, single):
    qw, ad, X, _ = make(31, 5, 64, 128, l1, l2, 12, op, single=single)
    Wt = oracle.dequantize(qw)
    Y = oracle.linear_fwd(Wt, ad, X)
    assert rel(Y, np_forward(Wt, ad, X)) < 1e-12
    base = oracle.linear_fwd(Wt, None, X)
    assert np.abs(Y - base).max() > 1e-3                  # the adapter term is visible here
    # outputs that the expansion leaves untouched equal the base layer exactly
    Q = 64 // l2
    untouched = np.ones(64, bool)
    if op == TRUNC:
        untouched[:Q] = False
    else:
        untouched[::l2] = False
    assert np.array_equal(Y[:, untouched], base[:, untouched])
    assert untouched.sum() == 64 - Q


@pytest.mark.parametrize("op", [TRUNC, SAMPLE])
def test_lambda_one_is_textbook_lora_for_every_operator(op):
    qw, ad, X, dY = make(32, 4, 32, 64, 1, 1, 6, op)
    Wt = oracle.dequantize(qw)
    ref = oracle.Adapter(1, 1, 6, ad.scaling, ad.A, ad.B, oracle.OP_AVGPOOL_REPEAT)
    assert np.array_equal(oracle.linear_fwd(Wt, ad, X), oracle.linear_fwd(Wt, ref, X))
    for a, b in zip(oracle.linear_bwd(Wt, ad, X, dY), oracle.linear_bwd(Wt, ref, X, dY)):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("op", [TRUNC, SAMPLE])
@pytest.mark.parametrize("single", [False, True])
def test_dense_equivalent_weight(op, single):
    l1, l2 = 4, 2
    qw, ad, X, dY = make(33, 6, 16, 64, l1, l2, 5, op, single=single)
    Wt = oracle.dequantize(qw)
    dW = oracle.dense_delta_w(16, 64, ad)
    assert np.array_equal(dW, np_delta_w_storage(ad, 16, 64)) or rel(dW, np_delta_w_storage(ad, 16, 64)) < 1e-15
    # exactly P*Q entries can be non-zero: nothing is spread over the discarded channels
    assert np.count_nonzero(dW) <= (64 // l1) * (16 // l2)
    Weff = Wt + ad.scaling * dW
    assert rel(oracle.linear_fwd(Wt, ad, X), X.astype(np.float64) @ Weff.T) < 1e-12
    dX, _, _ = oracle.linear_bwd(Wt, ad, X, dY)
    assert rel(dX, dY.astype(np.float64) @ Weff) < 1e-12


def test_discarded_channels_do_not_reach_the_adapter():
    # the ablation's explanation: truncation and sampling drop channels outright, so a change in a
    # dropped channel moves the output only through the frozen base weight
    l1, l2 = 4, 4
    for op in (TRUNC, SAMPLE):
        qw, ad, X, _ = make(34, 3, 16, 64, l1, l2, 4, op)
        Wt = oracle.dequantize(qw)
        kept = np.zeros(64, bool)
        if op == TRUNC:
            kept[:16] = True
        else:
            kept[::l1] = True
        X2 = X.copy()
        X2[:, ~kept] += 1.0
        d_full = oracle.linear_fwd(Wt, ad, X2) - oracle.linear_fwd(Wt, ad, X)
        d_base = oracle.linear_fwd(Wt, None, X2) - oracle.linear_fwd(Wt, None, X)
        assert rel(d_full, d_base) < 1e-12
    # AvgPool sees every channel
    qw, ad, X, _ = make(34, 3, 16, 64, l1, l2, 4, oracle.OP_AVGPOOL_REPEAT)
    Wt = oracle.dequantize(qw)
    X2 = X.copy(); X2[:, 1::l1] += 1.0
    d_full = oracle.linear_fwd(Wt, ad, X2) - oracle.linear_fwd(Wt, ad, X)
    d_base = oracle.linear_fwd(Wt, None, X2) - oracle.linear_fwd(Wt, None, X)
    assert rel(d_full, d_base) > 1e-3


@pytest.mark.parametrize("op", [TRUNC, SAMPLE])
@pytest.mark.parametrize("l1,l2,single", [(2, 4, False), (4, 2, False), (4, 4, True)])
def test_backward_finite_differences(op, l1, l2, single):
    T, d_out, d_in, r = 3, 8, 16, 5
    qw, ad, X, dY = make(35, T, d_out, d_in, l1, l2, r, op, s=1.3, single=single)
    Wt = oracle.dequantize(qw)
    G = dY.astype(np.float64)
    dX, dA, dB = oracle.linear_bwd(Wt, ad, X, dY)

    def loss(Xv, Av, Bv):
        return float((G * np_forward(Wt, oracle.Adapter(l1, l2, r, ad.scaling, Av, Bv, op), Xv)).sum())

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


def test_merge_into_beta_is_refused_for_the_alternative_operators():
    # the update is no longer constant over a quantization block, so it is not a shift of beta
    W = synth.normal(36, "W", (16, 128), 0.02)
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX)
    A = synth.round_to_bf16(synth.normal(36, "A", (2, 4), 0.2))
    B = synth.round_to_bf16(synth.normal(36, "B", (4, 2), 0.2))
    for op in (TRUNC, SAMPLE):
        with pytest.raises(ValueError):
            oracle.merge(qw, oracle.Adapter(64, 8, 4, 1.0, A, B, op))
        dW = oracle.dense_delta_w(16, 128, oracle.Adapter(64, 8, 4, 1.0, A, B, op))
        assert not np.all(dW[:, :64] == dW[:, :1])
