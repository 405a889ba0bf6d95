"""GPU parity for the alternative scale operators of the Sec. 4 ablation (truncation & zero padding,
interval sampling & zero fill) against the fp64 CPU oracle: forward, backward, single-matrix
adapter, dense 16-bit merge, and the refusal to fold them into per-block offsets."""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_17029_b200 import synth
from tests._parity import adapter_to_dev, gate_bf16, gate_strict, qweight_to_dev, rms, to_bf16_dev, to_np64

pytestmark = pytest.mark.gpu

OPS = [oracle.OP_TRUNCATE_ZEROPAD, oracle.OP_SAMPLE_ZEROFILL]


@pytest.fixture(scope="module")
def qb():
    from paper_2407_17029_b200 import binding
    return binding


@pytest.fixture(params=["tensor-core", "general"])
def path(request, monkeypatch):
    if request.param == "general":
        monkeypatch.setenv("QBLORA_FORCE_GENERAL", "1")
    else:
        monkeypatch.delenv("QBLORA_FORCE_GENERAL", raising=False)
    return request.param


def make_case(seed, T, d_out, d_in, l1, l2, r, op, qfmt=0, bi=64, bo=1, single=False):
    tag = f"scaleop/{seed}"
    W = synth.normal(seed, tag + "/W", (d_out, d_in), 0.02)
    X, _ = synth.make_activations(seed, tag + "/X", T, d_in, 0.0)
    dY = synth.round_to_bf16(synth.normal(seed, tag + "/dY", (T, d_out)))
    P, Q = d_in // l1, d_out // l2
    if single:
        A, B = synth.round_to_bf16(synth.normal(seed, tag + "/H", (P, Q), 0.01)), None
    else:
        A = synth.round_to_bf16(synth.normal(seed, tag + "/A", (P, r), 0.01))
        B = synth.round_to_bf16(synth.normal(seed, tag + "/B", (r, Q), 0.01))
    qw = oracle.quantize_blockwise(W, bi, bo, qfmt)
    return qw, oracle.Adapter(l1, l2, r, 1.0, A, B, op), X, dY


def touched(op, lam, n):
    """Full-size positions (of n) that the operator pair ties to a compressed one."""
    m = np.zeros(n, bool)
    if op == oracle.OP_TRUNCATE_ZEROPAD:
        m[:n // lam] = True
    else:
        m[::lam] = True
    return m


# Adapter-visible scalings.  These operators put the whole adapter term on 1 / lambda of the outputs
# (forward) and of the inputs (backward), so "equal RMS over the row" would make the written elements
# sqrt(lambda) times larger than everything else in the row and a single bf16 rounding of such an
# element would already exceed 1e-2 of the row's RMS.  Instead the adapter term is set to HALF of the
# base term's RMS on the elements it is written to -- fifty times the tolerance, so a dropped,
# shifted or mis-scaled adapter term cannot pass -- separately for the forward and the backward pass.
def visible_scaling_fwd(Wt, ad, X):
    m = touched(ad.scale_op, ad.lambda_out, Wt.shape[0])
    base = oracle.linear_fwd(Wt, None, X)
    one = oracle.Adapter(ad.lambda_in, ad.lambda_out, ad.rank, 1.0, ad.A, ad.B, ad.scale_op)
    term = oracle.linear_fwd(Wt, one, X) - base
    return float(np.float32(0.5 * rms(base[:, m]) / max(rms(term[:, m]), 1e-30)))


def visible_scaling_bwd(Wt, ad, X, dY):
    m = touched(ad.scale_op, ad.lambda_in, Wt.shape[1])
    base, _, _ = oracle.linear_bwd(Wt, None, X, dY)
    one = oracle.Adapter(ad.lambda_in, ad.lambda_out, ad.rank, 1.0, ad.A, ad.B, ad.scale_op)
    term = oracle.linear_bwd(Wt, one, X, dY, want_da=False, want_db=False)[0] - base
    return float(np.float32(0.5 * rms(base[:, m]) / max(rms(term[:, m]), 1e-30)))


CASES = [
    # T, d_out, d_in, l1, l2, r -- several tiles with ragged tails in every dimension
    (300, 320, 448, 64, 8, 48),
    (300, 320, 448, 4, 4, 48),
    (77, 136, 192, 2, 1, 16),
    (515, 768, 640, 8, 8, 64),
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("visible", [False, True])
def test_fwd_bwd_parity(qb, path, case, op, visible):
    T, d_out, d_in, l1, l2, r = case
    qw, ad, X, dY = make_case(71, T, d_out, d_in, l1, l2, r, op, qfmt=op - 1)
    Wt = oracle.dequantize(qw)
    dq, Xd, dYd = qweight_to_dev(qw), to_bf16_dev(X), to_bf16_dev(dY)
    # forward
    if visible:
        ad.scaling = visible_scaling_fwd(Wt, ad, X)
    ref = oracle.linear_fwd(Wt, ad, X)
    da = adapter_to_dev(ad)
    gate_strict(to_np64(qb.linear_fwd(dq, da, Xd, torch.float32)), ref, "Y f32")
    gate_bf16(to_np64(qb.linear_fwd(dq, da, Xd, torch.bfloat16)), ref, "Y bf16")
    if visible:
        base = oracle.linear_fwd(Wt, None, X)
        m = touched(op, l2, d_out)
        assert rms((ref - base)[:, m]) > 0.45 * rms(base[:, m])
        # the operator differs from AvgPool & repeat_interleave by far more than the tolerance
        other = oracle.Adapter(l1, l2, r, ad.scaling, ad.A, ad.B, oracle.OP_AVGPOOL_REPEAT)
        assert rms(oracle.linear_fwd(Wt, other, X) - ref) > 0.05 * rms(ref)
    # backward
    if visible:
        ad.scaling = visible_scaling_bwd(Wt, ad, X, dY)
        da = adapter_to_dev(ad)
    rdX, rdA, rdB = oracle.linear_bwd(Wt, ad, X, dY)
    dX, dA, dB = qb.linear_bwd(dq, da, Xd, dYd, torch.float32)
    gate_strict(to_np64(dX), rdX, "dX f32")
    gate_strict(to_np64(dA), rdA, "dA", per_row=False)
    gate_strict(to_np64(dB), rdB, "dB", per_row=False)
    dXb, _, _ = qb.linear_bwd(dq, da, Xd, dYd, torch.bfloat16, need_da=False, need_db=False)
    gate_bf16(to_np64(dXb), rdX, "dX bf16")
    if visible:
        base = oracle.linear_bwd(Wt, None, X, dY)[0]
        m = touched(op, l1, d_in)
        assert rms((rdX - base)[:, m]) > 0.45 * rms(base[:, m])


@pytest.mark.parametrize("op", OPS)
def test_untouched_outputs_equal_the_base_layer_bit_for_bit(qb, path, op):
    T, d_out, d_in, l1, l2, r = 200, 320, 448, 64, 8, 48
    qw, ad, X, _ = make_case(72, T, d_out, d_in, l1, l2, r, op)
    ad.scaling = 50.0
    dq, da, Xd = qweight_to_dev(qw), adapter_to_dev(ad), to_bf16_dev(X)
    Y = qb.linear_fwd(dq, da, Xd, torch.float32).cpu().numpy()
    Y0 = qb.linear_fwd(dq, None, Xd, torch.float32).cpu().numpy()
    untouched = ~touched(op, l2, d_out)
    assert np.array_equal(Y[:, untouched], Y0[:, untouched])
    assert not np.array_equal(Y[:, ~untouched], Y0[:, ~untouched])


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("case", [(150, 128, 512, 8, 8), (300, 320, 448, 64, 8)])
def test_single_matrix_adapter(qb, path, op, case):
    T, d_out, d_in, l1, l2 = case
    qw, ad, X, dY = make_case(73, T, d_out, d_in, l1, l2, 0, op, qfmt=1, single=True)
    Wt = oracle.dequantize(qw)
    ad.scaling = visible_scaling_fwd(Wt, ad, X)
    dq, Xd, dYd = qweight_to_dev(qw), to_bf16_dev(X), to_bf16_dev(dY)
    gate_strict(to_np64(qb.linear_fwd(dq, adapter_to_dev(ad), Xd, torch.float32)), oracle.linear_fwd(Wt, ad, X), "Y f32")
    ad.scaling = visible_scaling_bwd(Wt, ad, X, dY)
    rdX, rdH, _ = oracle.linear_bwd(Wt, ad, X, dY)
    dX, dH, _ = qb.linear_bwd(dq, adapter_to_dev(ad), Xd, dYd, torch.float32)
    gate_strict(to_np64(dX), rdX, "dX f32")
    gate_strict(to_np64(dH), rdH, "dH", per_row=False)


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("bi,bo", [(8, 8), (4, 8)])
def test_two_dimensional_blocks(qb, path, op, bi, bo):
    T, d_out, d_in, r = 130, 256, 320, 32
    qw, ad, X, dY = make_case(74, T, d_out, d_in, bi, 8, r, op, qfmt=1, bi=bi, bo=bo)
    Wt = oracle.dequantize(qw)
    ad.scaling = visible_scaling_fwd(Wt, ad, X)
    dq, Xd, dYd = qweight_to_dev(qw), to_bf16_dev(X), to_bf16_dev(dY)
    gate_strict(to_np64(qb.linear_fwd(dq, adapter_to_dev(ad), Xd, torch.float32)), oracle.linear_fwd(Wt, ad, X), "Y f32")
    ad.scaling = visible_scaling_bwd(Wt, ad, X, dY)
    rdX, rdA, rdB = oracle.linear_bwd(Wt, ad, X, dY)
    dX, dA, dB = qb.linear_bwd(dq, adapter_to_dev(ad), Xd, dYd, torch.float32)
    gate_strict(to_np64(dX), rdX, "dX f32")
    gate_strict(to_np64(dA), rdA, "dA", per_row=False)
    gate_strict(to_np64(dB), rdB, "dB", per_row=False)


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("case", [(320, 448, 64, 8, 48, 0), (136, 192, 4, 4, 16, 1)])
def test_dense_16bit_merge(qb, op, case):
    d_out, d_in, l1, l2, r, qfmt = case
    qw, ad, X, _ = make_case(75, 96, d_out, d_in, l1, l2, r, op, qfmt=qfmt)
    Wt = oracle.dequantize(qw)
    ad.scaling = visible_scaling_fwd(Wt, ad, X)
    ref = Wt + ad.scaling * oracle.dense_delta_w(d_out, d_in, ad)
    dq, da = qweight_to_dev(qw), adapter_to_dev(ad)
    Wm = qb.merge_dense(dq, da)
    got = to_np64(Wm)
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-30)          # one bf16 rounding
    Y = torch.matmul(to_bf16_dev(X).float(), Wm.float().t())
    gate_strict(to_np64(Y), oracle.linear_fwd(Wt, ad, X), "X W'^T vs adapted forward")


def test_offset_merge_refuses_the_alternative_operators(qb):
    qw, ad, _, _ = make_case(76, 8, 64, 128, 64, 8, 16, oracle.OP_AVGPOOL_REPEAT, qfmt=1)
    dq = qweight_to_dev(qw)
    qb.merge(dq, adapter_to_dev(ad))                        # the method's own pair merges
    for op in OPS:
        ad.scale_op = op
        with pytest.raises(qb.QbloraError) as e:
            qb.merge(dq, adapter_to_dev(ad))
        assert e.value.status == qb.ERR_INVALID_ARG
        with pytest.raises(qb.QbloraError) as e:
            qb.merge_noalloc(dq, adapter_to_dev(ad), torch.empty_like(dq.beta))
        assert e.value.status == qb.ERR_INVALID_ARG
    ad.scale_op = 3
    with pytest.raises(qb.QbloraError) as e:
        qb.linear_fwd(dq, adapter_to_dev(ad), to_bf16_dev(np.zeros((4, 128), np.float32)), torch.float32)
    assert e.value.status == qb.ERR_INVALID_ARG
