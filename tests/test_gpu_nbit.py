"""GPU parity for the N-bit min-max quantizer (Eq. 1 with N < 4): codes, alpha and beta bit for bit
against the CPU oracle, and the quantized weight used through the rest of the library (forward,
backward, offset merge, low-bit product) like any other min-max weight."""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_17029_b200 import synth
from tests._parity import (adapter_to_dev, gate_strict, to_bf16_dev, to_dev, to_np64, visible_scaling)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def qb():
    from paper_2407_17029_b200 import binding
    return binding


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
@pytest.mark.parametrize("shape,bi,bo", [((256, 1024), 64, 1), ((200, 192), 64, 1), ((64, 256), 8, 8), ((1, 64), 64, 1)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_quantize_nbit_bit_exact(qb, bits, shape, bi, bo, dtype):
    W = synth.normal(81, f"nbit/{shape}/{bi}x{bo}", shape, 0.02)
    W[0, :bi] = 0.25                      # a constant block
    if dtype == "bf16":
        W = synth.round_to_bf16(W)
        Wd = to_bf16_dev(W)
    else:
        Wd = to_dev(W)
    ref = oracle.quantize_blockwise(W, bi, bo, oracle.FMT_AFFINE_MINMAX, nbits=bits)
    got = qb.quantize_minmax_nbit(Wd, bits, bi, bo)
    codes = got.codes.cpu().numpy()
    assert np.array_equal(codes, ref.codes)
    top = max(int((codes & 15).max()), int((codes >> 4).max()))
    assert top == ((1 << bits) - 1 if W.size > bi * bo else 0)           # (the single-block case is all constant)
    assert np.array_equal(got.alpha.cpu().numpy().view(np.uint32), ref.alpha.view(np.uint32))
    assert np.array_equal(got.beta.cpu().numpy().view(np.uint32), ref.beta.view(np.uint32))
    if bits == 4:
        same = qb.quantize_blockwise(Wd, bi, bo, qb.FMT_AFFINE_MINMAX)
        assert torch.equal(same.codes, got.codes) and torch.equal(same.alpha, got.alpha) and torch.equal(same.beta, got.beta)


@pytest.mark.parametrize("bits", [2, 3])
def test_nbit_weight_through_the_layer(qb, bits):
    T, d_out, d_in, l1, l2, r = 300, 320, 448, 64, 8, 48
    W = synth.normal(82, "nbit/layer/W", (d_out, d_in), 0.02)
    X, _ = synth.make_activations(82, "nbit/layer/X", T, d_in, 0.0)
    dY = synth.round_to_bf16(synth.normal(82, "nbit/layer/dY", (T, d_out)))
    A = synth.round_to_bf16(synth.normal(82, "nbit/layer/A", (d_in // l1, r), 0.01))
    B = synth.round_to_bf16(synth.normal(82, "nbit/layer/B", (r, d_out // l2), 0.01))
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX, nbits=bits)
    Wt = oracle.dequantize(qw)
    ad = oracle.Adapter(l1, l2, r, 1.0, A, B)
    ad.scaling = visible_scaling(Wt, ad, X)
    dq = qb.quantize_minmax_nbit(to_dev(W), bits)
    da, Xd, dYd = adapter_to_dev(ad), to_bf16_dev(X), to_bf16_dev(dY)
    gate_strict(to_np64(qb.linear_fwd(dq, da, Xd, torch.float32)), oracle.linear_fwd(Wt, ad, X), "Y f32")
    rdX, rdA, rdB = oracle.linear_bwd(Wt, ad, X, dY)
    dX, dA, dB = qb.linear_bwd(dq, da, Xd, dYd, torch.float32)
    gate_strict(to_np64(dX), rdX, "dX f32")
    gate_strict(to_np64(dA), rdA, "dA", per_row=False)
    gate_strict(to_np64(dB), rdB, "dB", per_row=False)
    merged = qb.merge(dq, da)
    assert np.array_equal(merged.beta.cpu().numpy(), oracle.merge(qw, ad).beta)
    # (token counts as in the 4-bit merge-identity test: the merged operand carries the adapter inside the
    # bf16-rounded weight, so with only 7 pooled inputs rows with a small adapter term see a larger relative error)
    for Tl in (1, 16, 40):
        gate_strict(to_np64(qb.lowbit_gemm(merged, Xd[:Tl].contiguous(), torch.float32)),
                    oracle.linear_fwd(Wt, ad, X[:Tl]), f"merged low-bit product T={Tl}")


def test_nbit_rejects_bad_width(qb):
    W = to_dev(synth.normal(83, "nbit/bad", (8, 64), 0.02))
    for bits in (0, 5):
        with pytest.raises(qb.QbloraError) as e:
            qb.quantize_minmax_nbit(W, bits)
        assert e.value.status == qb.ERR_INVALID_ARG


@pytest.mark.parametrize("bits", [2, 4])
def test_quantize_ties_and_near_ties_bit_exact(qb, bits):
    # values on and within a few ulps of the rounding boundaries k + 1/2 of Eq. 1's grid: the library decides
    # these with the exact quotient, everything else without a division; both must agree with the oracle
    qmax = (1 << bits) - 1
    rng = np.random.Generator(np.random.Philox(key=84))
    rows = []
    for trial in range(256):
        alpha = np.float32(0.125) if trial % 4 == 0 else np.float32(rng.uniform(1e-3, 0.3))
        beta = np.float32(0.0) if trial % 4 == 0 else np.float32(rng.normal(0, 0.05))
        k = rng.integers(0, qmax, size=62)
        w = (beta + alpha * (k.astype(np.float32) + np.float32(0.5))).astype(np.float32)
        for step in range(int(rng.integers(0, 4))):                       # 0..3 ulps off the boundary, either way
            w = np.nextafter(w, np.float32(np.inf if trial % 2 else -np.inf))
        row = np.concatenate([[beta, np.float32(beta + alpha * qmax)], w]).astype(np.float32)   # pins min and max
        rows.append(row)
    W = np.stack(rows)
    ref = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX, nbits=bits)
    got = qb.quantize_minmax_nbit(to_dev(W), bits)
    assert np.array_equal(got.alpha.cpu().numpy().view(np.uint32), ref.alpha.view(np.uint32))
    assert np.array_equal(got.beta.cpu().numpy().view(np.uint32), ref.beta.view(np.uint32))
    assert np.array_equal(got.codes.cpu().numpy(), ref.codes)
    # the case is what it claims to be: a good share of the elements sits within 1e-5 of a boundary
    q = (W.astype(np.float64) - ref.beta.astype(np.float64)) / ref.alpha.astype(np.float64)
    assert np.mean(np.abs(q - np.floor(q) - 0.5) < 1e-5) > 0.5


def test_quantize_level_table_near_midpoints_bit_exact(qb):
    # level-table format: elements whose quotient w / absmax sits on or within a few ulps of a midpoint between
    # two levels (decided by the exact quotient in the library), mixed with ordinary ones
    rng = np.random.Generator(np.random.Philox(key=85))
    t = oracle.default_code_table().astype(np.float64)
    mids = ((t[:-1] + t[1:]) / 2).astype(np.float32)
    rows = []
    for trial in range(256):
        a = np.float32(0.5) if trial % 4 == 0 else np.float32(rng.uniform(1e-3, 0.3))
        j = rng.integers(0, 15, size=63)
        w = (a * mids[j]).astype(np.float32)
        for step in range(int(rng.integers(0, 4))):
            w = np.nextafter(w, np.float32(np.inf if trial % 2 else -np.inf))
        sign = np.float32(1.0 if trial % 3 else -1.0)
        rows.append(np.concatenate([[sign * a], w]).astype(np.float32))           # pins absmax
    W = np.stack(rows)
    W[::7, 1:] = synth.normal(85, "lvl/plain", (len(W[::7]), 63), 0.02).clip(-1e-3, 1e-3)
    ref = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_CODEBOOK_ABSMAX)
    got = qb.quantize_blockwise(to_dev(W), 64, 1, qb.FMT_CODEBOOK_ABSMAX)
    assert np.array_equal(got.alpha.cpu().numpy().view(np.uint32), ref.alpha.view(np.uint32))
    assert np.array_equal(got.codes.cpu().numpy(), ref.codes)
    v = W.astype(np.float64) / ref.alpha.astype(np.float64)
    near = np.abs(v[..., None] - mids.astype(np.float64)).min(axis=-1) < 1e-6
    assert near.mean() > 0.5


# ------------------------------------------------------------------------ dense 2- / 3-bit storage
@pytest.mark.parametrize("bits", [2, 3])
@pytest.mark.parametrize("shape", [(200, 192), (64, 1024), (1, 32)])
def test_pack_codes_bit_exact_and_round_trip(qb, bits, shape):
    from tests._parity import Guarded
    d_out, d_in = shape
    rng = np.random.default_rng(11)
    c = rng.integers(0, 1 << bits, size=(d_out, d_in), dtype=np.uint8)
    nib = (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
    ref = oracle.pack_codes(nib, d_in, bits)
    alpha = torch.ones((d_out, max(d_in // 32, 1)), device="cuda:0")
    qw = qb.QWeight(d_out, d_in, 32, 1, qb.FMT_AFFINE_MINMAX, [0.0] * 16, to_dev(nib), alpha, alpha.clone())
    packed = qb.pack_codes(qw, bits)
    assert packed.code_bits == bits and tuple(packed.codes.shape) == (d_out, d_in * bits // 8)
    assert np.array_equal(packed.codes.cpu().numpy(), ref)
    assert torch.equal(qb.unpack_codes(packed).codes, qw.codes)
    # outputs between guard bands (the kernels work on 32-code units)
    g = Guarded()
    out = g.alloc((d_out, d_in * bits // 8), torch.uint8)
    ws = g.alloc((256,), torch.uint8)
    assert qb._lib.qblora_pack_codes(qw.codes.data_ptr(), d_out, d_in, bits, out.data_ptr(), ws.data_ptr(), 256, None) == qb.OK
    g.check("pack_codes")
    assert torch.equal(out, packed.codes)
    # a code that needs more than `bits` bits is reported through the status word
    bad = qw.codes.clone()
    bad[0, 0] = 0x0F
    qbad = qb.QWeight(d_out, d_in, 32, 1, qb.FMT_AFFINE_MINMAX, [0.0] * 16, bad, alpha, alpha.clone())
    with pytest.raises(qb.QbloraError) as e:
        qb.pack_codes(qbad, bits)
    assert e.value.status == qb.ERR_INVALID_ARG


@pytest.mark.parametrize("bits", [2, 3])
def test_densely_stored_weight_through_every_call(qb, bits):
    # the same 2- / 3-bit weight stored one code per nibble and densely: every call that reads the codes gives the
    # same result bit for bit (the dense codes are expanded inside the workspace), and that result matches the oracle
    # computed from the oracle's own pack / unpack of the oracle's quantization
    from tests._parity import g_linear_bwd, g_linear_fwd, g_lowbit_gemm
    T, d_out, d_in, l1, l2, r = 300, 320, 512, 64, 8, 48
    W = synth.normal(83, "nbit/dense/W", (d_out, d_in), 0.02)
    X, _ = synth.make_activations(83, "nbit/dense/X", T, d_in, 0.0)
    dY = synth.round_to_bf16(synth.normal(83, "nbit/dense/dY", (T, d_out)))
    A = synth.round_to_bf16(synth.normal(83, "nbit/dense/A", (d_in // l1, r), 0.01))
    B = synth.round_to_bf16(synth.normal(83, "nbit/dense/B", (r, d_out // l2), 0.01))
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX, nbits=bits)
    qw.codes = oracle.unpack_codes(oracle.pack_codes(qw.codes, d_in, bits), d_in, bits)
    Wt = oracle.dequantize(qw)
    ad = oracle.Adapter(l1, l2, r, 1.0, A, B)
    ad.scaling = visible_scaling(Wt, ad, X)
    nib = qb.quantize_minmax_nbit(to_dev(W), bits)
    dense = qb.pack_codes(nib, bits)
    assert dense.codes.numel() * 8 == d_out * d_in * bits
    assert qb.workspace_bytes(qb.OP_LINEAR_FWD, dense, None, T) >= qb.workspace_bytes(qb.OP_LINEAR_FWD, nib, None, T) + d_out * d_in // 2
    da, Xd, dYd = adapter_to_dev(ad), to_bf16_dev(X), to_bf16_dev(dY)
    Y = g_linear_fwd(dense, da, Xd, torch.float32)
    assert torch.equal(Y, qb.linear_fwd(nib, da, Xd, torch.float32))
    gate_strict(to_np64(Y), oracle.linear_fwd(Wt, ad, X), "Y from dense codes")
    dX, dA, dB = g_linear_bwd(dense, da, Xd, dYd, torch.float32)
    nX, nA, nB = qb.linear_bwd(nib, da, Xd, dYd, torch.float32)
    assert torch.equal(dX, nX) and torch.equal(dA, nA) and torch.equal(dB, nB)
    gate_strict(to_np64(dX), oracle.linear_bwd(Wt, ad, X, dY)[0], "dX from dense codes")
    # offset merge keeps the dense codes; the merged dense weight serves the low-bit product at every token count
    merged = qb.merge(dense, da)
    assert merged.code_bits == bits and merged.codes.data_ptr() == dense.codes.data_ptr()
    assert np.array_equal(merged.beta.cpu().numpy().view(np.uint32), oracle.merge(qw, ad).beta.view(np.uint32))
    unmerged = oracle.linear_fwd(Wt, ad, X)
    for Tn in (1, 5, 16, T):
        Yl = g_lowbit_gemm(merged, Xd[:Tn].contiguous(), torch.float32)
        gate_strict(to_np64(Yl), unmerged[:Tn], f"low-bit product from dense codes, T={Tn}")
    # dense 16-bit merge
    Wm = qb.merge_dense(dense, da)
    assert torch.equal(Wm, qb.merge_dense(nib, da))
