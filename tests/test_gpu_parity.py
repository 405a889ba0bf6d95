"""GPU parity: every entry point of the C-ABI library against the fp64 CPU oracle, element by
element, on seeded inputs that span several tiles and ragged tails, plus edge cases."""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_17029_b200 import synth
from tests._parity import (DEV, Guarded, adapter_to_dev, g_linear_bwd, g_linear_fwd, g_lowbit_gemm, g_quantize, gate_bf16,
                           gate_strict, qweight_to_dev, rms, to_bf16_dev, to_dev, to_np64, visible_scaling)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def qb():
    from paper_2407_17029_b200 import binding
    return binding


@pytest.fixture(params=["tensor-core", "general"])
def path(request, monkeypatch):
    """Runs a test once on the tcgen05 path and once with the CUDA-core path forced."""
    if request.param == "general":
        monkeypatch.setenv("QBLORA_FORCE_GENERAL", "1")
    else:
        monkeypatch.delenv("QBLORA_FORCE_GENERAL", raising=False)
    return request.param


# ------------------------------------------------------------------------------------- quantizer
@pytest.mark.parametrize("qfmt", [0, 1])
@pytest.mark.parametrize("shape,bi,bo", [((256, 1024), 64, 1), ((200, 192), 64, 1), ((64, 256), 32, 1),
                                         ((64, 256), 8, 8), ((64, 256), 4, 8), ((1, 64), 64, 1)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_quantize_bit_exact(qb, qfmt, shape, bi, bo, dtype):
    W = synth.normal(31, f"qz/{shape}/{bi}x{bo}", shape, 0.02)
    W[0, :bi] = 0.0                       # a degenerate (all-zero / constant) block
    if dtype == "bf16":
        W = synth.round_to_bf16(W)
        Wd = to_bf16_dev(W)
    else:
        Wd = to_dev(W)
    ref = oracle.quantize_blockwise(W, bi, bo, qfmt)
    got = g_quantize(Wd, bi, bo, qfmt)              # outputs between guard bands
    assert np.array_equal(got.codes.cpu().numpy(), ref.codes)
    assert np.array_equal(got.alpha.cpu().numpy().view(np.uint32), ref.alpha.view(np.uint32))
    if qfmt == 1:
        assert np.array_equal(got.beta.cpu().numpy().view(np.uint32), ref.beta.view(np.uint32))
    else:
        assert got.beta is None


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_quantize_signed_zero_block_minimum(qb, dtype):
    # blocks whose minimum is a zero, with zeros of both signs in every order (within a lane's eight elements,
    # across lanes, across the halves of the block): beta comes out as +0 bit for bit, as in the oracle; also a
    # block of zeros of mixed sign only, and both formats' codes for the signed zeros.
    W = np.abs(synth.normal(34, "qz/pm0", (16, 256), 0.02)).astype(np.float32)
    pz, nz = np.float32(0.0), np.float32(-0.0)
    W[0, 0], W[0, 1] = pz, nz
    W[1, 0], W[1, 1] = nz, pz
    W[2, 3], W[2, 40] = pz, nz
    W[3, 3], W[3, 40] = nz, pz
    W[4, 64 + 63], W[4, 64] = nz, pz
    W[5, 128:192] = pz; W[5, 128:192:2] = nz
    W[6, 192:256] = nz
    W[7, 7] = nz
    if dtype == "bf16":
        W = synth.round_to_bf16(W)
        Wd = to_bf16_dev(W)
    else:
        Wd = to_dev(W)
    for qfmt in (0, 1):
        ref = oracle.quantize_blockwise(W, 64, 1, qfmt)
        got = qb.quantize_blockwise(Wd, 64, 1, qfmt)
        assert np.array_equal(got.codes.cpu().numpy(), ref.codes)
        assert np.array_equal(got.alpha.cpu().numpy().view(np.uint32), ref.alpha.view(np.uint32))
        if qfmt == 1:
            gb = got.beta.cpu().numpy().view(np.uint32)
            assert np.array_equal(gb, ref.beta.view(np.uint32))
            assert gb[0, 0] == 0 and gb[1, 0] == 0 and gb[5, 2] == 0 and gb[6, 3] == 0 and gb[7, 0] == 0
    # the general (any block shape) kernel takes the same decision
    ref = oracle.quantize_blockwise(W, 8, 8, 1)
    got = qb.quantize_blockwise(Wd, 8, 8, 1)
    assert np.array_equal(got.beta.cpu().numpy().view(np.uint32), ref.beta.view(np.uint32))
    assert np.array_equal(got.codes.cpu().numpy(), ref.codes)


@pytest.mark.parametrize("qfmt", [0, 1])
def test_quantize_non_finite_weights_stay_inside_their_block(qb, qfmt):
    # NaN / Inf weights are outside the method (Eq. 1 has no value for them): the call must neither fault nor let them
    # leak -- every block that holds only finite weights still comes out bit for bit as in the oracle, and every code of
    # a poisoned block is a valid 4-bit code.
    W = synth.normal(36, "qz/nonfinite", (32, 512), 0.02)
    clean = W.copy()
    W[3, 70] = np.nan
    W[5, 128] = np.inf
    W[5, 129] = -np.inf
    W[9, 0] = np.inf
    got = g_quantize(to_dev(W), 64, 1, qfmt)
    ref = oracle.quantize_blockwise(clean, 64, 1, qfmt)
    codes, alpha = got.codes.cpu().numpy(), got.alpha.cpu().numpy()
    poisoned = {(3, 1), (5, 2), (9, 0)}
    for o in range(32):
        for b in range(8):
            if (o, b) in poisoned:
                continue
            assert np.array_equal(codes[o, 32 * b:32 * b + 32], ref.codes[o, 32 * b:32 * b + 32])
            assert alpha[o, b].view(np.uint32) == ref.alpha[o, b].view(np.uint32)
            if qfmt == 1:
                assert got.beta.cpu().numpy()[o, b].view(np.uint32) == ref.beta[o, b].view(np.uint32)
    torch.cuda.synchronize()


def test_quantize_round_trip_on_device(qb):
    # Q(D(Q(W))) == Q(W) on the level-table format, dequantizing with the oracle in between
    W = synth.normal(32, "qz/rt", (128, 512), 0.02)
    q1 = qb.quantize_blockwise(to_dev(W), 64, 1, 0)
    o1 = oracle.QWeight(128, 512, 64, 1, 0, np.array(q1.code, np.float32), q1.codes.cpu().numpy(),
                        q1.alpha.cpu().numpy(), None)
    W1 = oracle.dequantize(o1).astype(np.float32)
    q2 = qb.quantize_blockwise(to_dev(W1), 64, 1, 0)
    assert torch.equal(q1.codes, q2.codes) and torch.equal(q1.alpha, q2.alpha)


def test_quantize_custom_table(qb):
    table = np.linspace(-1.0, 1.0, 16).astype(np.float32)
    W = synth.normal(33, "qz/custom", (32, 128), 0.5)
    ref = oracle.quantize_blockwise(W, 64, 1, 0, table)
    got = qb.quantize_blockwise(to_dev(W), 64, 1, 0, [float(x) for x in table])
    assert np.array_equal(got.codes.cpu().numpy(), ref.codes)


def test_quantize_level_table_midpoints_on_bucket_edges_and_tight_tables(qb):
    # The level-table quantizer finds a code through a table of 128 equal buckets over [-1, 1).  (a) A level table whose
    # midpoints are multiples of 1/16 puts every midpoint exactly on a bucket edge; the block holds the midpoints
    # themselves, their neighbours up to three ulps away and values a few 1e-7 .. 1e-5 beside them, at absmax 1 (the
    # scaled value is the weight itself) and at an absmax that makes every quotient inexact.  (b) A table with two levels
    # 0.002 apart cannot use the buckets and takes the search.  Codes and alpha equal the oracle's bit for bit.
    table = np.array([-1, -0.875, -0.75, -0.625, -0.5, -0.375, -0.25, -0.125, 0, 0.125, 0.25, 0.375, 0.5, 0.625, 0.75, 1.0],
                     dtype=np.float32)
    mids = ((table[:-1].astype(np.float64) + table[1:].astype(np.float64)) / 2).astype(np.float32)
    vals = [mids]
    for k in (1, 2, 3):
        up, dn = mids.copy(), mids.copy()
        for _ in range(k):
            up, dn = np.nextafter(up, np.float32(2)), np.nextafter(dn, np.float32(-2))
        vals += [up, dn]
    for off in (3e-7, 9e-7, 1.1e-6, 3e-6, 5e-6, 1e-5):
        vals += [(mids + np.float32(off)).astype(np.float32), (mids - np.float32(off)).astype(np.float32)]
    vals = np.concatenate(vals)                       # 19 x 15 = 285 values
    rows = []
    for scale in (1.0, 0.3, 1.7e-3):
        v = (vals * np.float32(scale)).astype(np.float32)
        v = np.concatenate([v, np.zeros((-len(v)) % 63, np.float32)]).reshape(-1, 63)
        blk = np.concatenate([np.full((v.shape[0], 1), scale, np.float32), v], axis=1)     # absmax element first
        rows.append(blk.reshape(1, -1))
    W = np.concatenate(rows, axis=0)
    assert W.shape[1] % 64 == 0
    ref = oracle.quantize_blockwise(W, 64, 1, 0, table)
    got = g_quantize(to_dev(W), 64, 1, 0, [float(x) for x in table])
    assert np.array_equal(got.codes.cpu().numpy(), ref.codes)
    assert np.array_equal(got.alpha.cpu().numpy().view(np.uint32), ref.alpha.view(np.uint32))
    tight = np.linspace(-1.0, 1.0, 16).astype(np.float32)
    tight[8] = tight[7] + np.float32(0.002)
    Wr = synth.normal(35, "qz/tight", (64, 512), 0.5)
    ref = oracle.quantize_blockwise(Wr, 64, 1, 0, tight)
    got = g_quantize(to_dev(Wr), 64, 1, 0, [float(x) for x in tight])
    assert np.array_equal(got.codes.cpu().numpy(), ref.codes)


# --------------------------------------------------------------------------- forward / backward
def make_case(seed, T, d_out, d_in, l1, l2, r, qfmt=0, ab_std=0.01, bi=64, bo=1, outliers=0.0):
    tag = f"case/{seed}"
    W = synth.normal(seed, tag + "/W", (d_out, d_in), 0.02)
    X, _ = synth.make_activations(seed, tag + "/X", T, d_in, outliers)
    dY = synth.round_to_bf16(synth.normal(seed, tag + "/dY", (T, d_out)))
    A = synth.round_to_bf16(synth.normal(seed, tag + "/A", (d_in // l1, r), ab_std))
    B = synth.round_to_bf16(synth.normal(seed, tag + "/B", (r, d_out // l2), ab_std))
    qw = oracle.quantize_blockwise(W, bi, bo, qfmt)
    ad = oracle.Adapter(l1, l2, r, 1.0, A, B)
    return qw, ad, X, dY


CASES = [
    # T, d_out, d_in, l1, l2, r  -- several 128-tiles with ragged tails in every dimension
    (300, 320, 448, 64, 8, 48),
    (300, 320, 448, 4, 4, 48),
    (77, 136, 192, 1, 1, 16),
    (515, 256, 640, 64, 8, 64),
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("qfmt", [0, 1])
@pytest.mark.parametrize("visible", [False, True])
def test_linear_fwd_parity(qb, path, case, qfmt, visible):
    T, d_out, d_in, l1, l2, r = case
    qw, ad, X, _ = make_case(41, T, d_out, d_in, l1, l2, r, qfmt)
    Wt = oracle.dequantize(qw)
    if visible:
        ad.scaling = visible_scaling(Wt, ad, X)
    ref = oracle.linear_fwd(Wt, ad, X)
    dq, da, Xd = qweight_to_dev(qw), adapter_to_dev(ad), to_bf16_dev(X)
    gate_strict(to_np64(g_linear_fwd(dq, da, Xd, torch.float32)), ref, "Y f32")         # guarded: outputs and workspace
    gate_bf16(to_np64(g_linear_fwd(dq, da, Xd, torch.bfloat16)), ref, "Y bf16")          # sit between guard bands
    if visible:
        base = oracle.linear_fwd(Wt, None, X)
        assert rms(ref - base) > 0.5 * rms(base)          # the adapter really is half of the output


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("qfmt", [0, 1])
@pytest.mark.parametrize("visible", [False, True])
def test_linear_bwd_parity(qb, path, case, qfmt, visible):
    T, d_out, d_in, l1, l2, r = case
    qw, ad, X, dY = make_case(42, T, d_out, d_in, l1, l2, r, qfmt)
    Wt = oracle.dequantize(qw)
    if visible:
        ad.scaling = visible_scaling(Wt, ad, X)
    rdX, rdA, rdB = oracle.linear_bwd(Wt, ad, X, dY)
    dq, da, Xd, dYd = qweight_to_dev(qw), adapter_to_dev(ad), to_bf16_dev(X), to_bf16_dev(dY)
    dX, dA, dB = g_linear_bwd(dq, da, Xd, dYd, torch.float32)
    gate_strict(to_np64(dX), rdX, "dX f32")
    gate_strict(to_np64(dA), rdA, "dA", per_row=False)
    gate_strict(to_np64(dB), rdB, "dB", per_row=False)
    dXb, _, _ = g_linear_bwd(dq, da, Xd, dYd, torch.bfloat16, need_da=False, need_db=False)
    gate_bf16(to_np64(dXb), rdX, "dX bf16")
    # skipping outputs leaves the others unchanged (bit for bit: the library is deterministic)
    _, dA2, dB2 = qb.linear_bwd(dq, da, Xd, dYd, need_dx=False)
    assert torch.equal(dA, dA2) and torch.equal(dB, dB2)


@pytest.mark.parametrize("d_out,d_in,T", [(4864, 128, 2100), (128, 4864, 2100), (4864, 128, 2400)])
def test_wide_tiles_several_rounds_and_ragged_tokens(qb, d_out, d_in, T):
    # 19 row tiles x 5 token positions of 512 = 95 tiles on 74 CTA pairs (two rounds); T = 2100 leaves 52 tokens
    # in the last position, so its tiles have an empty second half; T = 2400 leaves 352, a second half with 96
    # tokens.  (4864, 128) lays the forward's rows out this way, (128, 4864) the backward's.
    qw, ad, X, dY = make_case(47, T, d_out, d_in, 64, 8, 16, 1)
    Wt = oracle.dequantize(qw)
    dq, da, Xd, dYd = qweight_to_dev(qw), adapter_to_dev(ad), to_bf16_dev(X), to_bf16_dev(dY)
    gate_strict(to_np64(g_linear_fwd(dq, da, Xd, torch.float32)), oracle.linear_fwd(Wt, ad, X), "Y f32")
    rdX, rdA, rdB = oracle.linear_bwd(Wt, ad, X, dY)
    dX, dA, dB = g_linear_bwd(dq, da, Xd, dYd, torch.float32)
    gate_strict(to_np64(dX), rdX, "dX f32")
    gate_strict(to_np64(dA), rdA, "dA", per_row=False)
    gate_strict(to_np64(dB), rdB, "dB", per_row=False)


def test_zero_B_is_bit_identical_to_no_adapter(qb, path):
    qw, ad, X, dY = make_case(43, 300, 320, 448, 64, 8, 48)
    ad.B = np.zeros_like(ad.B)
    dq, da, Xd, dYd = qweight_to_dev(qw), adapter_to_dev(ad), to_bf16_dev(X), to_bf16_dev(dY)
    for dt in (torch.float32, torch.bfloat16):
        assert torch.equal(qb.linear_fwd(dq, da, Xd, dt), qb.linear_fwd(dq, None, Xd, dt))
    ref = oracle.linear_fwd(oracle.dequantize(qw), None, X)
    gate_strict(to_np64(qb.linear_fwd(dq, None, Xd, torch.float32)), ref, "base only")
    dX0, _, _ = qb.linear_bwd(dq, None, None, dYd, torch.float32)
    gate_strict(to_np64(dX0), oracle.linear_bwd(oracle.dequantize(qw), None, X, dY)[0], "dX base only")


def test_outlier_channels_and_general_block_shapes(qb):
    # 1% input channels x20 (the MLP config's activation recipe) and a 2-D quantization block
    qw, ad, X, dY = make_case(44, 200, 128, 512, 8, 8, 32, qfmt=1, bi=8, bo=8, outliers=0.01)
    Wt = oracle.dequantize(qw)
    ad.scaling = visible_scaling(Wt, ad, X)
    dq, da, Xd, dYd = qweight_to_dev(qw), adapter_to_dev(ad), to_bf16_dev(X), to_bf16_dev(dY)
    gate_strict(to_np64(qb.linear_fwd(dq, da, Xd, torch.float32)), oracle.linear_fwd(Wt, ad, X), "Y 2-D blocks")
    dX, dA, dB = qb.linear_bwd(dq, da, Xd, dYd, torch.float32)
    r = oracle.linear_bwd(Wt, ad, X, dY)
    gate_strict(to_np64(dX), r[0], "dX"); gate_strict(to_np64(dA), r[1], "dA", per_row=False); gate_strict(to_np64(dB), r[2], "dB", per_row=False)


def test_single_token_and_workspace_errors(qb):
    qw, ad, X, dY = make_case(45, 1, 128, 128, 64, 8, 16)
    Wt = oracle.dequantize(qw)
    dq, da, Xd = qweight_to_dev(qw), adapter_to_dev(ad), to_bf16_dev(X)
    gate_strict(to_np64(qb.linear_fwd(dq, da, Xd, torch.float32)), oracle.linear_fwd(Wt, ad, X), "T=1")
    small = torch.empty(16, dtype=torch.uint8, device=DEV)
    with pytest.raises(qb.QbloraError) as e:
        qb.linear_fwd(dq, da, Xd, ws=small)
    assert e.value.status == qb.ERR_WORKSPACE
    ws = qb.alloc_workspace(qb.OP_LINEAR_FWD, dq, da, 1)
    qb.linear_fwd(dq, da, Xd, ws=ws)
    assert qb.device_status(ws) == qb.OK


# ------------------------------------------------------------------------- merge + low-bit product
@pytest.mark.parametrize("single", [False, True])
@pytest.mark.parametrize("scaling", [1.0, 37.5, "visible"])
def test_merge_bit_exact_and_identity(qb, path, single, scaling):
    # 333 token rows (three token tiles with a ragged tail), every row gated.  With P = 7 pooled inputs the
    # adapter term varies strongly from token to token, so rows where it happens to be small are measured against
    # a small row RMS: the low-bit product has to keep the merged shift out of its bf16-rounded operand to pass.
    d_out, d_in, r = 320, 448, 48
    qw, ad, X, _ = make_case(51, 333, d_out, d_in, 64, 8, r, qfmt=1, ab_std=0.02)
    if single:
        ad = oracle.Adapter(64, 8, 0, scaling, synth.round_to_bf16(synth.normal(51, "H", (d_in // 64, d_out // 8), 0.02)), None)
    ad.scaling = visible_scaling(oracle.dequantize(qw), ad, X) if scaling == "visible" else scaling
    ref = oracle.merge(qw, ad)
    dq, da = qweight_to_dev(qw), adapter_to_dev(ad)
    codes0, alpha0 = dq.codes.clone(), dq.alpha.clone()
    g = Guarded()
    got = qb.merge(dq, da, ws=g.workspace(qb.OP_MERGE, dq, da, 0), beta_out=g.alloc(tuple(dq.beta.shape), torch.float32))
    g.check("merge")
    assert np.array_equal(got.beta.cpu().numpy().view(np.uint32), ref.beta.view(np.uint32))
    assert torch.equal(dq.codes, codes0) and torch.equal(dq.alpha, alpha0)          # untouched
    assert got.codes.data_ptr() == dq.codes.data_ptr()
    # merge identity: low-bit product on the merged weight == unmerged adapted forward
    Xd = to_bf16_dev(X)
    unmerged = oracle.linear_fwd(oracle.dequantize(qw), ad, X)
    gate_strict(to_np64(qb.lowbit_gemm(got, Xd, torch.float32)), unmerged, "merged low-bit vs unmerged fwd")
    gate_bf16(to_np64(qb.lowbit_gemm(got, Xd, torch.bfloat16)), unmerged, "merged low-bit vs unmerged fwd, bf16")
    for T in (1, 7, 16):      # the decode kernels on the same merged weight
        gate_strict(to_np64(qb.lowbit_gemm(got, Xd[:T].contiguous(), torch.float32)), unmerged[:T], f"merged decode T={T}")
    if not single:
        gate_strict(to_np64(qb.linear_fwd(dq, da, Xd, torch.float32)), unmerged, "unmerged fwd")
    # in place
    got2 = qb.merge(dq, da, in_place=True)
    assert got2.beta.data_ptr() == dq.beta.data_ptr() and torch.equal(got2.beta, got.beta)


def test_merge_rejects_misaligned_geometry(qb):
    qw, ad, _, _ = make_case(52, 4, 128, 128, 4, 4, 16, qfmt=1)
    with pytest.raises(qb.QbloraError) as e:
        qb.merge(qweight_to_dev(qw), adapter_to_dev(ad))
    assert e.value.status == qb.ERR_INVALID_ARG


@pytest.mark.parametrize("T", [1, 2, 3, 8, 16, 17, 150])
def test_lowbit_gemm_parity(qb, path, T):
    qw, _, X, _ = make_case(53, T, 328, 448, 64, 8, 16, qfmt=1)
    ref = oracle.lowbit_gemm(qw, X)
    dq, Xd = qweight_to_dev(qw), to_bf16_dev(X)
    gate_strict(to_np64(g_lowbit_gemm(dq, Xd, torch.float32)), ref, f"lowbit T={T} f32")
    gate_bf16(to_np64(g_lowbit_gemm(dq, Xd, torch.bfloat16)), ref, f"lowbit T={T} bf16")


@pytest.mark.parametrize("T", [1, 3, 16])
@pytest.mark.parametrize("log2_gain", [-40, 0, 22])
def test_lowbit_decode_token_range(qb, T, log2_gain):
    # The small-T path holds x in fp16 after a power-of-two prescale: tokens far above fp16's
    # largest value and far below its smallest normal must come out as exactly as ordinary ones.
    # One token carries a single huge outlier so that most of its elements sit 2^17 below its maximum.
    qw, _, X, _ = make_case(57, T, 328, 448, 64, 8, 16, qfmt=1)
    X = X.copy()
    X[0, 5] *= np.float32(2.0 ** 17)
    X = synth.round_to_bf16(X * np.float32(2.0 ** log2_gain))
    ref = oracle.lowbit_gemm(qw, X)
    dq, Xd = qweight_to_dev(qw), to_bf16_dev(X)
    gate_strict(to_np64(qb.lowbit_gemm(dq, Xd, torch.float32)), ref, f"lowbit range T={T} gain=2^{log2_gain}")


@pytest.mark.parametrize("T", [1, 5])
def test_lowbit_decode_wide_input(qb, T):
    # 896 groups per row: the one-token kernel's resident token fragments no longer fit beside its tile
    # ring, so T = 1 takes the kernel that streams them (the one T = 5 uses anyway); 72 rows = two
    # full row blocks and a ragged one.
    qw, _, X, _ = make_case(58, T, 72, 896 * 64, 64, 8, 16, qfmt=1)
    ref = oracle.lowbit_gemm(qw, X)
    dq, Xd = qweight_to_dev(qw), to_bf16_dev(X)
    gate_strict(to_np64(g_lowbit_gemm(dq, Xd, torch.float32)), ref, f"lowbit wide T={T}")


@pytest.mark.parametrize("case", [(300, 320, 448, 64, 8), (150, 128, 512, 8, 8), (77, 136, 192, 4, 4)])
@pytest.mark.parametrize("visible", [False, True])
def test_single_matrix_adapter_fwd_bwd(qb, path, case, visible):
    # Sec. 3.3's single matrix H [P][Q] (B == NULL) trained directly: forward s * repeat(x' H),
    # backward dH = x'^T dv (returned in dA) and dX with the pooled-input gradient dv H^T.
    T, d_out, d_in, l1, l2 = case
    qw, _, X, dY = make_case(61, T, d_out, d_in, l1, l2, 16, qfmt=1)
    H = synth.round_to_bf16(synth.normal(61, "H", (d_in // l1, d_out // l2), 0.02))
    ad = oracle.Adapter(l1, l2, 0, 1.0, H, None)
    Wt = oracle.dequantize(qw)
    if visible:
        ad.scaling = visible_scaling(Wt, ad, X)
    dq, da, Xd, dYd = qweight_to_dev(qw), adapter_to_dev(ad), to_bf16_dev(X), to_bf16_dev(dY)
    gate_strict(to_np64(g_linear_fwd(dq, da, Xd, torch.float32)), oracle.linear_fwd(Wt, ad, X), "Y single matrix")
    gate_bf16(to_np64(qb.linear_fwd(dq, da, Xd, torch.bfloat16)), oracle.linear_fwd(Wt, ad, X), "Y single matrix bf16")
    rdX, rdH, rdB = oracle.linear_bwd(Wt, ad, X, dY)
    assert rdB is None
    dX, dH, dB = g_linear_bwd(dq, da, Xd, dYd, torch.float32)
    assert dB is None and tuple(dH.shape) == H.shape
    gate_strict(to_np64(dX), rdX, "dX single matrix")
    gate_strict(to_np64(dH), rdH, "dH", per_row=False)


@pytest.mark.parametrize("d_out", [72, 4768])
def test_lowbit_one_token_split_tail(qb, d_out):
    # One token, few row blocks against the CTA count: the row blocks left after the whole rounds are cut
    # along K and summed across CTAs (3 row blocks x 4 parts; 149 row blocks = one whole round + 1 x 4).
    qw, _, X, _ = make_case(59, 1, d_out, 64 * 256, 64, 8, 16, qfmt=1)      # 16 K tiles
    ref = oracle.lowbit_gemm(qw, X)
    dq, Xd = qweight_to_dev(qw), to_bf16_dev(X)
    for _ in range(3):      # flags carry a per-launch epoch: repeated launches on one workspace
        ws = qb.alloc_workspace(qb.OP_LOWBIT_GEMM, dq, None, 1)
        for _ in range(2):
            gate_strict(to_np64(qb.lowbit_gemm(dq, Xd, torch.float32, ws=ws)), ref, f"lowbit split tail d_out={d_out}")
            assert qb.device_status(ws) == qb.OK


@pytest.mark.parametrize("T", [1, 2, 16])
@pytest.mark.parametrize("d_out,d_in", [(8, 256), (40, 512), (33 * 8, 256)])
def test_lowbit_decode_tiny_shapes(qb, T, d_out, d_in):
    # fewer output rows than one 32-row tile, a single K tile with unused groups, ragged row blocks
    qw, _, X, _ = make_case(62, T, d_out, d_in, 64, 8, 8, qfmt=1)
    ref = oracle.lowbit_gemm(qw, X)
    dq, Xd = qweight_to_dev(qw), to_bf16_dev(X)
    gate_strict(to_np64(g_lowbit_gemm(dq, Xd, torch.float32)), ref, f"lowbit tiny {d_out}x{d_in} T={T}")


@pytest.mark.parametrize("bi,bo", [(8, 8), (4, 8), (8, 1), (4, 2)])
@pytest.mark.parametrize("visible", [False, True])
def test_two_dimensional_blocks_fwd_bwd(qb, path, bi, bo, visible):
    # Sec. 3.3's native quantization blocks (lambda_1 x lambda_2 = 8 x 8, 4 x 8) in the min-max format, adapter
    # windows equal to the block (so the adapter stays mergeable); several tiles, ragged in every dimension.
    T, d_out, d_in = 300, 328, 448
    qw, ad, X, dY = make_case(63, T, d_out, d_in, bi, 8, 24, qfmt=1, bi=bi, bo=bo)
    Wt = oracle.dequantize(qw)
    if visible:
        ad.scaling = visible_scaling(Wt, ad, X)
    dq, da, Xd, dYd = qweight_to_dev(qw), adapter_to_dev(ad), to_bf16_dev(X), to_bf16_dev(dY)
    gate_strict(to_np64(g_linear_fwd(dq, da, Xd, torch.float32)), oracle.linear_fwd(Wt, ad, X), f"Y blocks {bi}x{bo}")
    rdX, rdA, rdB = oracle.linear_bwd(Wt, ad, X, dY)
    dX, dA, dB = g_linear_bwd(dq, da, Xd, dYd, torch.float32)
    gate_strict(to_np64(dX), rdX, f"dX blocks {bi}x{bo}")
    gate_strict(to_np64(dA), rdA, "dA", per_row=False)
    gate_strict(to_np64(dB), rdB, "dB", per_row=False)
    # prefill-shaped low-bit product on the merged weight equals the unmerged forward (merge identity)
    if 8 % bo == 0:
        merged = qb.merge(dq, da)
        gate_strict(to_np64(qb.lowbit_gemm(merged, Xd, torch.float32)), oracle.linear_fwd(Wt, ad, X), f"merged blocks {bi}x{bo}")


@pytest.mark.parametrize("case", [(320, 448, 64, 8, 48, 0, 64, 1), (136, 192, 4, 4, 16, 1, 64, 1), (128, 512, 8, 8, 0, 1, 8, 8)])
def test_dense_16bit_merge(qb, case):
    # W' = dequantized weight + s * dense adapter update (Sec. 3.1 / 3.2), rounded once to bf16; rank 0 = single
    # matrix H.  Then "zero inference overhead": X W'^T equals the adapted forward.
    d_out, d_in, l1, l2, r, qfmt, bi, bo = case
    qw, ad, X, _ = make_case(64, 96, d_out, d_in, l1, l2, max(r, 8), qfmt=qfmt, bi=bi, bo=bo)
    if r == 0:
        ad = oracle.Adapter(l1, l2, 0, 1.0, synth.round_to_bf16(synth.normal(64, "H", (d_in // l1, d_out // l2), 0.02)), None)
    Wt = oracle.dequantize(qw)
    ad.scaling = visible_scaling(Wt, ad, X)
    ref = Wt + ad.scaling * oracle.dense_delta_w(d_out, d_in, ad)
    dq, da = qweight_to_dev(qw), adapter_to_dev(ad)
    g = Guarded()
    Wg = g.alloc((d_out, d_in), torch.bfloat16)
    qb.merge_dense(dq, da, out=Wg, ws=g.workspace(qb.OP_MERGE_DENSE, dq, da, 0))
    g.check("merge_dense")
    got = to_np64(Wg)
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-30)          # one bf16 rounding
    base = to_np64(qb.merge_dense(dq, None))
    assert np.all(np.abs(base - Wt) <= 2.0 ** -8 * np.abs(Wt) + 1e-30)
    # served by the library's own bf16 GEMM, outputs and workspace between guard bands
    g = Guarded()
    Y = g.alloc((X.shape[0], d_out), torch.float32)
    qb.dense_gemm(Wg, to_bf16_dev(X), ws=g.alloc((256,), torch.uint8), out=Y)
    g.check("dense_gemm")
    gate_strict(to_np64(Y), oracle.linear_fwd(Wt, ad, X), "X W'^T vs adapted forward")


@pytest.mark.parametrize("shape", [(300, 320, 448, 64, 8, 48), (2048, 1024, 1024, 64, 8, 64), (515, 256, 640, 4, 4, 64)])
def test_back_to_back_calls_through_one_workspace_do_not_see_stale_adapter_inputs(qb, shape):
    # The fused contraction starts before the small adapter products in front of it have finished and waits for
    # them only where it needs their result.  Alternate two different inputs through ONE workspace, back to back
    # with no host synchronisation in between: a contraction that read the compressed adapter activation too
    # early would pick up the other input's values.  Every result must equal, bit for bit, the one computed alone.
    T, d_out, d_in, l1, l2, r = shape
    qw, ad, X0, dY0 = make_case(91, T, d_out, d_in, l1, l2, r)
    _, _, X1, dY1 = make_case(92, T, d_out, d_in, l1, l2, r)
    ad.scaling = 30.0                                     # the adapter term is a large part of every output
    dq, da = qweight_to_dev(qw), adapter_to_dev(ad)
    Xs, dYs = [to_bf16_dev(X0), to_bf16_dev(X1)], [to_bf16_dev(dY0), to_bf16_dev(dY1)]
    wf = qb.alloc_workspace(qb.OP_LINEAR_FWD, dq, da, T)
    wb = qb.alloc_workspace(qb.OP_LINEAR_BWD, dq, da, T)
    alone = []
    for k in range(2):
        Y = qb.linear_fwd(dq, da, Xs[k], torch.float32, ws=wf)
        dX, dA, dB = qb.linear_bwd(dq, da, Xs[k], dYs[k], torch.float32, ws=wb)
        torch.cuda.synchronize()
        alone.append((Y.clone(), dX.clone(), dA.clone(), dB.clone()))
    assert not torch.equal(alone[0][0], alone[1][0])
    results = []
    for it in range(60):
        k = it & 1
        Y = qb.linear_fwd(dq, da, Xs[k], torch.float32, ws=wf)
        dX, dA, dB = qb.linear_bwd(dq, da, Xs[k], dYs[k], torch.float32, ws=wb)
        results.append((k, Y, dX, dA, dB))
    torch.cuda.synchronize()
    for k, Y, dX, dA, dB in results:
        assert torch.equal(Y, alone[k][0]) and torch.equal(dX, alone[k][1])
        assert torch.equal(dA, alone[k][2]) and torch.equal(dB, alone[k][3])
    assert qb.device_status(wf) == 0 and qb.device_status(wb) == 0


def test_cuda_graph_replay_equals_eager_calls(qb):
    # forward + backward captured once through the C ABI (side stream, programmatic-dependent launches and all) and
    # replayed on changing inputs in static buffers: every replay equals the eager result for the same input
    T, d_out, d_in, l1, l2, r = 515, 256, 640, 64, 8, 64
    qw, ad, X0, dY0 = make_case(93, T, d_out, d_in, l1, l2, r)
    _, _, X1, dY1 = make_case(94, T, d_out, d_in, l1, l2, r)
    ad.scaling = 30.0
    dq, da = qweight_to_dev(qw), adapter_to_dev(ad)
    ins = [(to_bf16_dev(X0), to_bf16_dev(dY0)), (to_bf16_dev(X1), to_bf16_dev(dY1))]
    wf = qb.alloc_workspace(qb.OP_LINEAR_FWD, dq, da, T)
    wb = qb.alloc_workspace(qb.OP_LINEAR_BWD, dq, da, T)
    eager = []
    for X, dY in ins:
        Y = qb.linear_fwd(dq, da, X, torch.bfloat16, ws=wf)
        dX, dA, dB = qb.linear_bwd(dq, da, X, dY, torch.bfloat16, ws=wb)
        torch.cuda.synchronize()
        eager.append((Y.clone(), dX.clone(), dA.clone(), dB.clone()))
    Xs, dYs = torch.empty_like(ins[0][0]), torch.empty_like(ins[0][1])
    Y = torch.empty((T, d_out), dtype=torch.bfloat16, device=Xs.device)
    dX = torch.empty((T, d_in), dtype=torch.bfloat16, device=Xs.device)
    dA, dB = torch.empty_like(eager[0][2]), torch.empty_like(eager[0][3])
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        Xs.copy_(ins[0][0]); dYs.copy_(ins[0][1])
        qb.linear_fwd(dq, da, Xs, ws=wf, out=Y)                       # warm-up outside the capture (lazy set-up)
        qb.linear_bwd(dq, da, Xs, dYs, ws=wb, outs=(dX, dA, dB))
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            qb.linear_fwd(dq, da, Xs, ws=wf, out=Y)
            qb.linear_bwd(dq, da, Xs, dYs, ws=wb, outs=(dX, dA, dB))
        for it in range(12):
            k = it & 1
            Xs.copy_(ins[k][0]); dYs.copy_(ins[k][1])
            g.replay()
            st.synchronize()
            assert torch.equal(Y, eager[k][0]) and torch.equal(dX, eager[k][1]), f"replay {it}"
            assert torch.equal(dA, eager[k][2]) and torch.equal(dB, eager[k][3]), f"replay {it}"
    assert qb.device_status(wf) == 0 and qb.device_status(wb) == 0


@pytest.mark.parametrize("T", [9, 12, 16])
def test_lowbit_decode_k_outer_alternating_inputs_stress(qb, T):
    # The 2..16-token decode kernel hands shared-memory buffers (weight ring, token-fragment double buffer, row-block
    # sums) back to its producers with mbarrier arrivals that must not overtake the loads from those buffers.
    # 200 calls back to back with no host synchronisation, two inputs alternating through ONE workspace (so each
    # call's fragment area is rewritten while the previous call may still drain); several K tiles (the fragment
    # buffers are reused) and more than one pass of row blocks per CTA.  Every result equals the lone call's bit
    # for bit, and the lone call matches the oracle.
    d_out, d_in = 148 * 2 * 32 + 32 * 5 + 8, 64 * 16 * 5
    qw, _, X0, _ = make_case(71, T, d_out, d_in, 64, 8, 16, qfmt=1)
    X1 = synth.round_to_bf16(synth.normal(72, "stress/X1", (T, d_in)) * np.float32(3.0))
    dq = qweight_to_dev(qw)
    Xs = [to_bf16_dev(X0), to_bf16_dev(X1)]
    ws = qb.alloc_workspace(qb.OP_LOWBIT_GEMM, dq, None, T)
    alone = []
    for k in range(2):
        Y = qb.lowbit_gemm(dq, Xs[k], torch.float32, ws=ws)
        torch.cuda.synchronize()
        alone.append(Y.clone())
    gate_strict(to_np64(alone[0]), oracle.lowbit_gemm(qw, X0), f"decode T={T}")
    gate_strict(to_np64(alone[1]), oracle.lowbit_gemm(qw, X1), f"decode T={T}, second input")
    assert not torch.equal(alone[0], alone[1])
    outs = [torch.empty_like(alone[0]) for _ in range(200)]
    for it in range(200):
        qb.lowbit_gemm(dq, Xs[it & 1], ws=ws, out=outs[it])
    torch.cuda.synchronize()
    bad = [it for it in range(200) if not torch.equal(outs[it], alone[it & 1])]
    assert not bad, f"calls {bad[:10]} differ from the lone result"
    assert qb.device_status(ws) == qb.OK


@pytest.mark.parametrize("d_out", [72, 4768])
def test_lowbit_one_token_split_tail_graph_replay(qb, d_out):
    # ONE one-token call on a split-tail shape captured into a CUDA graph and replayed on alternating inputs in a
    # static buffer.  A replay carries the hand-over epoch it was captured with, so the owner of a row block must
    # not take the flags left by the previous replay for this replay's: every replay equals the eager result.
    qw, _, X0, _ = make_case(73, 1, d_out, 64 * 256, 64, 8, 16, qfmt=1)
    X1 = synth.round_to_bf16(synth.normal(74, "tail/X1", (1, 64 * 256)) * np.float32(2.0))
    dq = qweight_to_dev(qw)
    ins = [to_bf16_dev(X0), to_bf16_dev(X1)]
    ws = qb.alloc_workspace(qb.OP_LOWBIT_GEMM, dq, None, 1)
    eager = []
    for k in range(2):
        Y = qb.lowbit_gemm(dq, ins[k], torch.float32, ws=ws)
        torch.cuda.synchronize()
        eager.append(Y.clone())
    gate_strict(to_np64(eager[0]), oracle.lowbit_gemm(qw, X0), "split tail")
    assert not torch.equal(eager[0], eager[1])
    Xs = torch.empty_like(ins[0])
    Y = torch.empty_like(eager[0])
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        Xs.copy_(ins[0])
        qb.lowbit_gemm(dq, Xs, ws=ws, out=Y)
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            qb.lowbit_gemm(dq, Xs, ws=ws, out=Y)
        for it in range(50):
            k = it & 1
            Xs.copy_(ins[k])
            g.replay()
            st.synchronize()
            assert torch.equal(Y, eager[k]), f"replay {it}"
    assert qb.device_status(ws) == qb.OK


@pytest.mark.parametrize("T,d_out,d_in", [(300, 320, 448), (515, 264, 72), (1, 8, 64), (77, 1000, 1096)])
def test_dense_gemm_parity(qb, T, d_out, d_in):
    # the serving GEMM of the 16-bit deployment on its own: ragged tiles in every dimension, K not a multiple of 64
    W = synth.round_to_bf16(synth.normal(66, f"dg/W/{d_out}x{d_in}", (d_out, d_in), 0.02))
    X = synth.round_to_bf16(synth.normal(66, f"dg/X/{T}", (T, d_in)))
    ref = X.astype(np.float64) @ W.astype(np.float64).T
    Wd, Xd = to_bf16_dev(W), to_bf16_dev(X)
    for dt, gate in ((torch.float32, gate_strict), (torch.bfloat16, gate_bf16)):
        g = Guarded()
        Y = g.alloc((T, d_out), dt)
        ws = g.alloc((256,), torch.uint8)
        qb.dense_gemm(Wd, Xd, ws=ws, out=Y)
        g.check("dense_gemm")
        assert qb.device_status(ws) == qb.OK
        gate(to_np64(Y), ref, f"dense gemm {T}x{d_out}x{d_in}")
    # fp32 accumulation of exact bf16 products: far tighter than the gate
    assert np.abs(to_np64(qb.dense_gemm(Wd, Xd, torch.float32)) - ref).max() <= 1e-5 * np.sqrt(d_in)
