"""Pins for the oracle's block-wise 4-bit quantizer (Eq. 1; Sec. 3.2's level-table format).

None of these call the GPU library.  Each compares the oracle with something
fixed by the mathematics: closed forms, an independent numpy brute force, the
round-trip property, scipy's normal quantile for the default table.
"""
import os

import numpy as np
import pytest
from scipy.special import ndtri

import oracle
from paper_2407_17029_b200 import synth


def unpack(codes):
    lo = codes & 0x0F
    hi = codes >> 4
    return np.stack([lo, hi], axis=-1).reshape(codes.shape[0], -1)


def test_default_table_matches_closed_form_via_scipy():
    t = oracle.default_code_table()
    pos = [ndtri(0.5 + j / 17) / ndtri(0.5 + 8 / 17) for j in range(9)]
    neg = [-ndtri(0.5 + j / 15) / ndtri(0.5 + 7 / 15) for j in range(1, 8)]
    ref = np.array(sorted(neg) + pos, dtype=np.float32)
    assert t.dtype == np.float32 and t.shape == (16,)
    assert np.array_equal(t, ref)
    assert t[0] == -1.0 and t[7] == 0.0 and t[15] == 1.0
    assert np.all(np.diff(t) > 0)


def test_default_table_matches_golden_file():
    path = os.path.join(os.path.dirname(__file__), "golden", "default_code_table.txt")
    vals = [float.fromhex(l.strip()) for l in open(path) if l.strip() and not l.startswith("#")]
    assert np.array_equal(np.array(vals, dtype=np.float32), oracle.default_code_table())


@pytest.mark.parametrize("a", [1.0, 0.25, 0.0371])
def test_codebook_closed_form_levels_map_to_themselves(a):
    # a block equal to a*Tab (each level four times) quantizes to codes 0..15 and alpha = a
    t = oracle.default_code_table()
    row = np.tile(np.float32(a) * t, 4).astype(np.float32)
    W = np.stack([row, row[::-1].copy()])
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_CODEBOOK_ABSMAX)
    c = unpack(qw.codes)
    assert np.array_equal(c[0], np.tile(np.arange(16), 4))
    assert np.array_equal(c[1], np.tile(np.arange(16), 4)[::-1])
    assert qw.alpha[0, 0] == np.float32(a) and qw.alpha[1, 0] == np.float32(a)
    assert qw.beta is None
    assert np.allclose(oracle.dequantize(qw), W.astype(np.float64), rtol=1e-7, atol=0)


def test_affine_closed_form_grid_maps_to_integers():
    # block = beta + alpha*k, exactly representable: Eq. 1 min-max gives alpha, beta, codes = k
    alpha, beta = np.float32(0.125), np.float32(-1.0)
    k = np.tile(np.arange(16), 4)
    W = (beta + alpha * k).astype(np.float32)[None, :]
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX)
    assert qw.alpha[0, 0] == alpha and qw.beta[0, 0] == beta
    assert np.array_equal(unpack(qw.codes)[0], k)
    assert np.array_equal(oracle.dequantize(qw), W.astype(np.float64))


def _blocks(W, bi, bo):
    d_out, d_in = W.shape
    return W.reshape(d_out // bo, bo, d_in // bi, bi).transpose(0, 2, 1, 3).reshape(d_out // bo, d_in // bi, bo * bi)


def _unblocks(Cb, d_out, d_in, bi, bo):
    return Cb.reshape(d_out // bo, d_in // bi, bo, bi).transpose(0, 2, 1, 3).reshape(d_out, d_in)


@pytest.mark.parametrize("bi,bo", [(64, 1), (32, 1), (8, 8), (4, 8)])
def test_codebook_brute_force_nearest_level(bi, bo):
    W = synth.normal(3, f"bf/{bi}x{bo}", (64, 256), 0.02)
    t = oracle.default_code_table().astype(np.float64)
    qw = oracle.quantize_blockwise(W, bi, bo, oracle.FMT_CODEBOOK_ABSMAX)
    Wb = _blocks(W.astype(np.float64), bi, bo)
    amax = np.abs(Wb).max(axis=2)
    assert np.array_equal(qw.alpha, amax.astype(np.float32))          # alpha = absmax, exactly
    v = Wb / amax[..., None]
    dist = np.abs(v[..., None] - t)
    best = dist.argmin(axis=-1)
    srt = np.sort(dist, axis=-1)
    clear = (srt[..., 1] - srt[..., 0]) > 1e-6                        # away from ties
    got = _blocks(unpack(qw.codes), bi, bo)
    assert clear.mean() > 0.999
    assert np.array_equal(got[clear], best[clear])


@pytest.mark.parametrize("bi,bo", [(64, 1), (32, 1), (8, 8), (4, 8)])
def test_affine_brute_force_rounding(bi, bo):
    W = synth.normal(4, f"af/{bi}x{bo}", (64, 256), 0.02)
    qw = oracle.quantize_blockwise(W, bi, bo, oracle.FMT_AFFINE_MINMAX)
    Wb = _blocks(W.astype(np.float64), bi, bo)
    mn, mx = Wb.min(axis=2), Wb.max(axis=2)
    assert np.array_equal(qw.beta, mn.astype(np.float32))             # beta = min (Eq. 1)
    a = (mx - mn) / 15.0                                              # alpha = (max-min)/(2^4-1)
    assert np.allclose(qw.alpha, a, rtol=3e-7, atol=0)
    q = (Wb - mn[..., None]) / a[..., None]
    clear = np.abs(q - np.floor(q) - 0.5) > 1e-4
    got = _blocks(unpack(qw.codes), bi, bo)
    assert np.array_equal(got[clear], np.clip(np.rint(q), 0, 15).astype(np.uint8)[clear])
    # extremes: the minimum maps to code 0, the maximum to code 15
    assert np.all(np.take_along_axis(got, Wb.argmin(axis=2)[..., None], 2) == 0)
    assert np.all(np.take_along_axis(got, Wb.argmax(axis=2)[..., None], 2) == 15)


def test_codebook_extremes_and_round_trip_bit_exact():
    W = synth.normal(5, "rt/W", (96, 512), 0.02)
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_CODEBOOK_ABSMAX)
    c = unpack(qw.codes).reshape(96, 8, 64)
    Wb = W.reshape(96, 8, 64)
    am = np.abs(Wb).argmax(axis=2)
    top = np.take_along_axis(c, am[..., None], 2)[..., 0]
    sign = np.sign(np.take_along_axis(Wb, am[..., None], 2)[..., 0])
    assert np.array_equal(top, np.where(sign > 0, 15, 0))             # absmax element -> level +-1
    # Q(D(Q(W))) == Q(W) bit for bit, and D(Q(D(.))) == D(.)
    W1 = oracle.dequantize(qw)
    qw2 = oracle.quantize_blockwise(W1.astype(np.float32), 64, 1, oracle.FMT_CODEBOOK_ABSMAX)
    assert np.array_equal(qw2.codes, qw.codes)
    assert np.array_equal(qw2.alpha.view(np.uint32), qw.alpha.view(np.uint32))
    assert np.array_equal(oracle.dequantize(qw2), W1)


def test_affine_round_trip_codes_stable():
    W = synth.normal(6, "rt/Wa", (64, 256), 0.02)
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX)
    W1 = oracle.dequantize(qw)
    qw2 = oracle.quantize_blockwise(W1.astype(np.float32), 64, 1, oracle.FMT_AFFINE_MINMAX)
    assert np.array_equal(qw2.codes, qw.codes)
    assert np.array_equal(qw2.beta, qw.beta)
    assert np.allclose(qw2.alpha, qw.alpha, rtol=5e-7, atol=0)
    # quantization error is at most half a step (Eq. 1)
    err = np.abs(W1 - W.astype(np.float64)).reshape(64, 4, 64)
    assert np.all(err <= 0.5 * qw.alpha[..., None].astype(np.float64) * (1 + 1e-5))


def test_degenerate_blocks():
    W = np.zeros((2, 128), dtype=np.float32)
    W[1, 64:] = 0.3125
    q0 = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_CODEBOOK_ABSMAX)
    c0 = unpack(q0.codes)
    assert np.all(c0[0] == 7) and np.all(c0[1, :64] == 7) and np.all(c0[1, 64:] == 15)
    assert np.array_equal(oracle.dequantize(q0), W.astype(np.float64))
    q1 = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX)
    assert np.all(unpack(q1.codes) == 0) and np.all(q1.alpha == 0)
    assert np.array_equal(oracle.dequantize(q1), W.astype(np.float64))


def test_packing_low_nibble_is_even_column():
    t = oracle.default_code_table()
    W = np.zeros((1, 64), dtype=np.float32)
    W[0, 0] = t[15]      # code 15 at column 0
    W[0, 1] = t[0]       # code 0 at column 1 (absmax is 1.0 either way)
    W[0, 2:] = t[9]
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_CODEBOOK_ABSMAX)
    assert qw.codes[0, 0] == 0x0F and qw.codes[0, 1] == 0x99


def test_bad_geometry_rejected():
    W = np.zeros((4, 96), dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.quantize_blockwise(W, 64, 1, 0)


def test_codebook_tie_goes_to_lower_index():
    # an element sitting exactly on the midpoint between levels j and j+1 takes code j
    t = oracle.default_code_table()
    mids = ((t[:-1].astype(np.float64) + t[1:].astype(np.float64)) / 2).astype(np.float32)
    W = np.zeros((1, 64), dtype=np.float32)
    W[0, 0] = 1.0                                  # absmax = 1, so w/alpha = w exactly
    W[0, 1:16] = mids
    W[0, 16:31] = np.nextafter(mids, np.float32(2.0))
    c = unpack(oracle.quantize_blockwise(W, 64, 1, 0).codes)[0]
    assert np.array_equal(c[1:16], np.arange(15))
    assert np.array_equal(c[16:31], np.arange(1, 16))


def test_affine_tie_rounds_half_to_even():
    W = np.zeros((1, 64), dtype=np.float32)
    W[0, 1] = 15.0                                 # min 0, max 15 -> alpha = 1, beta = 0
    W[0, 2:6] = [0.5, 1.5, 2.5, 13.5]
    c = unpack(oracle.quantize_blockwise(W, 64, 1, 1).codes)[0]
    assert list(c[2:6]) == [0, 2, 2, 14]


def test_zero_minimum_is_stored_as_positive_zero():
    # Eq. 1: beta = min(w).  +0 and -0 compare equal, so "min" does not say which one a zero minimum is;
    # the stored beta is +0 whatever the order and signs of the zeros in the block, and codes / alpha do
    # not depend on it (w - (+0) and w - (-0) round to the same code).
    base = np.zeros((1, 64), dtype=np.float32)
    base[0, 2:] = np.linspace(0.0, 1.5, 62, dtype=np.float32)
    ref = None
    for z0, z1 in [(0.0, 0.0), (-0.0, 0.0), (0.0, -0.0), (-0.0, -0.0)]:
        W = base.copy()
        W[0, 0], W[0, 1] = np.float32(z0), np.float32(z1)
        qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX)
        assert qw.beta.view(np.uint32)[0, 0] == 0            # +0.0 bit pattern
        assert qw.alpha[0, 0] == np.float32(np.float32(1.5) / np.float32(15.0))
        if ref is None:
            ref = qw
        assert np.array_equal(qw.codes, ref.codes) and np.array_equal(qw.alpha, ref.alpha)
    # a block of zeros of mixed sign is degenerate: alpha = 0, beta = +0, codes 0
    W = np.zeros((1, 64), dtype=np.float32)
    W[0, ::2] = np.float32(-0.0)
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX)
    assert qw.beta.view(np.uint32)[0, 0] == 0 and qw.alpha[0, 0] == 0 and not qw.codes.any()
    # a negative minimum is untouched
    W[0, 5] = np.float32(-0.25)
    assert oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX).beta[0, 0] == np.float32(-0.25)


# ----------------------------------------------------------------- N-bit grids (Eq. 1 with N < 4)
@pytest.mark.parametrize("nbits", [1, 2, 3])
def test_nbit_closed_form_grid_maps_to_integers(nbits):
    # block = beta + alpha*k, k = 0 .. 2^N-1: Eq. 1 min-max returns alpha, beta and codes = k exactly
    levels = 1 << nbits
    alpha, beta = np.float32(0.25), np.float32(-0.75)
    k = np.tile(np.arange(levels), 64 // levels)
    W = (beta + alpha * k).astype(np.float32)[None, :]
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX, nbits=nbits)
    assert qw.alpha[0, 0] == alpha and qw.beta[0, 0] == beta
    assert np.array_equal(unpack(qw.codes)[0], k)
    assert np.array_equal(oracle.dequantize(qw), W.astype(np.float64))


@pytest.mark.parametrize("nbits", [2, 3])
@pytest.mark.parametrize("bi,bo", [(64, 1), (8, 8)])
def test_nbit_brute_force_rounding_and_error_bound(nbits, bi, bo):
    qmax = (1 << nbits) - 1
    W = synth.normal(5, f"nbit/{nbits}/{bi}x{bo}", (64, 256), 0.02)
    qw = oracle.quantize_blockwise(W, bi, bo, oracle.FMT_AFFINE_MINMAX, nbits=nbits)
    Wb = _blocks(W.astype(np.float64), bi, bo)
    mn, mx = Wb.min(axis=2), Wb.max(axis=2)
    assert np.array_equal(qw.beta, mn.astype(np.float32))
    a = (mx - mn) / qmax                                              # alpha = (max-min)/(2^N-1)
    assert np.allclose(qw.alpha, a, rtol=3e-7, atol=0)
    q = (Wb - mn[..., None]) / a[..., None]
    clear = np.abs(q - np.floor(q) - 0.5) > 1e-4
    got = _blocks(unpack(qw.codes), bi, bo)
    assert got.max() == qmax and got.min() == 0                      # the whole N-bit range and nothing beyond it
    assert np.array_equal(got[clear], np.clip(np.rint(q), 0, qmax).astype(np.uint8)[clear])
    # rounding to the nearest grid point: |w - w~| <= alpha / 2 (small slack for the fp32 steps)
    err = np.abs(_blocks(oracle.dequantize(qw), bi, bo) - Wb)
    assert np.all(err <= 0.5 * qw.alpha.astype(np.float64)[..., None] * (1 + 1e-5))
    # one bit less doubles the step: the worst error grows accordingly
    qw4 = oracle.quantize_blockwise(W, bi, bo, oracle.FMT_AFFINE_MINMAX)
    assert np.abs(oracle.dequantize(qw4) - W).max() < err.max()


def test_nbit_four_is_the_default_and_round_trip_is_stable():
    W = synth.normal(6, "nbit/rt", (32, 128), 0.02)
    q4 = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX)
    q4b = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX, nbits=4)
    assert np.array_equal(q4.codes, q4b.codes) and np.array_equal(q4.alpha, q4b.alpha)
    for nbits in (2, 3):
        q = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX, nbits=nbits)
        again = oracle.quantize_blockwise(oracle.dequantize(q).astype(np.float32), 64, 1,
                                          oracle.FMT_AFFINE_MINMAX, nbits=nbits)
        assert np.mean(unpack(again.codes) == unpack(q.codes)) > 0.995       # codes stable under a second pass
    with pytest.raises(ValueError):
        oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX, nbits=5)
    with pytest.raises(ValueError):
        oracle.quantize_blockwise(W, 64, 1, oracle.FMT_CODEBOOK_ABSMAX, nbits=3)


# ----------------------------------------------------------------- dense N-bit storage (N = 2, 3)
def test_pack_two_bit_layout_by_hand():
    # codes 0,1,2,3 in one byte: code j in bits 2j..2j+1 -> 0b11_10_01_00
    nib = np.array([[0x10, 0x32, 0x03, 0x21]], dtype=np.uint8)     # codes 0,1,2,3,3,0,1,2 (low nibble = even column)
    packed = oracle.pack_codes(nib, 8, 2)
    assert packed.shape == (1, 2)
    assert packed[0, 0] == 0b11100100 and packed[0, 1] == 0b10010011


def test_pack_three_bit_layout_by_hand():
    # codes 0..7 -> the 24-bit number sum_j j << 3j = 0o76543210, little-endian in three bytes
    nib = np.array([[0x10, 0x32, 0x54, 0x76]], dtype=np.uint8)
    packed = oracle.pack_codes(nib, 8, 3)
    assert packed.shape == (1, 3)
    value = int("76543210", 8)
    assert [int(b) for b in packed[0]] == [value & 0xFF, (value >> 8) & 0xFF, (value >> 16) & 0xFF]
    # a second group lands in the next three bytes and does not touch the first
    nib2 = np.array([[0x10, 0x32, 0x54, 0x76, 0x77, 0x77, 0x77, 0x77]], dtype=np.uint8)
    p2 = oracle.pack_codes(nib2, 16, 3)
    assert np.array_equal(p2[0, :3], packed[0]) and [int(b) for b in p2[0, 3:]] == [0xFF, 0xFF, 0xFF]


@pytest.mark.parametrize("nbits", [2, 3])
def test_pack_round_trip_sizes_and_refusals(nbits):
    rng = np.random.default_rng(5)
    d_out, d_in = 7, 192
    c = rng.integers(0, 1 << nbits, size=(d_out, d_in), dtype=np.uint8)
    nib = (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
    packed = oracle.pack_codes(nib, d_in, nbits)
    assert packed.shape == (d_out, d_in * nbits // 8)                 # N/8 bytes per weight
    assert np.array_equal(oracle.unpack_codes(packed, d_in, nbits), nib)
    # independent restatement: the row's bit string, least significant bit first
    bits = ((c[:, :, None] >> np.arange(nbits)[None, None, :]) & 1).reshape(d_out, -1)
    assert np.array_equal(np.packbits(bits, axis=1, bitorder="little"), packed)
    # a code that needs more than N bits is refused
    bad = nib.copy()
    bad[0, 0] = 0x0F
    with pytest.raises(ValueError):
        oracle.pack_codes(bad, d_in, nbits)
    # the quantizer's N-bit grid fits, and dequantizing the round-tripped codes changes nothing
    W = np.random.default_rng(6).standard_normal((4, 128)).astype(np.float32)
    qw = oracle.quantize_blockwise(W, 64, 1, oracle.FMT_AFFINE_MINMAX, nbits=nbits)
    rt = oracle.unpack_codes(oracle.pack_codes(qw.codes, 128, nbits), 128, nbits)
    assert np.array_equal(rt, qw.codes)
