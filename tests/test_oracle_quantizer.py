"""Pins for the oracle's block quantiser (E4M3 codes, E8M0 scales).

Each check compares the oracle against something other than itself: torch's
own float8 casts, a brute-force nearest-value search over the 127 magnitudes
of the format, or an invariant of the scale rule.
"""
import math

import numpy as np
import pytest
import torch

from oracle import mxfp8


def _format_magnitudes():
    """The non-negative E4M3 values, from the format definition (bias 7, three
    mantissa bits, subnormals at exponent field 0, 0x7F reserved for NaN)."""
    vals = []
    for code in range(0x7F):
        e, m = code >> 3, code & 7
        vals.append((m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7))
    return vals


def _brute_encode(y):
    """Nearest representable magnitude; ties go to the even code; saturate at 448."""
    vals = _format_magnitudes()
    a = min(abs(y), 448.0)
    best = min(range(len(vals)), key=lambda c: (abs(vals[c] - a), c & 1))
    return best | (0x80 if math.copysign(1.0, y) < 0 else 0)


def test_decode_matches_torch_float8():
    codes = np.arange(256, dtype=np.uint8)
    ours = mxfp8.e4m3_decode(codes)
    theirs = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    finite = ~np.isnan(theirs)
    assert set(np.flatnonzero(~finite)) == {0x7F, 0xFF}
    assert np.array_equal(ours[finite], theirs[finite])
    assert np.isnan(ours[~finite]).all()
    assert ours[0x7E] == 448.0 and ours[0x01] == 2.0 ** -9 and ours[0x08] == 2.0 ** -6


def test_encode_roundtrip_all_codes():
    codes = np.array([c for c in range(256) if c & 0x7F != 0x7F], dtype=np.uint8)
    assert np.array_equal(mxfp8.e4m3_encode(mxfp8.e4m3_decode(codes)), codes)


def test_encode_matches_torch_cast_and_midpoints():
    vals = np.array(_format_magnitudes())
    mids = (vals[:-1] + vals[1:]) / 2                      # exact ties
    near = np.concatenate([mids * (1 - 2.0 ** -20), mids * (1 + 2.0 ** -20)])
    rng = np.random.default_rng(0)
    rand = rng.uniform(-448, 448, 20000)
    small = rng.uniform(-2.0 ** -5, 2.0 ** -5, 5000)
    y = np.concatenate([vals, -vals, mids, -mids, near, rand, small]).astype(np.float32)
    ours = mxfp8.e4m3_encode(y.astype(np.float64))
    theirs = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(ours, theirs)


def test_encode_matches_brute_force_search():
    rng = np.random.default_rng(1)
    ys = np.concatenate([rng.normal(0, 100, 3000), rng.normal(0, 0.01, 1000),
                         [0.0, -0.0, 448.0, 449.0, 464.0, 465.0, 1e9, -1e9, 2.0 ** -10, 3 * 2.0 ** -10,
                          2.0 ** -10 * 1.0001, -2.0 ** -10]])
    got = mxfp8.e4m3_encode(ys)
    for y, c in zip(ys, got):
        assert c == _brute_encode(float(y)), (y, c)


def test_encode_special_values():
    got = mxfp8.e4m3_encode(np.array([np.nan, np.inf, -np.inf, 1e30, -0.0, 0.0]))
    assert list(got) == [0x7F, 0x7E, 0xFE, 0x7E, 0x80, 0x00]


def test_scale_rule_by_definition_and_invariants():
    """Every positive finite BF16 magnitude as a block maximum: the exponent is the
    smallest one that maps it to at most 448 (checked by direct search), so the
    scaled maximum lies in (224, 448] and its code lies in [0x76, 0x7E]."""
    bits = np.arange(0x0080, 0x7F80, dtype=np.uint32) << 16   # positive normal BF16 values
    amax = bits.view(np.float32).astype(np.float64)
    e = mxfp8.e8m0_exponent(amax)
    unclamped = (e > -127) & (e < 127)
    scaled = np.ldexp(amax, -e)
    assert np.all(scaled[unclamped] <= 448.0) and np.all(scaled[unclamped] > 224.0)
    # smallest: one less would overflow 448
    assert np.all(np.ldexp(amax[unclamped], -(e[unclamped] - 1)) > 448.0)
    codes = mxfp8.e4m3_encode(scaled[unclamped])
    assert codes.min() >= 0x76 and codes.max() <= 0x7E
    # direct search on a sample
    for a in amax[:: 997]:
        ee = -127
        while a * 2.0 ** -ee > 448.0 and ee < 127:
            ee += 1
        assert ee == mxfp8.e8m0_exponent(a)
    assert mxfp8.e8m0_exponent(0.0) == -127
    assert mxfp8.e8m0_exponent(448.0) == 0 and mxfp8.e8m0_exponent(448.0001) == 1
    assert mxfp8.e8m0_exponent(1.75) == -8 and mxfp8.e8m0_exponent(1.76) == -7


def test_scale_bytes_decode_like_torch_e8m0():
    rng = np.random.default_rng(2)
    x = rng.normal(0, 1, (4, 64)) * np.exp2(rng.integers(-20, 20, (4, 1)))
    codes, scales = mxfp8.quantize(x, axis=-1)
    s_torch = torch.from_numpy(scales.copy()).view(torch.float8_e8m0fnu).to(torch.float64).numpy()
    v_torch = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    expect = v_torch * np.repeat(s_torch, 32, axis=-1)
    assert np.array_equal(mxfp8.dequantize(codes, scales), expect)


def test_quantize_block_geometry_and_axis():
    """Blocks are 32 consecutive elements along the named axis: scaling one block
    by 2**k moves only that block's scale byte; the other axis is untouched."""
    rng = np.random.default_rng(3)
    x = rng.normal(0, 1, (64, 96))
    c0, s0 = mxfp8.quantize(x, axis=-1)
    assert c0.shape == (64, 96) and s0.shape == (64, 3)
    x2 = x.copy()
    x2[5, 32:64] *= 2.0 ** 9
    c1, s1 = mxfp8.quantize(x2, axis=-1)
    assert np.array_equal(c0, c1)
    d = s1.astype(int) - s0.astype(int)
    assert d[5, 1] == 9 and np.count_nonzero(d) == 1
    ct, st = mxfp8.quantize(x, axis=0)
    assert ct.shape == (64, 96) and st.shape == (2, 96)
    c_ref, s_ref = mxfp8.quantize(x.T.copy(), axis=-1)
    assert np.array_equal(ct, c_ref.T) and np.array_equal(st, s_ref.T)
    with pytest.raises(ValueError):
        mxfp8.quantize(np.zeros((4, 48)))


def test_dequantisation_error_bound_and_zero_blocks():
    rng = np.random.default_rng(4)
    x = rng.normal(0, 1, (128, 128))
    xq = mxfp8.fake_quant(x, axis=-1)
    blk = np.abs(x).reshape(128, 4, 32)
    amax = blk.max(-1, keepdims=True)
    normal = (blk >= amax * 2.0 ** -14)            # scaled value in the normal range of E4M3
    rel = np.abs(xq - x).reshape(128, 4, 32) / blk
    assert rel[normal].max() <= 2.0 ** -4
    z = np.zeros((2, 64))
    z[1, 40] = -0.0
    c, s = mxfp8.quantize(z)
    assert np.all(s == 0) and c[1, 40] == 0x80 and np.count_nonzero(c) == 1


def test_round_bf16_matches_torch():
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.normal(0, 1, 5000), rng.normal(0, 1e-3, 5000), [1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8]])
    x32 = x.astype(np.float32)
    ours = mxfp8.round_bf16(x32.astype(np.float64))
    theirs = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(ours, theirs)


def test_round_bf16_underflows_gradually_like_torch():
    """Below 2**-126 BF16 has subnormals of spacing 2**-133: torch's cast is the reference there too, and
    float64 values far below the format (probabilities of far keys in BF16 mode) round to zero, not NaN."""
    bits = np.arange(0, 0x01000000, 0x1357, dtype=np.uint32)           # FP32 subnormals and the first normal binades
    x32 = np.concatenate([bits.view(np.float32), -bits.view(np.float32),
                          np.float32(2.0) ** np.arange(-149, -120).astype(np.float32) * np.float32(1.5)])
    ours = mxfp8.round_bf16(x32.astype(np.float64))
    theirs = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(ours, theirs)
    tiny = np.array([1e-300, -1e-310, 5e-324, 2.0 ** -135, 2.0 ** -134, 3 * 2.0 ** -135])
    want = np.array([0.0, -0.0, 0.0, 0.0, 0.0, 2.0 ** -133])            # ties to even; 3/4 of the step rounds up
    got = mxfp8.round_bf16(tiny)
    assert np.array_equal(got, want) and not np.isnan(got).any()
