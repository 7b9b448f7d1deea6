"""Oracle quantiser: E4M3 codes with E8M0 block scales (test infrastructure only).

The paper's kernel quantises every attention-core operand to E4M3 with
round-to-nearest-even and saturation at +-448 and applies block scales to the
matmul results (Appendix "Operands, Scaling, and Accumulation", Eq.
app_kernel_quantizer).  This build keeps the code format and replaces the
paper's FP32 scale ``amax/448`` per row block by an MXFP8-style scale: one
power of two (E8M0 byte) per 32 consecutive elements along the contraction
dimension, chosen as the smallest power of two that maps the block maximum to
at most 448 -- the power-of-two analogue of "the block maximum maps to 448".

Everything is float64/integer numpy; nothing here is shared with the CUDA path.
"""
import numpy as np

BLOCK = 32
E4M3_MAX = 448.0


def e4m3_decode(codes):
    """Value of each E4M3 ("fn": no infinities, 0x7F/0xFF are NaN) byte, as float64."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    expo = (c >> 3) & 0xF
    mant = (c & 0x7).astype(np.float64)
    normal = np.ldexp(1.0 + mant / 8.0, expo - 7)
    subnormal = np.ldexp(mant / 8.0, -6)
    mag = np.where(expo == 0, subnormal, normal)
    mag = np.where((c & 0x7F) == 0x7F, np.nan, mag)
    return sign * mag


def e4m3_encode(y):
    """Round float64 values to E4M3 bytes: nearest, ties to even mantissa,
    magnitudes above 448 saturate to 448 (Eq. app_kernel_quantizer: C_8).
    The sign of zero is kept; NaN gives 0x7F; +-Inf gives +-448."""
    y = np.asarray(y, dtype=np.float64)
    neg = np.signbit(y)
    a = np.abs(y)
    isnan = np.isnan(a)
    a = np.where(isnan, 0.0, a)
    a = np.minimum(a, E4M3_MAX)
    # a = m * 2**ex with m in [0.5, 1): binade exponent E = ex - 1.
    _, ex = np.frexp(a)
    E = np.maximum(ex - 1, -6)              # below 2**-6 the grid is the subnormal one
    quantum = np.ldexp(1.0, E - 3)          # spacing of representable values in that binade
    qn = np.rint(a / quantum)               # rint rounds halves to even; division is exact
    val = qn * quantum                      # representable magnitude (may be next binade)
    _, ex2 = np.frexp(val)
    E2 = ex2 - 1
    is_sub = (val < np.ldexp(1.0, -6))
    mant_norm = np.rint(np.ldexp(val, -(E2 - 3))) - 8      # 0..7
    code_norm = ((E2 + 7).astype(np.int64) << 3) | mant_norm.astype(np.int64)
    code_sub = np.rint(np.ldexp(val, 9)).astype(np.int64)  # 0..7 (8 is the first normal)
    code = np.where(is_sub, code_sub, code_norm)
    code = np.where(val == 0.0, 0, code)
    code = np.where(isnan, 0x7F, code)
    code = code | np.where(neg & ~isnan, 0x80, 0)
    return code.astype(np.uint8)


def e8m0_exponent(amax):
    """Unbiased block exponent e: the smallest integer with amax * 2**-e <= 448,
    clamped to [-127, 127]; an all-zero block takes -127 (stored byte 0).
    With amax = 1.m * 2**E this is E - 8, plus one when 1.m > 1.75 (448 = 1.75 * 2**8)."""
    amax = np.asarray(amax, dtype=np.float64)
    m, ex = np.frexp(amax)                  # amax = m * 2**ex, m in [0.5, 1)
    E = ex - 1
    e = E - 8 + (2.0 * m > 1.75)
    e = np.where(amax == 0.0, -127, e)
    e = np.where(np.isfinite(amax), e, 127)
    return np.clip(e, -127, 127).astype(np.int64)


def quantize(x, axis=-1):
    """Quantise ``x`` in blocks of 32 consecutive elements along ``axis``
    (blocks aligned to multiples of 32 of the absolute index).

    Returns (codes uint8, same shape as x; scale bytes uint8 with ``axis``
    reduced by 32).  Scale byte = e + 127."""
    x = np.asarray(x, dtype=np.float64)
    xm = np.moveaxis(x, axis, -1)
    n = xm.shape[-1]
    if n % BLOCK:
        raise ValueError("length along the block axis must be a multiple of 32")
    blk = xm.reshape(xm.shape[:-1] + (n // BLOCK, BLOCK))
    amax = np.max(np.abs(np.where(np.isnan(blk), 0.0, blk)), axis=-1)
    e = e8m0_exponent(amax)
    y = np.ldexp(blk, -e[..., None])        # exact scaling by a power of two
    codes = e4m3_encode(y).reshape(xm.shape)
    scales = (e + 127).astype(np.uint8)
    return np.moveaxis(codes, -1, axis), np.moveaxis(scales, -1, axis)


def dequantize(codes, scales, axis=-1):
    """Value of each element: decode(code) * 2**(scale byte - 127)."""
    cm = np.moveaxis(np.asarray(codes), axis, -1)
    sm = np.moveaxis(np.asarray(scales), axis, -1).astype(np.int64) - 127
    n = cm.shape[-1]
    v = e4m3_decode(cm).reshape(cm.shape[:-1] + (n // BLOCK, BLOCK))
    out = np.ldexp(v, sm[..., None]).reshape(cm.shape)
    return np.moveaxis(out, -1, axis)


def fake_quant(x, axis=-1):
    """dequantize(quantize(x)): the value the tensor cores see for each element."""
    c, s = quantize(x, axis)
    return dequantize(c, s, axis)


def round_bf16(x):
    """Round float64 to the nearest BF16 value (8 significand bits, ties to even);
    returned as float64.  Below 2**-126 the grid is that of the BF16 subnormals (spacing 2**-133,
    gradual underflow to zero); overflow is outside the tested range."""
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    _, ex = np.frexp(a)
    quantum = np.ldexp(1.0, np.maximum(ex - 1 - 7, -133))
    r = np.rint(a / quantum) * quantum
    r = np.where(a == 0.0, 0.0, r)
    return np.copysign(r, x)


def round_f32(x):
    """Round float64 to the nearest FP32 value, returned as float64."""
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)
