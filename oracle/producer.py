"""CPU oracle of the operand producer that precedes the quantiser -- TEST INFRASTRUCTURE ONLY.

Paper, Appendix "Operands, Scaling, and Accumulation": q and k arrive in BF16 after QK
normalisation; where rotary embedding is used the producer applies it in FP32 and rounds the
rotated channels to BF16; q is then multiplied by tau = d**-0.5 in FP32 and the FP32 mean key over
sequence positions (separately for each channel and KV head) is subtracted from k; the results are
quantised.  Rotary pairs are (c, c + d/2) over the whole head (the generators' convention).

Plain numpy; every FP32 / BF16 rounding is written out so that the CUDA producer can be compared
bit for bit:
    t  = fl32(x2 * sin)            r1 = fl32(x1 * cos - t)       (one fused multiply-add)
    t' = fl32(x1 * sin)            r2 = fl32(x2 * cos + t')
    r  = bf16(r1 | r2)
    mean_c = fl32( (sum_n r_nc) / N )   with the sum exact (BF16 terms in float64)
    y = fl32( fl32(r - mean) * scale )  (either step is skipped when not requested)
Only ``tests/`` may import this module.
"""
import numpy as np

from . import mxfp8


def _fl32(x):
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


def rope_half_split(x, cos, sin):
    """Rotary embedding of ``x`` [..., N, d] with FP32 tables ``cos``, ``sin`` [N, d/2]; rotated
    channels rounded to BF16.  Inputs are BF16- or FP32-representable float64 arrays."""
    x = np.asarray(x, dtype=np.float64)
    half = x.shape[-1] // 2
    c, s = _fl32(cos), _fl32(sin)
    x1, x2 = x[..., :half], x[..., half:]
    # float64 holds x*c exactly (24-bit by 24-bit); adding the FP32 term is exact too unless the
    # two differ by more than 2^5 in magnitude, where the extra rounding sits 2^-29 below the FP32
    # one: rounding the float64 result to FP32 reproduces a fused multiply-add
    r1 = _fl32(x1 * c - _fl32(x2 * s))
    r2 = _fl32(x2 * c + _fl32(x1 * s))
    return mxfp8.round_bf16(np.concatenate([r1, r2], axis=-1))


def token_mean(x):
    """FP32 mean over sequence positions of ``x`` [B, H, N, d] per (batch, head, channel); the sum is
    exact for BF16 terms."""
    x = np.asarray(x, dtype=np.float64)
    return _fl32(x.sum(axis=-2) / x.shape[-2])


def fused_operand(x, cos=None, sin=None, scale=None, center=False):
    """The tensor the quantiser sees: optional rotary embedding (BF16-rounded), optional subtraction
    of the FP32 token mean, optional FP32 multiplication by ``scale``.  Returns (y, mean or None)."""
    y = np.asarray(x, dtype=np.float64)
    if cos is not None:
        y = rope_half_split(y, cos, sin)
    mean = None
    if center:
        mean = token_mean(y)
        y = _fl32(y - mean[..., None, :])
    if scale is not None:
        y = _fl32(y * _fl32(scale))
    return y, mean


def rope_tables(n_tokens, head_dim, base=10000.0):
    """FP32 cos / sin tables [N, d/2] of the standard rotary embedding (positions 0..N-1)."""
    half = head_dim // 2
    inv_freq = (np.float32(base) ** (-(np.arange(half, dtype=np.float32) / np.float32(half)))).astype(np.float32)
    ang = (np.arange(n_tokens, dtype=np.float32)[:, None] * inv_freq[None, :]).astype(np.float32)
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)
