"""Pins of the producer oracle (rotary embedding, tau fold, key centering) against facts it does not restate."""
import numpy as np
import torch

from oracle import attention as A
from oracle import mxfp8
from oracle import producer as P


def _bf16(x):
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16).to(torch.float32).numpy().astype(np.float64)


def _inputs(seed, B=1, H=2, N=64, d=32):
    rng = np.random.default_rng(seed)
    return _bf16(rng.standard_normal((B, H, N, d)))


def test_rope_is_a_rotation_and_matches_complex_multiplication():
    x = _inputs(1)
    cos, sin = P.rope_tables(64, 32)
    r = P.rope_half_split(x, cos, sin)
    half = 16
    z = (x[..., :half] + 1j * x[..., half:]) * (cos.astype(np.float64) + 1j * sin.astype(np.float64))
    want = np.concatenate([z.real, z.imag], axis=-1)
    # BF16 rounding of the rotated channels: half an ulp of 8 significant bits
    assert np.all(np.abs(r - want) <= 2.0 ** -8 * np.abs(want) + 1e-30)
    assert np.array_equal(r, _bf16(r))
    # norms of the pairs are preserved up to that rounding
    assert np.allclose((r[..., :half] ** 2 + r[..., half:] ** 2), (x[..., :half] ** 2 + x[..., half:] ** 2), rtol=2.0 ** -6, atol=1e-6)
    # position 0 is the identity (cos 1, sin 0), exactly
    assert np.array_equal(r[..., 0, :], x[..., 0, :])
    # the library tables agree with the workload generator's rotary embedding
    from paper_2609_37852_b200 import workloads
    t = torch.from_numpy(x.astype(np.float32))
    ref = workloads._rope_half_split(t).to(torch.bfloat16).to(torch.float32).numpy().astype(np.float64)
    assert np.mean(ref != r) < 0.02 and np.abs(ref - r).max() <= 2.0 ** -7 * np.abs(ref).max()


def test_token_mean_is_the_correctly_rounded_exact_mean():
    x = _inputs(2, N=96)
    m = P.token_mean(x)
    from fractions import Fraction
    for (b, h, c) in [(0, 0, 0), (0, 1, 7), (0, 1, 31)]:
        exact = sum(Fraction(float(v)) for v in x[b, h, :, c]) / 96
        assert float(np.float32(float(exact))) == m[b, h, c]


def test_key_centering_leaves_softmax_attention_unchanged():
    """Subtracting one vector from every key shifts each score row by a constant (paper: centering
    preserves softmax before quantisation in exact arithmetic)."""
    rng = np.random.default_rng(3)
    q, k, v = (rng.standard_normal((1, 2, 48, 16)) for _ in range(3))
    kc, mean = P.fused_operand(_bf16(k), center=True)
    O0, L0 = A.ref_forward(q, _bf16(k), v, 0.25, True)
    O1, L1 = A.ref_forward(q, kc, v, 0.25, True)
    # kc carries one FP32 rounding per element
    assert np.abs(O0 - O1).max() <= 1e-5
    shift = 0.25 * np.einsum("bhnd,bhd->bhn", q, mean)
    assert np.abs((L0 - L1) - shift).max() <= 1e-5
    assert np.abs(kc.sum(axis=-2)).max() <= 48 * 2.0 ** -24 * np.abs(_bf16(k)).max() * 4


def test_tau_fold_equals_the_softmax_scale():
    rng = np.random.default_rng(4)
    q, k, v = (_bf16(rng.standard_normal((1, 1, 40, 64))) for _ in range(3))
    tau = 64 ** -0.5                                   # a power of two: the fold is exact
    qs, _ = P.fused_operand(q, scale=tau)
    O0, L0 = A.ref_forward(q, k, v, tau, False)
    O1, L1 = A.ref_forward(qs, k, v, 1.0, False)
    assert np.array_equal(O0, O1) and np.array_equal(L0, L1)
    # and it only moves the scale bytes of the quantised operand
    c0, e0 = mxfp8.quantize(q)
    c1, e1 = mxfp8.quantize(qs)
    assert np.array_equal(c0, c1) and np.array_equal(e0.astype(int) - 3, e1.astype(int))


def test_fused_operand_order_of_operations():
    x = _inputs(5)
    cos, sin = P.rope_tables(64, 32)
    y, mean = P.fused_operand(x, cos, sin, scale=0.3, center=True)
    r = P.rope_half_split(x, cos, sin)
    assert np.array_equal(mean, P.token_mean(r))
    f32 = lambda a: np.asarray(a, np.float64).astype(np.float32).astype(np.float64)
    assert np.array_equal(y, f32(f32(r - mean[..., None, :]) * f32(0.3)))
    assert np.array_equal(y, f32(y))
