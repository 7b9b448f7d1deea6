"""Pins for the oracle's attention paths.

The reference path is pinned to torch's scaled_dot_product_attention with
autograd in float64, to central finite differences, to the textbook softmax
Jacobian and to closed forms.  The emulated-FP8 path is pinned to the reference
path (quantisers switched off; grid-valued operands), to the identities the
paper proves (zero row sums under the matched correction, the stale-delta
residual and its operand-error decomposition, zero column sums of dK) and to a
loop-by-loop restatement with its own scalar quantiser on a tiny shape.
"""
import math

import numpy as np
import pytest
import torch

from oracle import attention as A
from oracle import mxfp8


def _rand(B, Hq, Hkv, N, dqk, dv, seed=0, dO_std=1.0):
    rng = np.random.default_rng(seed)
    q = rng.normal(0, 1, (B, Hq, N, dqk))
    k = rng.normal(0, 1, (B, Hkv, N, dqk))
    v = rng.normal(0, 1, (B, Hkv, N, dv))
    dO = rng.normal(0, dO_std, (B, Hq, N, dv))
    return q, k, v, dO


# ---------------------------------------------------------------- reference path

@pytest.mark.parametrize("causal", [False, True])
def test_reference_matches_sdpa_autograd(causal):
    B, Hq, Hkv, N, dqk, dv = 2, 4, 2, 48, 16, 24
    q, k, v, dO = _rand(B, Hq, Hkv, N, dqk, dv, seed=1)
    scale = 0.3
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v))
    G = Hq // Hkv
    out = torch.nn.functional.scaled_dot_product_attention(
        tq, tk.repeat_interleave(G, dim=1), tv.repeat_interleave(G, dim=1), is_causal=causal, scale=scale)
    out.backward(torch.tensor(dO))
    O, LSE = A.ref_forward(q, k, v, scale, causal)
    dQ, dK, dV, D = A.ref_backward(q, k, v, dO, scale, causal)
    assert np.abs(O - out.detach().numpy()).max() < 1e-12
    assert np.abs(dQ - tq.grad.numpy()).max() < 1e-12
    assert np.abs(dK - tk.grad.numpy()).max() < 1e-12
    assert np.abs(dV - tv.grad.numpy()).max() < 1e-12
    # LSE against torch.logsumexp of the explicit scores
    S = scale * torch.einsum("bhid,bhjd->bhij", tq.detach(), tk.detach().repeat_interleave(G, dim=1))
    if causal:
        S = S.masked_fill(torch.triu(torch.ones(N, N, dtype=torch.bool), 1), -math.inf)
    assert np.abs(LSE - torch.logsumexp(S, -1).numpy()).max() < 1e-12


def test_reference_gradient_by_central_differences():
    """N=16, d=8 (the tiny configuration's finite-difference check): d/dx of
    L = sum(O * dO) by central differences, step 1e-5."""
    q, k, v, dO = _rand(1, 1, 1, 16, 8, 8, seed=2)
    scale = 1 / math.sqrt(8)
    dQ, dK, dV, _ = A.ref_backward(q, k, v, dO, scale, True)

    def loss(q_, k_, v_):
        return float((A.ref_forward(q_, k_, v_, scale, True)[0] * dO).sum())

    h = 1e-5
    for name, x, g in (("q", q, dQ), ("k", k, dK), ("v", v, dV)):
        num = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            old = x[idx]
            x[idx] = old + h
            lp = loss(q, k, v)
            x[idx] = old - h
            lm = loss(q, k, v)
            x[idx] = old
            num[idx] = (lp - lm) / (2 * h)
        assert np.abs(num - g).max() < 1e-7, name


def test_reference_softmax_jacobian_and_identities():
    q, k, v, dO = _rand(1, 2, 1, 40, 16, 16, seed=3)
    scale = 0.25
    O, _ = A.ref_forward(q, k, v, scale, True)
    dQ, dK, dV, D, internals = A.ref_backward(q, k, v, dO, scale, True, return_internals=True)
    for (b, h), t in internals.items():
        P, dP, dS = t["P"], t["dP"], t["dS"]
        for i in range(P.shape[0]):
            J = np.diag(P[i]) - np.outer(P[i], P[i])        # textbook softmax Jacobian
            assert np.abs(J @ dP[i] - dS[i]).max() < 1e-13
        assert np.abs(dS.sum(-1)).max() < 1e-13             # Eq. 1: zero row sums
    assert np.abs(D - (dO * O).sum(-1)).max() < 1e-13       # exact saved-output identity
    assert np.abs(dK.sum(axis=2)).max() < 1e-12             # zero column sums of dK


def test_reference_closed_forms():
    rng = np.random.default_rng(4)
    N, d = 33, 8
    v = rng.normal(0, 1, (1, 1, N, d))
    k = rng.normal(0, 1, (1, 1, N, d))
    q = np.zeros((1, 1, N, d))
    O, LSE = A.ref_forward(q, k, v, 1.0, True)
    prefix_mean = np.cumsum(v[0, 0], 0) / np.arange(1, N + 1)[:, None]
    assert np.abs(O[0, 0] - prefix_mean).max() < 1e-13
    assert np.abs(LSE[0, 0] - np.log(np.arange(1, N + 1))).max() < 1e-13
    # one token: O = V, no gradient reaches Q or K
    q1, k1, v1, dO1 = _rand(1, 1, 1, 1, 4, 4, seed=5)
    O1, _ = A.ref_forward(q1, k1, v1, 0.5, True)
    dQ1, dK1, dV1, _ = A.ref_backward(q1, k1, v1, dO1, 0.5, True)
    assert np.array_equal(O1, v1) and np.all(dQ1 == 0) and np.all(dK1 == 0) and np.array_equal(dV1, dO1)


# ---------------------------------------------------------------- emulated path

@pytest.mark.parametrize("causal", [False, True])
def test_emulated_path_with_quantisers_off_is_the_reference(causal):
    q, k, v, dO = _rand(2, 4, 2, 64, 32, 32, seed=6)
    scale = 0.2
    O, LSE = A.ref_forward(q, k, v, scale, causal)
    dQ, dK, dV, D = A.ref_backward(q, k, v, dO, scale, causal)
    O2, LSE2 = A.emu_forward(q, k, v, scale, causal, prec="none")
    D2 = A.emu_delta(q, k, v, dO, LSE2, scale, causal, prec="none", exact_stats=True)
    dQ2, dK2, dV2, rs, ra = A.emu_backward(q, k, v, dO, LSE2, D2, scale, causal, prec="none")
    for a, b in ((O, O2), (LSE, LSE2), (D, D2), (dQ, dQ2), (dK, dK2), (dV, dV2)):
        assert np.abs(a - b).max() < 1e-12
    assert np.abs(rs).max() < 1e-13


def _scalar_quant_block(xs):
    """Independent scalar restatement of the block quantiser: returns dequantised values."""
    vals = []
    for code in range(0x7F):
        e, m = code >> 3, code & 7
        vals.append((m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7))
    amax = max(abs(x) for x in xs)
    if amax == 0:
        return [0.0] * len(xs)
    e = -127
    while amax * 2.0 ** -e > 448.0:
        e += 1
    out = []
    for x in xs:
        a = min(abs(x) * 2.0 ** -e, 448.0)
        c = min(range(len(vals)), key=lambda c: (abs(vals[c] - a), c & 1))
        out.append(math.copysign(vals[c] * 2.0 ** e, x))
    return out


def _fq_loops(x, axis):
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros_like(x)
    R, C = x.shape
    if axis == 1:
        for r in range(R):
            for c0 in range(0, C, 32):
                out[r, c0:c0 + 32] = _scalar_quant_block(list(x[r, c0:c0 + 32]))
    else:
        for c in range(C):
            for r0 in range(0, R, 32):
                out[r0:r0 + 32, c] = _scalar_quant_block(list(x[r0:r0 + 32, c]))
    return out


def test_emulated_fp8_against_loop_restatement():
    """One head, N=64, d=32: explicit loops over i, j, c with a scalar quantiser."""
    N, d = 64, 32
    q, k, v, dO = _rand(1, 1, 1, N, d, d, seed=7, dO_std=0.1)
    scale = 1 / math.sqrt(d)
    Qr, Kr, Vr, dOr = (_fq_loops(x[0, 0], 1) for x in (q, k, v, dO))
    Qc, Kc, Vc, dOc = (_fq_loops(x[0, 0], 0) for x in (q, k, v, dO))
    log2e = math.log2(math.e)
    p = np.zeros((N, N)); l = np.zeros(N); lse = np.zeros(N)
    for i in range(N):
        s2 = [scale * sum(Qr[i, c] * Kr[j, c] for c in range(d)) * log2e for j in range(i + 1)]
        M = math.ceil(max(s2))
        for j in range(i + 1):
            p[i, j] = 2.0 ** (s2[j] - M)
        l[i] = p[i].sum()
        lse[i] = float(np.float32((M + math.log2(l[i])) * math.log(2.0)))
    Ph = _fq_loops(p, 1)
    O = np.zeros((N, d))
    for i in range(N):
        for c in range(d):
            O[i, c] = sum(Ph[i, j] * Vc[j, c] for j in range(N)) / l[i]
    O_or, LSE_or = A.emu_forward(q, k, v, scale, True)
    assert np.array_equal(LSE_or[0, 0], lse)
    assert np.array_equal(O_or[0, 0], mxfp8.round_bf16(O))
    # backward
    P = np.zeros((N, N)); dP = np.zeros((N, N))
    for i in range(N):
        for j in range(i + 1):
            P[i, j] = math.exp(scale * sum(Qr[i, c] * Kr[j, c] for c in range(d)) - lse[i])
        for j in range(N):
            dP[i, j] = sum(dOr[i, c] * Vr[j, c] for c in range(d))
    D = np.array([np.float32(sum(P[i, j] * dP[i, j] for j in range(N))) for i in range(N)], dtype=np.float64)
    dS = P * (dP - D[:, None])
    Pi, dSi, dSj = _fq_loops(P, 0), _fq_loops(dS, 0), _fq_loops(dS, 1)
    dV = Pi.T @ dOc
    dK = scale * dSi.T @ Qc
    dQ = scale * dSj @ Kc
    D_or = A.emu_delta(q, k, v, dO, LSE_or, scale, True)
    dQ_or, dK_or, dV_or, rs, ra = A.emu_backward(q, k, v, dO, LSE_or, D_or, scale, True)
    assert np.abs(D_or[0, 0] - D).max() <= 1e-7 * np.abs(D).max()
    for got, want in ((dQ_or, dQ), (dK_or, dK), (dV_or, dV)):
        want = mxfp8.round_bf16(want)
        # identical up to BF16 ties decided by the last float64 bit of a sum
        assert np.mean(got[0, 0] != want) < 2e-3
        assert np.abs(got[0, 0] - want).max() <= 2.0 ** -7 * np.abs(want).max()


def test_forward_shift_invariance_and_tile_order():
    """Any integer shift of the row maximum gives the same probability codes, so an
    online kernel with a running integer maximum reproduces the one-shot definition."""
    N, d = 256, 64
    q, k, v, dO = _rand(1, 2, 1, N, d, d, seed=8)
    scale = 1 / math.sqrt(d)
    O0, L0, t0 = A.emu_forward(q, k, v, scale, True, return_internals=True)
    for shift in (1, 7):
        O1, L1, t1 = A.emu_forward(q, k, v, scale, True, max_shift=shift, return_internals=True)
        for key in t0:
            c0, s0 = mxfp8.quantize(t0[key]["p"])
            c1, s1 = mxfp8.quantize(t1[key]["p"])
            assert np.array_equal(c0, c1)
            live = c0.reshape(N, -1, 32).any(-1)
            assert np.all((s0.astype(int) - s1.astype(int))[live] == shift)
        assert np.array_equal(O0, O1)
        assert np.abs(L0 - L1).max() < 1e-6
    # online: 64-key tiles, running integer maximum, rescale by powers of two
    Qh, Kh, Vc = mxfp8.fake_quant(q[0, 0]), mxfp8.fake_quant(k[0, 0]), mxfp8.fake_quant(v[0, 0], 0)
    for T in (64, 128):
        acc = np.zeros((N, d)); l = np.zeros(N); M = np.full(N, -np.inf)
        for j0 in range(0, N, T):
            s2 = scale * (Qh @ Kh[j0:j0 + T].T) * A.LOG2E
            s2 = np.where(np.arange(j0, j0 + T)[None, :] > np.arange(N)[:, None], -np.inf, s2)
            Mn = np.maximum(M, np.ceil(s2.max(-1)))
            alive = np.isfinite(Mn)
            Mn_safe = np.where(alive, Mn, 0.0)
            alpha = np.where(np.isfinite(M), np.exp2(M - Mn_safe), 0.0)
            p = np.where(alive[:, None], np.exp2(s2 - Mn_safe[:, None]), 0.0)
            l = l * alpha + p.sum(-1)
            acc = acc * alpha[:, None] + mxfp8.fake_quant(p) @ Vc[j0:j0 + T]
            M = Mn
        O_online = mxfp8.round_bf16(acc / l[:, None])
        assert np.mean(O_online != O0[0, 0]) < 1e-3          # only last-bit float64 ties may differ
        assert np.abs(O_online - O0[0, 0]).max() <= 2.0 ** -7 * np.abs(O0[0, 0]).max()


def test_forward_zero_queries_gives_prefix_mean_of_quantised_values():
    rng = np.random.default_rng(9)
    N, d = 96, 32
    v = rng.normal(0, 1, (1, 1, N, d)); k = rng.normal(0, 1, (1, 1, N, d)); q = np.zeros((1, 1, N, d))
    O, LSE = A.emu_forward(q, k, v, 1.0, True)
    Vc = mxfp8.fake_quant(v[0, 0], 0)
    want = mxfp8.round_bf16(np.cumsum(Vc, 0) / np.arange(1, N + 1)[:, None])
    assert np.abs(O[0, 0] - want).max() <= 2.0 ** -8 * np.abs(want).max()
    assert np.abs(LSE[0, 0] - np.log(np.arange(1, N + 1))).max() < 1e-6


def test_grid_valued_operands_make_forward_operand_error_vanish():
    """Q = 0 and V already on the E4M3 grid with one exponent per block: p~ = 1 is
    exactly representable, so the emulated output equals the reference output up
    to its BF16 store."""
    rng = np.random.default_rng(10)
    N, d = 64, 32
    codes = rng.integers(0x30, 0x50, (N, d)).astype(np.uint8)
    v = mxfp8.e4m3_decode(codes)[None, None]
    k = rng.normal(0, 1, (1, 1, N, d)); q = np.zeros((1, 1, N, d))
    O_ref, _ = A.ref_forward(q, k, v, 1.0, True)
    O_emu, _ = A.emu_forward(q, k, v, 1.0, True)
    want = mxfp8.round_bf16(O_ref)
    # equal except where the last float64 bit of a sum decides a BF16 tie
    assert np.mean(O_emu != want) < 5e-3
    assert np.all(np.abs(O_emu - want) <= 2.0 ** -7 * np.abs(want))


def _setup_fp8(seed=11, causal=True, N=128, d=64, Hq=4, Hkv=2):
    q, k, v, dO = _rand(1, Hq, Hkv, N, d, d, seed=seed, dO_std=0.05)
    q, k, v, dO = (mxfp8.round_bf16(x) for x in (q, k, v, dO))
    scale = 1 / math.sqrt(d)
    return q, k, v, dO, scale, causal


def test_matched_delta_zero_row_sums_and_affine_identity():
    q, k, v, dO, scale, causal = _setup_fp8()
    O, LSE = A.emu_forward(q, k, v, scale, causal, exact_stats=True)
    D = A.emu_delta(q, k, v, dO, LSE, scale, causal, exact_stats=True)
    dQ, dK, dV, rs, ra, t = A.emu_backward(q, k, v, dO, LSE, D, scale, causal, return_internals=True)
    # Eq. 5.  Row 0 sees one key (P = 1, dS = 0 analytically): only rounding dust is
    # left there, bounded by |D| * |1 - sum P|, hence the second term.
    dust = np.stack([[(t[(b, h)]["P"] * np.abs(t[(b, h)]["dP"])).sum(-1) for h in range(q.shape[1])]
                     for b in range(q.shape[0])])
    assert np.all(np.abs(rs) <= 1e-12 * ra + 1e-14 * dust)
    # for any correction c: sum_j P_ij (dP_ij - c) = D_matched_i - c * sum_j P_ij
    for c in (0.0, 1.0):
        cc = np.full_like(D, c)
        _, _, dVc, rsc, _ = A.emu_backward(q, k, v, dO, LSE, cc, scale, causal)
        for (b, h), tt in t.items():
            sumP = tt["P"].sum(-1)
            assert np.abs(sumP - 1).max() < 1e-12
            assert np.abs(rsc[b, h] - (D[b, h] - c * sumP)).max() < 1e-12
        assert np.array_equal(dVc, dV)        # the correction never reaches dV
    # the paper's two-run probe recovers the matched correction: R(0) / (R(0) - R(1))
    _, _, _, r0, _ = A.emu_backward(q, k, v, dO, LSE, np.zeros_like(D), scale, causal)
    _, _, _, r1, _ = A.emu_backward(q, k, v, dO, LSE, np.ones_like(D), scale, causal)
    assert np.abs(r0 / (r0 - r1) - D).max() < 1e-12


def test_fp32_storage_of_lse_bounds_the_residual():
    q, k, v, dO, scale, causal = _setup_fp8(seed=12)
    O, LSE = A.emu_forward(q, k, v, scale, causal)
    D = A.emu_delta(q, k, v, dO, LSE, scale, causal)
    _, _, _, rs, ra, t = A.emu_backward(q, k, v, dO, LSE, D, scale, causal, return_internals=True)
    for (b, h), tt in t.items():
        bound = 1e-5 * ra[b, h] + 2.0 ** -19 * (tt["P"] * np.abs(tt["dP"])).sum(-1)
        assert np.all(np.abs(rs[b, h]) <= bound)


def test_stale_delta_residual_and_decomposition():
    q, k, v, dO, scale, causal = _setup_fp8(seed=13)
    O, LSE, fwd = A.emu_forward(q, k, v, scale, causal, exact_stats=True, return_internals=True)
    Dm = A.emu_delta(q, k, v, dO, LSE, scale, causal, exact_stats=True)
    Ds = A.emu_delta(q, k, v, dO, LSE, scale, causal, mode="stale", o=O, exact_stats=True)
    _, _, dVm, rsm, ram = A.emu_backward(q, k, v, dO, LSE, Dm, scale, causal)
    dQs, dKs, dVs, rss, ras, t = A.emu_backward(q, k, v, dO, LSE, Ds, scale, causal, return_internals=True)
    assert np.array_equal(dVm, dVs)
    G = q.shape[1] // k.shape[1]
    for (b, h), tt in t.items():
        g = h // G
        # row sum of the stale score gradient = matched minus stale correction (Appendix proof, step 2)
        assert np.abs(rss[b, h] - (Dm[b, h] - Ds[b, h])).max() < 1e-12
        # operand-error decomposition (Eq. 2) with the extra term that two V copies bring,
        # using the unrounded output and adding the BF16 storage term of the saved O
        P = tt["P"]
        Phat = fwd[(b, h)]["Ph"] / fwd[(b, h)]["l"][:, None]
        Vr, Vc = mxfp8.fake_quant(v[b, g], -1), mxfp8.fake_quant(v[b, g], 0)
        dOr = mxfp8.fake_quant(dO[b, h], -1)
        O_unrounded = Phat @ Vc
        term_p = (dOr * ((P - Phat) @ Vr)).sum(-1)
        term_v = (dOr * (Phat @ (Vr - Vc))).sum(-1)
        term_g = ((dOr - dO[b, h]) * O_unrounded).sum(-1)
        term_store = (dO[b, h] * (O_unrounded - O[b, h])).sum(-1)
        assert np.abs(rss[b, h] - (term_p + term_v + term_g + term_store)).max() < 1e-12
    r_m = A.residual_ratio(rsm, ram)[..., 64:]
    r_s = A.residual_ratio(rss, ras)[..., 64:]
    assert np.nanmedian(r_s) >= 100 * np.nanmedian(r_m)
    assert np.nanmedian(r_s) > 1e-4


def test_consistent_dO_residual_identity_and_ordering():
    """Consistent dO (Section 3.3): with dO^ in the saved-output shortcut the gradient-quantisation
    term of the stale residual disappears; what is left is the probability-quantisation term of
    Eq. delta_consistent_do_residual, plus (this build's number format) the term of the two V
    copies and the BF16 storage of O.  Median residuals order stale > consistent > matched."""
    q, k, v, dO, scale, causal = _setup_fp8(seed=21)
    O, LSE, fwd = A.emu_forward(q, k, v, scale, causal, exact_stats=True, return_internals=True)
    Dm = A.emu_delta(q, k, v, dO, LSE, scale, causal, exact_stats=True)
    Ds = A.emu_delta(q, k, v, dO, LSE, scale, causal, mode="stale", o=O, exact_stats=True)
    Dc = A.emu_delta(q, k, v, dO, LSE, scale, causal, mode="consistent", o=O, exact_stats=True)
    _, _, _, rsm, ram = A.emu_backward(q, k, v, dO, LSE, Dm, scale, causal)
    _, _, _, rss, ras = A.emu_backward(q, k, v, dO, LSE, Ds, scale, causal)
    _, _, _, rsc, rac, t = A.emu_backward(q, k, v, dO, LSE, Dc, scale, causal, return_internals=True)
    G = q.shape[1] // k.shape[1]
    for (b, h), tt in t.items():
        g = h // G
        assert np.abs(rsc[b, h] - (Dm[b, h] - Dc[b, h])).max() < 1e-12
        P = tt["P"]
        Phat = fwd[(b, h)]["Ph"] / fwd[(b, h)]["l"][:, None]
        Vr, Vc = mxfp8.fake_quant(v[b, g], -1), mxfp8.fake_quant(v[b, g], 0)
        dOr = mxfp8.fake_quant(dO[b, h], -1)
        O_unrounded = Phat @ Vc
        term_p = (dOr * ((P - Phat) @ Vr)).sum(-1)           # the paper's remaining term
        term_v = (dOr * (Phat @ (Vr - Vc))).sum(-1)          # two V copies (1x32 blocks per contraction dim)
        term_store = (dOr * (O_unrounded - O[b, h])).sum(-1)   # BF16 storage of the saved output
        assert np.abs(rsc[b, h] - (term_p + term_v + term_store)).max() < 1e-12
    med = lambda rs, ra: np.nanmedian(A.residual_ratio(rs, ra)[..., 64:])
    assert med(rss, ras) > med(rsc, rac) > 100 * med(rsm, ram)


def test_postcast_statistics_and_key_common_mode():
    """Post-cast row sums (Appendix "dS Quantization Residuals"): equal to the pre-cast ones when the
    cast is the identity; bounded by the E4M3 half-ulp otherwise; and the key-gradient sum identity
    of Eq. app_ds_gqa_key_sum, which ties sum_j dK_j to the row sums of the cast operand."""
    q, k, v, dO, scale, causal = _setup_fp8(seed=22)
    O, LSE = A.emu_forward(q, k, v, scale, causal, exact_stats=True)
    D = A.emu_delta(q, k, v, dO, LSE, scale, causal, exact_stats=True)
    dQ, dK, dV, rs, ra, t = A.emu_backward(q, k, v, dO, LSE, D, scale, causal, round_out=False, return_internals=True)
    G = q.shape[1] // k.shape[1]
    for (b, h), tt in t.items():
        ps, pa = A.postcast_row_sums(q, k, v, dO, LSE[b, h], D[b, h], scale, causal, b=b, h=h)
        assert np.array_equal(ps, tt["dS_q"].sum(-1)) and np.array_equal(pa, np.abs(tt["dS_q"]).sum(-1))
        # round to nearest with 3 mantissa bits: every element moves by at most 2^-4 of the block maximum
        assert np.all(np.abs(ps - rs[b, h]) <= 2.0 ** -4 * ra[b, h] + 1e-300)
        r_post, r_own, kappa = A.postcast_residuals(rs[b, h], ra[b, h], ps, pa)
        live = ra[b, h] > 0
        assert np.all(np.abs(kappa[live]) <= 2.0 ** -4)
        assert np.nanmedian(r_post[64:]) > 10 * np.nanmedian(A.residual_ratio(rs[b, h], ra[b, h])[64:])
        # identity cast: nothing changes
        ps0, pa0 = A.postcast_row_sums(q, k, v, dO, LSE[b, h], D[b, h], scale, causal, prec="none", b=b, h=h)
        _, _, _, rs0, ra0 = A.emu_backward(q, k, v, dO, LSE, D, scale, causal, prec="none")
        assert np.allclose(ps0, rs0[b, h], atol=1e-15) and np.allclose(pa0, ra0[b, h], rtol=1e-13)
    # key-gradient sum: sum_j dK_{g,j} = scale * sum_{h in g} sum_i Q^c_{h,i} * (sum_j dS^i_{h,ij})
    for b in range(q.shape[0]):
        for g in range(k.shape[1]):
            want = np.zeros(q.shape[-1])
            for h in range(g * G, (g + 1) * G):
                want += scale * (mxfp8.fake_quant(q[b, h], 0) * t[(b, h)]["dS_k"].sum(-1)[:, None]).sum(0)
            assert np.abs(dK[b, g].sum(0) - want).max() <= 1e-12 * max(1.0, np.abs(want).max())
    cK = A.key_common_mode(dK)
    assert cK.shape == dK.shape[:2] and np.all((cK >= 0) & (cK <= np.sqrt(dK.shape[2]) + 1e-9))


def test_key_common_mode_hand_worked():
    """Eq. app_ds_key_gradient_sum on numbers small enough to do by hand: the norm of the SUM OVER KEYS of
    the key gradients of one (batch, KV head), over the root of the sum over keys of their squared norms.
      head 0: dK_0 = (3, 4), dK_1 = (3, -4), dK_2 = (0, 0): sum = (6, 0), norm 6; squared norms 25 + 25 + 0,
              root sqrt(50) -> c_K = 6 / sqrt(50) = 0.6 sqrt(2).  (Summing over channels instead of keys
              would give rows (7), (-1), (0), i.e. sqrt(50) / sqrt(50) = 1.)
      head 1: (1, 0), (0, 1), (-1, -1): the key gradients cancel -> c_K = 0.
      head 2: three equal rows (1, 2): sum (3, 6), norm 3 sqrt(5); root sqrt(15) -> c_K = sqrt(3), the upper
              bound sqrt(N) of the statistic."""
    dK = np.array([[[[3.0, 4.0], [3.0, -4.0], [0.0, 0.0]],
                    [[1.0, 0.0], [0.0, 1.0], [-1.0, -1.0]],
                    [[1.0, 2.0], [1.0, 2.0], [1.0, 2.0]]]])
    cK = A.key_common_mode(dK)
    assert cK.shape == (1, 3)
    assert np.allclose(cK[0], [0.6 * np.sqrt(2.0), 0.0, np.sqrt(3.0)], rtol=0, atol=1e-15)
    # per head: permuting the keys of a head changes nothing, scaling a head changes nothing
    assert np.allclose(A.key_common_mode(dK[:, :, ::-1] * 7.0), cK, atol=1e-15)


def test_postcast_residuals_hand_worked():
    """Eq. app_ds_quantization_residuals and Eq. app_ds_signed_increment on four rows done by hand
    (l = sum |dS| before the cast, l' = sum |dS'| after it):
      row 0: sum dS = 0.5, l = 2, sum dS' = 0.75, l' = 3:  r_post = 0.75 / 2 = 0.375 (NOT 0.75 / 3),
             r_post,own = 0.75 / 3 = 0.25, kappa = (0.75 - 0.5) / 2 = 0.125
      row 1: sum dS = -0.2, l = 0.8, the cast gradient vanishes (0, 0): r_post = 0 (the row is kept),
             r_post,own undefined (the own-denominator statistic drops the row), kappa = +0.2 / 0.8 = 0.25
      row 2: l = 0: the row is outside the row set, everything undefined
      row 3: sum dS = 0.4, l = 1.6, sum dS' = -0.4, l' = 1.0: r_post = 0.25, r_post,own = 0.4,
             kappa = (-0.4 - 0.4) / 1.6 = -0.5 (signed)."""
    rs = np.array([0.5, -0.2, 0.0, 0.4]); ra = np.array([2.0, 0.8, 0.0, 1.6])
    ps = np.array([0.75, 0.0, 0.0, -0.4]); pa = np.array([3.0, 0.0, 0.0, 1.0])
    r_post, r_own, kappa = A.postcast_residuals(rs, ra, ps, pa)
    assert np.allclose(r_post[[0, 1, 3]], [0.375, 0.0, 0.25], atol=1e-15) and np.isnan(r_post[2])
    assert np.allclose(r_own[[0, 3]], [0.25, 0.4], atol=1e-15) and np.isnan(r_own[1]) and np.isnan(r_own[2])
    assert np.allclose(kappa[[0, 1, 3]], [0.125, 0.25, -0.5], atol=1e-15) and np.isnan(kappa[2])
    # the pre-cast statistic of the same equation
    r_pre = A.residual_ratio(rs, ra)
    assert np.allclose(r_pre[[0, 1, 3]], [0.25, 0.25, 0.25], atol=1e-15) and np.isnan(r_pre[2])


def test_one_rounding_tie_carries_a_percent_of_dq_on_the_stress_recipe():
    """Why the aligned-outlier stress case bounds dQ by 2e-2 instead of 5e-3.  On that recipe (scores with
    a standard deviation of ~70) rows are one-hot to ~1e-5, so a head's score gradient sits in a handful
    of elements.  One of them, row 566 / key 381 of head 2 at the size the GPU stress test uses, is the
    maximum of its 32-key block and lies 4e-6 (relative) from the midpoint of two E4M3 codes: an FP32
    evaluation of dS = P (dP - D) (approximate exp2, products rounded to 2^-24) is not accurate enough to
    land on the float64 side of that tie every time.  Landing on the other side changes that one code by
    one E4M3 step, which is 11 % of the row's dQ and 1.0e-2 of the whole dQ tensor in relative Frobenius
    norm -- twice the 5e-3 tolerance from a single element."""
    from paper_2609_37852_b200 import workloads
    w = workloads.WORKLOADS["gqa8k_outlier"].scaled(heads_q=4, heads_kv=2, seqlen=640, recipe="outlier_rope_aligned")
    q, k, v, dO = (x.float().numpy().astype(np.float64) for x in workloads.make_inputs(w))
    O, LSE = A.emu_forward(q, k, v, w.softmax_scale, True)
    D = A.emu_delta(q, k, v, dO, LSE, w.softmax_scale, True).astype(np.float32).astype(np.float64)
    dQ, dK, dV, rs, ra, t = A.emu_backward(q, k, v, dO, LSE, D, w.softmax_scale, True, return_internals=True)
    h, r, j = 2, 566, 381
    dS = t[(0, h)]["dS"]
    blk = dS[r, (j // 32) * 32:(j // 32) * 32 + 32]
    assert abs(dS[r, j]) == np.abs(blk).max()                        # it sets the block's scale ...
    e = int(np.ceil(np.log2(np.abs(blk).max() / 448.0)))             # ... 2^e, the smallest with amax * 2^-e <= 448
    y = abs(dS[r, j]) / 2.0 ** e
    assert 224.0 < y <= 448.0
    spacing = 2.0 ** (np.floor(np.log2(y)) - 3)                      # E4M3: 3 mantissa bits
    frac = (y / spacing) % 1.0
    tie_distance = abs(frac - 0.5) * spacing / y                     # relative to the value
    assert tie_distance < 1e-5, tie_distance
    assert t[(0, h)]["dS_q"][r, j] == np.floor(y / spacing) * spacing * 2.0 ** e     # float64 lands below the tie
    # the neighbouring code instead: one step of that element, through the key's operand row, into dQ
    kc = mxfp8.fake_quant(k[0, h // 2], 0)
    d_row = w.softmax_scale * spacing * 2.0 ** e * kc[j]
    assert 0.08 < np.linalg.norm(d_row) / np.linalg.norm(dQ[0, h, r]) < 0.14
    whole = np.linalg.norm(d_row) / np.linalg.norm(dQ)
    assert 8e-3 < whole < 1.3e-2, whole
    # such a tie needs the value within a few 1e-6 of a midpoint: one element in ~1e4, met here by the
    # largest element of its block in a head whose gradient lives in few elements
    worst = max(np.abs(t[(0, hh)]["dS"]).max() for hh in range(4))
    assert abs(dS[r, j]) > 0.3 * worst


def test_protected_dP_variant():
    """Protected dP (Appendix "Protected dP"): dP from BF16 operands, everything else FP8.  The matched
    correction built from that dP still zeroes the row sums (Eq. 5 only needs P normalised and one dP);
    with the stale correction the residual is the saved-output mismatch seen through BF16 dO and V."""
    q, k, v, dO, scale, causal = _setup_fp8(seed=23)
    O, LSE, fwd = A.emu_forward(q, k, v, scale, causal, exact_stats=True, return_internals=True)
    Dm = A.emu_delta(q, k, v, dO, LSE, scale, causal, exact_stats=True, dp_prec="bf16")
    Ds = A.emu_delta(q, k, v, dO, LSE, scale, causal, mode="stale", o=O, exact_stats=True)
    _, _, dVm, rsm, ram = A.emu_backward(q, k, v, dO, LSE, Dm, scale, causal, dp_prec="bf16")
    dQs, dKs, dVs, rss, ras, t = A.emu_backward(q, k, v, dO, LSE, Ds, scale, causal, dp_prec="bf16", return_internals=True)
    assert np.nanmedian(A.residual_ratio(rsm, ram)[..., 64:]) < 1e-12
    assert np.array_equal(dVm, dVs)                     # dV does not see dP
    _, _, dV8, _, _ = A.emu_backward(q, k, v, dO, LSE, Ds, scale, causal)
    assert np.array_equal(dVs, dV8)
    G = q.shape[1] // k.shape[1]
    for (b, h), tt in t.items():
        g = h // G
        assert np.abs(rss[b, h] - (Dm[b, h] - Ds[b, h])).max() < 1e-12
        dOb, Vb = mxfp8.round_bf16(dO[b, h]), mxfp8.round_bf16(v[b, g])
        assert np.array_equal(tt["dP"], dOb @ Vb.T)     # BF16 inputs: the rounding is the identity here
        Phat = fwd[(b, h)]["Ph"] / fwd[(b, h)]["l"][:, None]
        Vc = mxfp8.fake_quant(v[b, g], 0)
        want = (dOb * ((tt["P"] - Phat) @ Vb)).sum(-1) + (dOb * (Phat @ (Vb - Vc))).sum(-1) \
            + (dOb * (Phat @ Vc - O[b, h])).sum(-1)
        assert np.abs(rss[b, h] - want).max() < 1e-12
    # dK / dQ differ from the all-FP8 gradients only through dP
    dQ8, dK8, _, _, _ = A.emu_backward(q, k, v, dO, LSE, Ds, scale, causal)
    assert not np.array_equal(dQs, dQ8)
    assert np.linalg.norm(dQs - dQ8) / np.linalg.norm(dQ8) < 0.2


def test_subset_functions_agree_with_full_pass():
    q, k, v, dO, scale, causal = _setup_fp8(seed=14)
    O, LSE = A.emu_forward(q, k, v, scale, causal)
    D = A.emu_delta(q, k, v, dO, LSE, scale, causal)
    dQ, dK, dV, rs, ra = A.emu_backward(q, k, v, dO, LSE, D, scale, causal)
    rows = np.array([0, 5, 31, 32, 100, 127])
    O_r, L_r = A.emu_forward(q, k, v, scale, causal, rows=rows)
    assert np.array_equal(O_r, O[:, :, rows]) and np.array_equal(L_r, LSE[:, :, rows])
    D_r = A.emu_delta(q, k, v, dO, LSE, scale, causal, rows=rows)
    assert np.array_equal(D_r, D[:, :, rows])
    dq_r, rs_r, ra_r = A.emu_backward_rows(q, k, v, dO, LSE[0, 3], D[0, 3], scale, causal, 0, 3, rows)
    assert np.array_equal(dq_r, dQ[0, 3, rows]) and np.allclose(rs_r, rs[0, 3, rows], rtol=0, atol=1e-15)
    cols = np.arange(32, 96)
    dk_c, dv_c = A.emu_backward_cols(q, k, v, dO, LSE[0], D[0], scale, causal, 0, 1, cols)
    assert np.array_equal(dk_c, dK[0, 1, cols]) and np.array_equal(dv_c, dV[0, 1, cols])


def test_fp8_error_band_against_reference():
    """FP8 operands with three mantissa bits: the emulated path must sit a few
    percent from the unquantised one -- not at 1e-6 (nothing quantised) and not
    at 50 % (a wrong block axis or exponent)."""
    q, k, v, dO, scale, causal = _setup_fp8(seed=15, N=256)
    O_ref, LSE_ref = A.ref_forward(q, k, v, scale, causal)
    dQ_ref, dK_ref, dV_ref, _ = A.ref_backward(q, k, v, dO, scale, causal)
    O, LSE = A.emu_forward(q, k, v, scale, causal)
    D = A.emu_delta(q, k, v, dO, LSE, scale, causal)
    dQ, dK, dV, _, _ = A.emu_backward(q, k, v, dO, LSE, D, scale, causal)
    rel = lambda a, b: np.linalg.norm(a - b) / np.linalg.norm(b)
    for got, want in ((O, O_ref), (dQ, dQ_ref), (dK, dK_ref), (dV, dV_ref)):
        assert 3e-3 < rel(got, want) < 8e-2
    assert rel(LSE, LSE_ref) < 1e-2
    # BF16-operand mode is an order of magnitude closer
    O16, L16 = A.emu_forward(q, k, v, scale, causal, prec="bf16")
    assert rel(O16, O_ref) < 1e-2
