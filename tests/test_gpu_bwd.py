"""attn_fp8_bwd_delta and attn_fp8_bwd against the oracle's emulated-FP8 backward."""
import numpy as np
import pytest
import torch

from oracle import attention as A
from paper_2609_37852_b200 import workloads
from tests.util import rel_fro, to_np, worst_row_error

pytestmark = pytest.mark.gpu

TOL_GRAD = 5e-3     # relative Frobenius error on dQ, dK, dV
TOL_DELTA = 1e-4    # relative Frobenius error on the row correction (FP32 sums of identical operands)


def run_all(w, q, k, v, dO, delta_mode=0, diagnostics=True, bf16=False):
    from paper_2609_37852_b200 import binding
    params = binding.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                                w.softmax_scale, delta_mode=delta_mode,
                                precision=binding.ATTN_PREC_BF16 if bf16 else binding.ATTN_PREC_MXFP8)
    prep = binding.attn_fp8_prepare_bf16 if bf16 else binding.attn_fp8_quantize
    qq, kq, vq, dOq = (prep(x.cuda()) for x in (q, k, v, dO))
    o, lse, ws = binding.attn_fp8_fwd(params, qq, kq, vq)
    binding.attn_fp8_read_status(ws)
    dO_bf = dO.cuda().to(torch.bfloat16)
    delta, ws = binding.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, dO_bf16=dO_bf, o_bf16=o)
    binding.attn_fp8_read_status(ws)
    dq, dk, dv, rs, ra, ws = binding.attn_fp8_bwd(params, qq, kq, vq, dOq, lse, delta, diagnostics=diagnostics)
    binding.attn_fp8_read_status(ws)
    return dict(o=o, lse=lse, delta=delta, dq=dq, dk=dk, dv=dv, rs=rs, ra=ra)


CASES = [
    ("tiny", {}),
    ("tiny", dict(causal=True, seqlen=384)),
    ("gqa4k", dict(batch=2, heads_q=4, heads_kv=2, seqlen=640)),
    ("gqa8k_outlier", dict(heads_q=4, heads_kv=1, seqlen=768)),
    ("long64k", dict(heads_q=2, heads_kv=1, seqlen=1152)),
]


@pytest.mark.parametrize("name,kw", CASES)
def test_matched_backward_matches_oracle(name, kw):
    w = workloads.WORKLOADS[name].scaled(**kw)
    q, k, v, dO = workloads.make_inputs(w)
    got = run_all(w, q, k, v, dO)
    qn, kn, vn, dOn = (to_np(x) for x in (q, k, v, dO))
    # the oracle consumes the GPU's saved LSE, exactly as the GPU backward does (the forward
    # test has already compared that LSE with the oracle's own)
    lse = to_np(got["lse"])
    D_or = A.emu_delta(qn, kn, vn, dOn, lse, w.softmax_scale, w.causal)
    assert rel_fro(to_np(got["delta"]), D_or) <= TOL_DELTA
    delta = to_np(got["delta"])
    dQ, dK, dV, rs, ra = A.emu_backward(qn, kn, vn, dOn, lse, delta, w.softmax_scale, w.causal)
    assert rel_fro(to_np(got["dq"]), dQ) <= TOL_GRAD
    assert rel_fro(to_np(got["dk"]), dK) <= TOL_GRAD
    assert rel_fro(to_np(got["dv"]), dV) <= TOL_GRAD
    # and no single row of substance is far off (ten times the tensor tolerance)
    for n_, ref in (("dq", dQ), ("dk", dK), ("dv", dV)):
        assert worst_row_error(to_np(got[n_]), ref) <= 10 * TOL_GRAD, n_
    # pre-cast row statistics
    assert rel_fro(to_np(got["ra"]), ra) <= 1e-3
    # zero-row-sum invariant on the GPU's own statistics: |sum_j dS| <= 1e-5 sum_j |dS|, plus the
    # allowance |D| * |1 - sum_j P| with |1 - sum_j P| <= one ulp of the FP32-stored LSE_i + 2^-20
    # (storage of LSE, FP32 summation of l, approximate exp2); rows that see a single key have
    # dS = 0 analytically and only that dust
    g_rs, g_ra = to_np(got["rs"]), to_np(got["ra"])
    dust = np.zeros_like(g_rs)
    for b in range(w.batch):
        for h in range(w.heads_q):
            gidx = h // (w.heads_q // w.heads_kv)
            from oracle import mxfp8
            P = A._probabilities(mxfp8.fake_quant(qn[b, h]), mxfp8.fake_quant(kn[b, gidx]), lse[b, h],
                                 w.softmax_scale, w.causal, np.arange(w.seqlen), np.arange(w.seqlen))
            dP = mxfp8.fake_quant(dOn[b, h]) @ mxfp8.fake_quant(vn[b, gidx]).T
            dust[b, h] = (P * np.abs(dP)).sum(-1)
    ulp_lse = np.spacing(np.abs(lse).astype(np.float32)).astype(np.float64)
    assert np.all(np.abs(g_rs) <= 1e-5 * g_ra + (ulp_lse + 2.0 ** -20) * dust)
    # the strict per-row form, on rows i >= 64 with a non-zero denominator (the paper's row set):
    # it holds for (almost) every row unless attention is nearly one-hot, where sum_j |dS| itself
    # collapses towards the dust; the median stays at FP32 rounding level in every workload
    live = g_ra[..., 64:] > 0
    r_pre = np.abs(g_rs[..., 64:][live]) / g_ra[..., 64:][live]
    print(f"\n[{name}] r_pre median {np.median(r_pre):.3e} p99 {np.quantile(r_pre, 0.99):.3e} max {r_pre.max():.3e} "
          f"strict-ok {np.mean(r_pre <= 1e-5):.4f}")
    assert np.median(r_pre) <= 1e-5
    if w.recipe in ("iid", "qknorm"):
        assert np.mean(r_pre <= 1e-5) > 0.999


def _check_backward(w, q, k, v, dO, got, prec):
    qn, kn, vn, dOn = (to_np(x) for x in (q, k, v, dO))
    lse = to_np(got["lse"])
    D_or = A.emu_delta(qn, kn, vn, dOn, lse, w.softmax_scale, w.causal, prec=prec)
    assert rel_fro(to_np(got["delta"]), D_or) <= TOL_DELTA
    delta = to_np(got["delta"])
    dQ, dK, dV, rs, ra = A.emu_backward(qn, kn, vn, dOn, lse, delta, w.softmax_scale, w.causal, prec=prec)
    assert rel_fro(to_np(got["dq"]), dQ) <= TOL_GRAD
    assert rel_fro(to_np(got["dk"]), dK) <= TOL_GRAD
    assert rel_fro(to_np(got["dv"]), dV) <= TOL_GRAD
    for n_, ref in (("dq", dQ), ("dk", dK), ("dv", dV)):
        assert worst_row_error(to_np(got[n_]), ref) <= 10 * TOL_GRAD, n_
    assert rel_fro(to_np(got["ra"]), ra) <= 1e-3
    g_rs, g_ra = to_np(got["rs"]), to_np(got["ra"])
    live = g_ra[..., 64:] > 0
    r_pre = np.abs(g_rs[..., 64:][live]) / g_ra[..., 64:][live]
    print(f"\n[{w.name} {prec}] r_pre median {np.median(r_pre):.3e} max {r_pre.max():.3e}")
    assert np.median(r_pre) <= 1e-5


@pytest.mark.parametrize("name,kw", [
    ("mla8k", dict(heads_q=2, heads_kv=2, seqlen=640)),                  # qk 192 / v 128
    ("gqa8k_d256", dict(heads_q=4, heads_kv=2, seqlen=640)),             # 256 / 256
    ("gqa8k_d256", dict(heads_q=2, heads_kv=1, seqlen=384, causal=False)),
])
def test_backward_wide_heads_matches_oracle(name, kw):
    """Head dims above 128: dQ columns split over CTAs, dV and dK in separate key-major passes."""
    w = workloads.WORKLOADS[name].scaled(**kw)
    q, k, v, dO = workloads.make_inputs(w)
    got = run_all(w, q, k, v, dO)
    _check_backward(w, q, k, v, dO, got, "mxfp8")


@pytest.mark.parametrize("name,kw", [
    ("tiny", {}),
    ("tiny", dict(causal=True, seqlen=384)),
    ("gqa4k", dict(batch=2, heads_q=4, heads_kv=2, seqlen=640)),
    ("gqa8k_outlier", dict(heads_q=4, heads_kv=1, seqlen=768)),
    ("mla8k", dict(heads_q=4, heads_kv=2, seqlen=640)),              # (192, 128): dV and dK in separate passes
    ("gqa8k_d256", dict(heads_q=4, heads_kv=2, seqlen=640)),         # (256, 256): dK in two column passes
    ("gqa8k_d256", dict(heads_q=2, heads_kv=2, seqlen=384, causal=False)),
])
def test_backward_bf16_mode_matches_oracle(name, kw):
    """BF16 mode against the oracle's BF16-operand path."""
    w = workloads.WORKLOADS[name].scaled(**kw)
    q, k, v, dO = workloads.make_inputs(w)
    got = run_all(w, q, k, v, dO, bf16=True)
    _check_backward(w, q, k, v, dO, got, "bf16")


def test_stale_mode_changes_only_delta_dq_dk():
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=4, heads_kv=2, seqlen=512)
    q, k, v, dO = workloads.make_inputs(w)
    m = run_all(w, q, k, v, dO, delta_mode=0)
    s = run_all(w, q, k, v, dO, delta_mode=1)
    assert torch.equal(m["o"], s["o"]) and torch.equal(m["lse"], s["lse"]) and torch.equal(m["dv"], s["dv"])
    assert not torch.equal(m["delta"], s["delta"])
    assert not torch.equal(m["dq"], s["dq"]) and not torch.equal(m["dk"], s["dk"])
    qn, kn, vn, dOn = (to_np(x) for x in (q, k, v, dO))
    D_stale = A.emu_delta(qn, kn, vn, dOn, to_np(s["lse"]), w.softmax_scale, w.causal, mode="stale", o=to_np(s["o"]))
    assert rel_fro(to_np(s["delta"]), D_stale) <= 1e-5
    dQ, dK, dV, rs, ra = A.emu_backward(qn, kn, vn, dOn, to_np(s["lse"]), to_np(s["delta"]), w.softmax_scale, w.causal)
    assert rel_fro(to_np(s["dq"]), dQ) <= TOL_GRAD and rel_fro(to_np(s["dk"]), dK) <= TOL_GRAD
    # stale residual is orders of magnitude above the matched one
    r_m = np.abs(to_np(m["rs"])) / to_np(m["ra"])
    r_s = np.abs(to_np(s["rs"])) / to_np(s["ra"])
    assert np.nanmedian(r_s[..., 64:]) >= 100 * np.nanmedian(r_m[..., 64:])
    assert rel_fro(to_np(s["rs"]), rs) <= 1e-2


def test_consistent_dO_mode():
    """Consistent dO: the saved-output shortcut with the FP8 dO operand; residual between stale and matched."""
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=4, heads_kv=2, seqlen=512)
    q, k, v, dO = workloads.make_inputs(w)
    m = run_all(w, q, k, v, dO, delta_mode=0)
    s = run_all(w, q, k, v, dO, delta_mode=1)
    c = run_all(w, q, k, v, dO, delta_mode=2)
    assert torch.equal(m["o"], c["o"]) and torch.equal(m["lse"], c["lse"]) and torch.equal(m["dv"], c["dv"])
    qn, kn, vn, dOn = (to_np(x) for x in (q, k, v, dO))
    D_c = A.emu_delta(qn, kn, vn, dOn, to_np(c["lse"]), w.softmax_scale, w.causal, mode="consistent", o=to_np(c["o"]))
    assert rel_fro(to_np(c["delta"]), D_c) <= 1e-5
    dQ, dK, dV, rs, ra = A.emu_backward(qn, kn, vn, dOn, to_np(c["lse"]), to_np(c["delta"]), w.softmax_scale, w.causal)
    assert rel_fro(to_np(c["dq"]), dQ) <= TOL_GRAD and rel_fro(to_np(c["dk"]), dK) <= TOL_GRAD
    med = lambda d: np.nanmedian((np.abs(to_np(d["rs"])) / to_np(d["ra"]))[..., 64:])
    print(f"\nmedian r_pre: stale {med(s):.3e} consistent {med(c):.3e} matched {med(m):.3e}")
    assert med(s) > med(c) > 100 * med(m)


@pytest.mark.parametrize("bf16", [False, True])
def test_postcast_statistics(bf16):
    """Post-cast probe: row sums of the cast score gradient the dQ matmul consumes."""
    from paper_2609_37852_b200 import binding
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=4, heads_kv=2, seqlen=512)
    q, k, v, dO = workloads.make_inputs(w)
    prec = "bf16" if bf16 else "mxfp8"
    params = binding.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                                w.softmax_scale, precision=binding.ATTN_PREC_BF16 if bf16 else binding.ATTN_PREC_MXFP8)
    prep = binding.attn_fp8_prepare_bf16 if bf16 else binding.attn_fp8_quantize
    qq, kq, vq, dOq = (prep(x.cuda()) for x in (q, k, v, dO))
    o, lse, ws = binding.attn_fp8_fwd(params, qq, kq, vq)
    delta, ws = binding.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, workspace=ws)
    dq0, rs0, ra0, ws = binding.attn_fp8_bwd_dq(params, qq, kq, vq, dOq, lse, delta, diagnostics=True, workspace=ws)
    dq, rs, ra, ps, pa, ws = binding.attn_fp8_bwd_dq_postcast(params, qq, kq, vq, dOq, lse, delta, workspace=ws)
    binding.attn_fp8_read_status(ws)
    assert torch.equal(dq, dq0) and torch.equal(rs, rs0) and torch.equal(ra, ra0)
    qn, kn, vn, dOn = (to_np(x) for x in (q, k, v, dO))
    for h in range(w.heads_q):
        ps_or, pa_or = A.postcast_row_sums(qn, kn, vn, dOn, to_np(lse[0, h]), to_np(delta[0, h]), w.softmax_scale,
                                           w.causal, prec=prec, b=0, h=h)
        assert rel_fro(to_np(pa[0, h]), pa_or) <= 1e-3
        # a code that rounds the other way moves a row sum by one E4M3 step of one element
        assert np.abs(to_np(ps[0, h]) - ps_or).max() <= 2e-2 * np.abs(pa_or).max()
        assert rel_fro(to_np(ps[0, h]), ps_or) <= (0.2 if bf16 else 5e-2)
    r_post, r_own, kappa = A.postcast_residuals(to_np(rs), to_np(ra), to_np(ps), to_np(pa))
    r_pre = A.residual_ratio(to_np(rs), to_np(ra))
    print(f"\n[{prec}] median r_pre {np.nanmedian(r_pre[..., 64:]):.2e} r_post {np.nanmedian(r_post[..., 64:]):.2e} "
          f"r_post_own {np.nanmedian(r_own[..., 64:]):.2e} mean kappa {np.nanmean(kappa[..., 64:]):.2e}")
    assert np.nanmedian(r_post[..., 64:]) > 10 * np.nanmedian(r_pre[..., 64:])
    assert np.nanmax(np.abs(kappa)) <= 2.0 ** -4


@pytest.mark.parametrize("name,kw,delta_mode", [
    ("gqa4k", dict(batch=1, heads_q=4, heads_kv=2, seqlen=640), 1),      # the paper's pairing: stale correction
    ("gqa4k", dict(batch=1, heads_q=4, heads_kv=2, seqlen=384), 0),      # matched correction from the protected dP
    ("tiny", dict(causal=True, seqlen=384), 1),                          # d = 64
])
def test_protected_dP_precision(name, kw, delta_mode):
    """dP = dO V^T from BF16 operands, the other products FP8 (paper Appendix "Protected dP")."""
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS[name].scaled(**kw)
    q, k, v, dO = workloads.make_inputs(w)
    base = dict(batch=w.batch, seqlen=w.seqlen, heads_q=w.heads_q, heads_kv=w.heads_kv, head_dim_qk=w.head_dim_qk,
                head_dim_v=w.head_dim_v, causal=w.causal, softmax_scale=w.softmax_scale, delta_mode=delta_mode)
    p8 = B.AttnParams(**base)
    pp = B.AttnParams(precision=B.ATTN_PREC_MXFP8_PROTECTED_DP, **base)
    qq, kq, vq, dOq = (B.attn_fp8_quantize(x.cuda()) for x in (q, k, v, dO))
    v_bf, dO_bf = v.cuda().to(torch.bfloat16), dO.cuda().to(torch.bfloat16)
    vp, dOp = B.protect_dp_operand(vq, v_bf), B.protect_dp_operand(dOq, dO_bf)
    o, lse, ws = B.attn_fp8_fwd(pp, qq, kq, vq)
    o8, lse8, _ = B.attn_fp8_fwd(p8, qq, kq, vq)
    assert torch.equal(o, o8) and torch.equal(lse, lse8)                 # the forward does not know about it
    delta, ws = B.attn_fp8_bwd_delta(pp, qq, kq, vp, dOp, lse, dO_bf16=dO_bf, o_bf16=o, workspace=ws)
    dq, dk, dv, rs, ra, ws = B.attn_fp8_bwd(pp, qq, kq, vp, dOp, lse, delta, diagnostics=True, workspace=ws)
    B.attn_fp8_read_status(ws)
    qn, kn, vn, dOn = (to_np(x) for x in (q, k, v, dO))
    lse_n, delta_n = to_np(lse), to_np(delta)
    if delta_mode == 0:
        D = A.emu_delta(qn, kn, vn, dOn, lse_n, w.softmax_scale, w.causal, dp_prec="bf16")
        assert rel_fro(delta_n, D) <= TOL_DELTA
    dQ, dK, dV, rs_or, ra_or = A.emu_backward(qn, kn, vn, dOn, lse_n, delta_n, w.softmax_scale, w.causal, dp_prec="bf16")
    assert rel_fro(to_np(dq), dQ) <= TOL_GRAD and rel_fro(to_np(dk), dK) <= TOL_GRAD and rel_fro(to_np(dv), dV) <= TOL_GRAD
    assert rel_fro(to_np(ra), ra_or) <= 1e-3
    r_pre = A.residual_ratio(to_np(rs), to_np(ra))[..., 64:]
    if delta_mode == 0:
        assert np.nanmedian(r_pre) <= 1e-5
    else:
        assert np.nanmedian(r_pre) > 1e-5                                # the stale residual remains
        assert rel_fro(to_np(rs), rs_or) <= 1e-2
    # it differs from the all-FP8 gradient pass only through dP
    dq8, dk8, dv8, _, _, _ = B.attn_fp8_bwd(p8, qq, kq, vq, dOq, lse, delta)
    assert torch.equal(dv, dv8) and not torch.equal(dq, dq8)


def test_backward_is_reproducible():
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=4, heads_kv=2, seqlen=512)
    q, k, v, dO = workloads.make_inputs(w)
    a = run_all(w, q, k, v, dO)
    b = run_all(w, q, k, v, dO)
    for key in ("delta", "dq", "dk", "dv", "rs", "ra"):
        assert torch.equal(a[key], b[key]), key


@pytest.mark.parametrize("name,kw", [
    ("gqa4k", dict(batch=1, heads_q=4, heads_kv=2, seqlen=384)),
    ("gqa8k_outlier", dict(heads_q=4, heads_kv=2, seqlen=512)),
])
def test_whole_chain_against_an_oracle_that_never_sees_gpu_values(name, kw):
    """The other backward tests hand the GPU's saved LSE and D to the oracle's gradient pass (as the GPU
    gradient pass gets them).  Here the oracle runs its own chain end to end -- forward, its LSE into its
    correction pass, its D into its gradient pass -- and the GPU's outputs are compared with that."""
    w = workloads.WORKLOADS[name].scaled(**kw)
    q, k, v, dO = workloads.make_inputs(w)
    got = run_all(w, q, k, v, dO)
    qn, kn, vn, dOn = (to_np(x) for x in (q, k, v, dO))
    O, LSE = A.emu_forward(qn, kn, vn, w.softmax_scale, w.causal)
    D = A.emu_delta(qn, kn, vn, dOn, LSE, w.softmax_scale, w.causal)
    dQ, dK, dV, _, _ = A.emu_backward(qn, kn, vn, dOn, LSE, D, w.softmax_scale, w.causal)
    assert rel_fro(to_np(got["o"]), O) <= 2e-3 and rel_fro(to_np(got["lse"]), LSE) <= 2e-3
    assert rel_fro(to_np(got["delta"]), D) <= TOL_DELTA
    for n_, ref in (("dq", dQ), ("dk", dK), ("dv", dV)):
        assert rel_fro(to_np(got[n_]), ref) <= TOL_GRAD, n_
        assert worst_row_error(to_np(got[n_]), ref) <= 10 * TOL_GRAD, n_


def test_bench_residual_statistics_match_the_oracle_helpers():
    """bench.py forms r_pre, r_post, kappa and c_K from the instrumented dQ pass with torch; the same
    numbers from the oracle's (pinned) helpers, on the same kernel outputs."""
    import bench
    from paper_2609_37852_b200 import binding
    w = workloads.WORKLOADS["gqa8k_outlier"].scaled(heads_q=4, heads_kv=2, seqlen=512)
    q, k, v, dO = workloads.make_inputs(w)
    params = binding.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                                w.softmax_scale)
    qq, kq, vq, dOq = (binding.attn_fp8_quantize(x.cuda()) for x in (q, k, v, dO))
    o, lse, ws = binding.attn_fp8_fwd(params, qq, kq, vq)
    delta, ws = binding.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, workspace=ws)
    dq, rs, ra, ps, pa, ws = binding.attn_fp8_bwd_dq_postcast(params, qq, kq, vq, dOq, lse, delta, workspace=ws)
    dk, dv, ws = binding.attn_fp8_bwd_dkdv(params, qq, kq, vq, dOq, lse, delta, workspace=ws)
    binding.attn_fp8_read_status(ws)
    stats = bench.residual_statistics(rs, ra, ps, dk)
    rsn, ran, psn, pan = (to_np(t)[..., 64:].ravel() for t in (rs, ra, ps, pa))
    live = ran > 0
    r_post, r_own, kappa = A.postcast_residuals(rsn[live], ran[live], psn[live], pan[live])
    r_pre = A.residual_ratio(rsn[live], ran[live])
    assert np.isclose(stats["r_pre_median"], np.median(r_pre), rtol=1e-12, atol=0)
    assert np.isclose(stats["r_post_median"], np.median(r_post), rtol=1e-12, atol=0)
    assert np.isclose(stats["kappa_mean"], np.mean(kappa), rtol=1e-9, atol=1e-18)
    assert np.isclose(stats["key_common_mode_median"], np.median(A.key_common_mode(to_np(dk))), rtol=1e-12, atol=0)
    assert np.isclose(stats["strict_ok_frac"], np.mean(r_pre <= 1e-5), rtol=0, atol=1e-12)
