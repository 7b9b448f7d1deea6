"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The oracle cannot finish these sizes in full, so outputs are sampled where each sample is
independent of the rest: query rows for O, LSE, D, dQ and the row statistics (a query row only
needs that row of Q, dO and all keys), and 32-key column groups for dK / dV (a key column only
needs that key and all queries; the oracle is fed the GPU's full LSE and D, which the row samples
have just checked).  Bounds are the ones of the small-size tests.
"""
import numpy as np
import pytest
import torch

from oracle import attention as A
from paper_2609_37852_b200 import workloads
from tests.util import rel_fro, to_np

pytestmark = pytest.mark.gpu


def _run(w, tensors, prec="mxfp8", strict_floor=0.999):
    from paper_2609_37852_b200 import binding as B
    params = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                          w.softmax_scale, precision=B.ATTN_PREC_BF16 if prec == "bf16" else B.ATTN_PREC_MXFP8)
    dev = [x.cuda() for x in tensors]
    if prec == "bf16":
        qq, kq, vq, dOq = (B.attn_fp8_prepare_bf16(x) for x in dev)
    else:                                     # as bench.py does: the four operands in one quantiser launch
        (qq, kq, vq, dOq), _ = B.attn_fp8_quantize_batch(dev)
    o, lse, ws = B.attn_fp8_fwd(params, qq, kq, vq)
    delta, ws = B.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, workspace=ws)
    dq, dk, dv, rs, ra, ws = B.attn_fp8_bwd(params, qq, kq, vq, dOq, lse, delta, diagnostics=True, workspace=ws)
    # once more through the instrumented entry point that also returns sum_j P |dP^| per row
    dq2, rs2, ra2, dust, ws = B.attn_fp8_bwd_dq_rowprobe(params, qq, kq, vq, dOq, lse, delta, workspace=ws)
    B.attn_fp8_read_status(ws)
    assert torch.equal(dq2, dq) and torch.equal(rs2, rs) and torch.equal(ra2, ra)
    got = dict(o=o, lse=lse, delta=delta, dq=dq, dk=dk, dv=dv, rs=rs, ra=ra, dust=dust)
    _assert_row_sum_invariant_on_every_row(got, strict_floor)
    return got


def _assert_row_sum_invariant_on_every_row(got, strict_floor):
    """|sum_j dS| <= 1e-5 sum_j |dS| + (ulp(LSE_i) + c_i) sum_j P |dP^| on EVERY row of every head.  The
    second term is what is left of delta_i (1 - sum_j P_ij): the FP32 storage of LSE (one ulp), and the FP32
    summation of the normaliser and of delta over the row's keys, c_i = 2^-20 up to 8192 keys and growing
    in proportion to the key count beyond (the worst case of a sum of 2^-24 roundings, one per 32-key block).
    It is all there is on rows whose dS vanishes analytically.

    The strict form without the second term is also counted, on rows i >= 64 with a non-zero
    sum_j |dS|: its share must reach ``strict_floor``, a floor per workload a little under what the
    kernels measure (1.0 on the diffuse recipes; 0.908 on the outlier-channel recipe and 0.990-0.996 on
    the heavy-tailed one, whose nearly one-hot rows have dS -> 0 and keep only the second term), and
    the median of the ratio must stay under 1e-5 everywhere."""
    rs, ra, dust, lse = (got[n].double() for n in ("rs", "ra", "dust", "lse"))
    a = got["lse"].abs()
    ulp = (torch.nextafter(a, torch.full_like(a, float("inf"))) - a).double()
    keys = torch.arange(1, rs.shape[-1] + 1, device=rs.device, dtype=torch.float64)
    c = 2.0 ** -20 * torch.clamp(keys / 8192.0, min=1.0)
    ok = rs.abs() <= 1e-5 * ra + (ulp + c) * dust
    assert bool(ok.all()), f"{int((~ok).sum())} of {ok.numel()} rows break the bound"
    rs64, ra64 = rs[..., 64:], ra[..., 64:]
    ratio = (rs64.abs() / ra64)[ra64 > 0]
    share = float((ratio <= 1e-5).double().mean())
    assert share >= strict_floor, f"strict form holds on {share:.4f} of the rows, floor {strict_floor}"
    assert float(ratio.median()) <= 1e-5


def _check_sampled(w, tensors, got, heads, rows, col_groups, seed, prec="mxfp8"):
    """``heads``: (batch, query head) pairs to sample; ``rows`` query rows per head; ``col_groups``
    number of 32-key groups per sampled KV head."""
    q, k, v, dO = tensors
    G = w.heads_q // w.heads_kv
    rng = np.random.default_rng(seed)
    N = w.seqlen
    for (b, h) in heads:
        g = h // G
        # one-head views (float64 copies of just what the oracle needs)
        qh, dOh = to_np(q[b:b + 1, h:h + 1]), to_np(dO[b:b + 1, h:h + 1])
        kh, vh = to_np(k[b:b + 1, g:g + 1]), to_np(v[b:b + 1, g:g + 1])
        r = np.unique(np.concatenate([[0, 1, 63, 64, 127, 128, N - 1], rng.integers(0, N, rows)]))
        O_or, LSE_or = A.emu_forward(qh, kh, vh, w.softmax_scale, w.causal, rows=r, prec=prec)
        assert rel_fro(to_np(got["o"][b, h])[r], O_or[0, 0]) <= 2e-3
        lse_gpu = to_np(got["lse"][b, h])
        assert rel_fro(lse_gpu[r], LSE_or[0, 0]) <= 2e-3
        assert np.abs(lse_gpu[r] - LSE_or[0, 0]).max() <= 2e-4 * max(1.0, np.abs(LSE_or).max())
        lse_full = lse_gpu[None, None]
        D_or = A.emu_delta(qh, kh, vh, dOh, lse_full, w.softmax_scale, w.causal, rows=r, prec=prec)
        d_gpu = to_np(got["delta"][b, h])
        assert rel_fro(d_gpu[r], D_or[0, 0]) <= 1e-4
        dq_or, rs_or, ra_or = A.emu_backward_rows(qh, kh, vh, dOh, lse_gpu, d_gpu, w.softmax_scale, w.causal, 0, 0, r,
                                                  prec=prec)
        assert rel_fro(to_np(got["dq"][b, h])[r], dq_or) <= 5e-3
        g_rs, g_ra = to_np(got["rs"][b, h])[r], to_np(got["ra"][b, h])[r]
        assert rel_fro(g_ra, ra_or) <= 1e-3
        # zero-row-sum invariant, same form as in the small-size test: 1e-5 of sum|dS| plus
        # |D| |1 - sum P| with |1 - sum P| <= one ulp of the FP32-stored LSE + 2^-20
        P = A._probabilities(A._fq(qh[0, 0], -1, prec), A._fq(kh[0, 0], -1, prec), lse_gpu, w.softmax_scale,
                             w.causal, r, np.arange(N))
        dust = (P * np.abs(A._fq(dOh[0, 0], -1, prec)[r] @ A._fq(vh[0, 0], -1, prec).T)).sum(-1)
        ulp = np.spacing(np.abs(lse_gpu[r]).astype(np.float32)).astype(np.float64)
        assert np.all(np.abs(g_rs) <= 1e-5 * g_ra + (ulp + 2.0 ** -20) * dust)
        assert rel_fro(to_np(got["dust"][b, h])[r], dust) <= 1e-3             # the kernel's own sum_j P |dP^|
        live = (g_ra > 0) & (r >= 64)
        r_pre = np.abs(g_rs[live]) / g_ra[live]
        print(f"\n[{w.name} b{b} h{h}] sampled r_pre median {np.median(r_pre):.2e} max {r_pre.max():.2e}")
        if w.recipe in ("iid", "qknorm", "plain"):
            assert np.median(r_pre) <= 1e-5
    # dK / dV: all query heads of the sampled KV heads, a few 32-key groups each
    for (b, g) in sorted({(b, h // G) for (b, h) in heads}):
        hs = slice(g * G, (g + 1) * G)
        qg, dOg = to_np(q[b:b + 1, hs]), to_np(dO[b:b + 1, hs])
        kg, vg = to_np(k[b:b + 1, g:g + 1]), to_np(v[b:b + 1, g:g + 1])
        lse_g, d_g = to_np(got["lse"][b, hs]), to_np(got["delta"][b, hs])
        starts = np.unique(np.concatenate([[0, N - 32], 32 * rng.integers(0, N // 32, col_groups)]))
        cols = np.concatenate([np.arange(s, s + 32) for s in starts])
        dk_or, dv_or = A.emu_backward_cols(qg, kg, vg, dOg, lse_g, d_g, w.softmax_scale, w.causal, 0, 0, cols, prec=prec)
        assert rel_fro(to_np(got["dk"][b, g])[cols], dk_or) <= 5e-3
        assert rel_fro(to_np(got["dv"][b, g])[cols], dv_or) <= 5e-3


def test_bench_workload_full_size_sampled():
    """gqa8k_outlier: B=1, 32/8 heads, N=8192, d=128 -- the workload bench.py times."""
    w = workloads.WORKLOADS["gqa8k_outlier"]
    tensors = workloads.make_inputs(w)
    got = _run(w, tensors, strict_floor=0.90)
    _check_sampled(w, tensors, got, heads=[(0, 0), (0, 13), (0, 31)], rows=48, col_groups=3, seed=1)


def test_gqa4k_full_size_sampled():
    """gqa4k: B=2, 16/4 heads, N=4096, d=128, QK-normalised."""
    w = workloads.WORKLOADS["gqa4k"]
    tensors = workloads.make_inputs(w)
    got = _run(w, tensors)
    _check_sampled(w, tensors, got, heads=[(0, 2), (1, 15)], rows=48, col_groups=3, seed=2)


def test_long_context_sampled():
    """long64k recipe at 16384 tokens (32/8 heads would need minutes of host-side generation at
    65536; the kernels have no size-dependent path beyond the tile loop counts)."""
    w = workloads.WORKLOADS["long64k"].scaled(seqlen=16384, heads_q=8, heads_kv=2)
    tensors = workloads.make_inputs(w)
    got = _run(w, tensors, strict_floor=0.99)
    _check_sampled(w, tensors, got, heads=[(0, 5)], rows=32, col_groups=2, seed=3)


def test_long_context_full_size_sampled():
    """long64k as configured: B=1, 32/8 heads, N=65536, d=128 (16384 work items per query-major kernel,
    2.7 GB of operands); about a minute of host-side input generation.  With ATTN_FP8_FULL_SAMPLE=1 four
    query heads of four KV groups are sampled: ~70 query rows each (O, LSE, D, dQ and the row
    statistics: 280 rows) and 18 groups of 32 keys of each of those KV heads (dK, dV over all four
    query heads of the group: 72 groups), five minutes in all; by default two heads, 39 rows
    and 10 key groups each."""
    import os
    full = os.environ.get("ATTN_FP8_FULL_SAMPLE") == "1"
    w = workloads.WORKLOADS["long64k"]
    tensors = workloads.make_inputs(w)
    got = _run(w, tensors, strict_floor=0.98)
    heads = [(0, 0), (0, 9), (0, 22), (0, 31)] if full else [(0, 0), (0, 31)]    # the cost is per sampled head
    _check_sampled(w, tensors, got, heads=heads, rows=64 if full else 32, col_groups=16 if full else 8, seed=3)


def test_mla_full_size_sampled():
    """mla8k: B=1, 16/16 heads, N=8192, qk head dim 192, v head dim 128."""
    w = workloads.WORKLOADS["mla8k"]
    tensors = workloads.make_inputs(w)
    got = _run(w, tensors)
    _check_sampled(w, tensors, got, heads=[(0, 3), (0, 15)], rows=32, col_groups=2, seed=4)


def test_d256_full_size_sampled():
    """gqa8k_d256: B=1, 8/2 heads, N=8192, head dim 256."""
    w = workloads.WORKLOADS["gqa8k_d256"]
    tensors = workloads.make_inputs(w)
    got = _run(w, tensors)
    _check_sampled(w, tensors, got, heads=[(0, 1), (0, 7)], rows=32, col_groups=2, seed=5)


def test_bench_workload_bf16_mode_sampled():
    """gqa8k_outlier in BF16 mode (the reference-point configuration bench.py --precision bf16 times)."""
    w = workloads.WORKLOADS["gqa8k_outlier"]
    tensors = workloads.make_inputs(w)
    got = _run(w, tensors, prec="bf16", strict_floor=0.90)
    _check_sampled(w, tensors, got, heads=[(0, 6), (0, 31)], rows=32, col_groups=2, seed=6, prec="bf16")


def test_wide_heads_bf16_mode_sampled():
    """The two wide-head configurations in BF16 mode at N = 8192 (their reference points): (192, 128)
    with 4 of the 16 heads and (256, 256) with 2 query heads on one KV head, enough for every tile
    count and pass of the full configuration."""
    w = workloads.WORKLOADS["mla8k"].scaled(heads_q=4, heads_kv=4)
    tensors = workloads.make_inputs(w)
    got = _run(w, tensors, prec="bf16")
    _check_sampled(w, tensors, got, heads=[(0, 2)], rows=24, col_groups=2, seed=7, prec="bf16")
    w = workloads.WORKLOADS["gqa8k_d256"].scaled(heads_q=2, heads_kv=1)
    tensors = workloads.make_inputs(w)
    got = _run(w, tensors, prec="bf16")
    _check_sampled(w, tensors, got, heads=[(0, 1)], rows=24, col_groups=2, seed=8, prec="bf16")
