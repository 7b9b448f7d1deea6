"""attn_fp8_fwd against the oracle's emulated-FP8 forward."""
import numpy as np
import pytest
import torch

from oracle import attention as A
from paper_2609_37852_b200 import workloads
from tests.util import rel_fro, to_np, worst_row_error

pytestmark = pytest.mark.gpu

TOL_O = 2e-3      # relative Frobenius error on O and LSE


def run_fwd(w, q, k, v, bf16=False):
    from paper_2609_37852_b200 import binding
    params = binding.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                                w.softmax_scale, precision=binding.ATTN_PREC_BF16 if bf16 else binding.ATTN_PREC_MXFP8)
    prep = binding.attn_fp8_prepare_bf16 if bf16 else binding.attn_fp8_quantize
    qq = prep(q.cuda(), want_col=False)
    kq = prep(k.cuda(), want_col=False)
    vq = prep(v.cuda(), want_row=False)
    o, lse, ws = binding.attn_fp8_fwd(params, qq, kq, vq)
    binding.attn_fp8_read_status(ws)
    return o, lse


@pytest.mark.parametrize("name,kw", [
    ("tiny", {}),
    ("tiny", dict(causal=True, seqlen=384)),
    ("gqa4k", dict(batch=2, heads_q=4, heads_kv=2, seqlen=640)),
    ("gqa8k_outlier", dict(heads_q=4, heads_kv=2, seqlen=1024)),
    ("long64k", dict(heads_q=2, heads_kv=1, seqlen=1152)),
])
def test_forward_matches_oracle(name, kw):
    w = workloads.WORKLOADS[name].scaled(**kw)
    q, k, v, dO = workloads.make_inputs(w)
    o, lse = run_fwd(w, q, k, v)
    O_or, LSE_or = A.emu_forward(to_np(q), to_np(k), to_np(v), w.softmax_scale, w.causal)
    assert rel_fro(to_np(o), O_or) <= TOL_O
    assert rel_fro(to_np(lse), LSE_or) <= TOL_O
    assert np.abs(to_np(lse) - LSE_or).max() <= 2e-4 * max(1.0, np.abs(LSE_or).max())
    assert worst_row_error(to_np(o), O_or) <= 10 * TOL_O           # no single output row of substance far off


@pytest.mark.parametrize("name,kw", [
    ("mla8k", dict(heads_q=2, heads_kv=2, seqlen=640)),                  # qk 192 / v 128
    ("gqa8k_d256", dict(heads_q=4, heads_kv=2, seqlen=640)),             # 256 / 256
    ("gqa8k_d256", dict(heads_q=2, heads_kv=1, seqlen=384, causal=False)),
])
def test_forward_wide_heads_matches_oracle(name, kw):
    """Head dims above 128: two 128-byte chunks per operand row, two scale tiles per row tile."""
    w = workloads.WORKLOADS[name].scaled(**kw)
    q, k, v, dO = workloads.make_inputs(w)
    o, lse = run_fwd(w, q, k, v)
    O_or, LSE_or = A.emu_forward(to_np(q), to_np(k), to_np(v), w.softmax_scale, w.causal)
    assert rel_fro(to_np(o), O_or) <= TOL_O
    assert rel_fro(to_np(lse), LSE_or) <= TOL_O


@pytest.mark.parametrize("name,kw", [
    ("tiny", {}),
    ("tiny", dict(causal=True, seqlen=384)),
    ("gqa4k", dict(batch=2, heads_q=4, heads_kv=2, seqlen=640)),
    ("gqa8k_outlier", dict(heads_q=4, heads_kv=2, seqlen=1024)),
])
def test_forward_bf16_mode_matches_oracle(name, kw):
    """BF16 mode against the oracle's BF16-operand path (same dataflow, rounding instead of block scaling)."""
    w = workloads.WORKLOADS[name].scaled(**kw)
    q, k, v, dO = workloads.make_inputs(w)
    o, lse = run_fwd(w, q, k, v, bf16=True)
    O_or, LSE_or = A.emu_forward(to_np(q), to_np(k), to_np(v), w.softmax_scale, w.causal, prec="bf16")
    assert rel_fro(to_np(o), O_or) <= TOL_O
    assert rel_fro(to_np(lse), LSE_or) <= TOL_O


def test_forward_is_reproducible():
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=4, heads_kv=2, seqlen=512)
    q, k, v, dO = workloads.make_inputs(w)
    o1, l1 = run_fwd(w, q, k, v)
    o2, l2 = run_fwd(w, q, k, v)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
