"""Ragged sequence lengths: fewer tokens than a multiple of 128.

The caller pads Q, K, V and dO with zero rows to the next multiple of 128 and says how many keys are
real (attn_params_t.keys_valid).  Without the causal mask the kernels mask the padded keys; under the
causal mask real queries never see them.  The oracle runs the unpadded problem (padded only to the next
multiple of 32 where its block quantiser needs it, which under the causal mask changes nothing for the
real tokens), with its own LSE and correction all the way, and the real rows of every output are
compared; the gradient rows of padded keys must be exactly zero.
"""
import numpy as np
import pytest
import torch

from oracle import attention as A
from paper_2609_37852_b200 import workloads
from tests.util import rel_fro, to_np, worst_row_error

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,kw,n_real,bf16", [
    ("gqa4k", dict(batch=1, heads_q=4, heads_kv=2, causal=True), 300, False),     # ends inside a 32-token block
    ("gqa4k", dict(batch=2, heads_q=4, heads_kv=2, causal=True), 416, False),
    ("gqa4k", dict(batch=1, heads_q=4, heads_kv=2, causal=False), 320, False),    # padded keys masked in every row
    ("tiny", dict(batch=1, heads_q=2, heads_kv=1, causal=False), 224, False),     # d = 64, FP32 source
    ("tiny", dict(batch=1, heads_q=2, heads_kv=1, causal=False), 32, False),      # a single block of real keys
    ("mla8k", dict(heads_q=2, heads_kv=2, causal=False), 352, False),             # wide heads: (192, 128)
    ("gqa8k_d256", dict(heads_q=2, heads_kv=1, causal=False), 160, False),
    ("gqa4k", dict(batch=1, heads_q=2, heads_kv=1, causal=False), 160, True),     # BF16 mode
    ("gqa8k_outlier", dict(heads_q=4, heads_kv=1, causal=True), 200, True),
])
def test_ragged_lengths_match_the_unpadded_oracle(name, kw, n_real, bf16):
    from paper_2609_37852_b200 import binding as B
    n_alloc = -(-n_real // 128) * 128
    w = workloads.WORKLOADS[name].scaled(seqlen=n_alloc, **kw)
    real = [x[:, :, :n_real].contiguous() for x in workloads.make_inputs(w)]       # the caller's tensors
    if bf16:
        real = [x.to(torch.bfloat16) for x in real]
    padded = [B.pad_tokens(x.cuda()) for x in real]
    assert all(x.shape[2] == n_alloc for x in padded)
    params = B.AttnParams(w.batch, n_alloc, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                          w.softmax_scale, precision=B.ATTN_PREC_BF16 if bf16 else B.ATTN_PREC_MXFP8,
                          keys_valid=n_real)
    prep = B.attn_fp8_prepare_bf16 if bf16 else B.attn_fp8_quantize
    qq, kq, vq, dOq = (prep(x) for x in padded)
    o, lse, ws = B.attn_fp8_fwd(params, qq, kq, vq)
    delta, ws = B.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, workspace=ws)
    dq, dk, dv, rs, ra, ws = B.attn_fp8_bwd(params, qq, kq, vq, dOq, lse, delta, diagnostics=True, workspace=ws)
    B.attn_fp8_read_status(ws)
    for t in (o, lse, delta, dq, dk, dv):
        assert bool(torch.isfinite(t.float()).all())
    # gradient rows of padded keys
    assert float(dk[:, :, n_real:].float().abs().max()) == 0.0 if n_real < n_alloc else True
    assert float(dv[:, :, n_real:].float().abs().max()) == 0.0 if n_real < n_alloc else True

    # the oracle on the real tokens (under the causal mask: zero rows up to the next multiple of 32)
    n_or = -(-n_real // 32) * 32
    assert w.causal or n_or == n_real
    prec = "bf16" if bf16 else "mxfp8"
    qn, kn, vn, dOn = (to_np(B.pad_tokens(x, 32)) for x in real)
    O, LSE = A.emu_forward(qn, kn, vn, w.softmax_scale, w.causal, prec=prec)
    D = A.emu_delta(qn, kn, vn, dOn, LSE, w.softmax_scale, w.causal, prec=prec)
    dQ, dK, dV, _, _ = A.emu_backward(qn, kn, vn, dOn, LSE, D, w.softmax_scale, w.causal, prec=prec)
    v = slice(0, n_real)
    assert rel_fro(to_np(o)[:, :, v], O[:, :, v]) <= 2e-3
    assert rel_fro(to_np(lse)[:, :, v], LSE[:, :, v]) <= 2e-3
    assert rel_fro(to_np(delta)[:, :, v], D[:, :, v]) <= 1e-3          # the oracle's own LSE, not the kernel's
    for got, want, n_ in ((dq, dQ, "dq"), (dk, dK, "dk"), (dv, dV, "dv")):
        assert rel_fro(to_np(got)[:, :, v], want[:, :, v]) <= 5e-3, n_
        assert worst_row_error(to_np(got)[:, :, v], want[:, :, v]) <= 5e-2, n_
    # the zero-row-sum invariant on the real rows
    r = (to_np(rs)[:, :, v].__abs__() / np.maximum(to_np(ra)[:, :, v], 1e-300))[..., min(64, n_real // 2):]
    assert float(np.median(r)) <= 1e-5


def test_keys_valid_is_validated():
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=2, heads_kv=1, seqlen=256)
    q, k, v, _ = (x.cuda() for x in workloads.make_inputs(w))
    qq, kq, vq = B.attn_fp8_quantize(q), B.attn_fp8_quantize(k), B.attn_fp8_quantize(v)
    for bad in (128, 257, -1):                  # a whole tile of padding, more keys than allocated, negative
        with pytest.raises(B.AttnFp8Error) as e:
            B.attn_fp8_fwd(B.AttnParams(1, 256, 2, 1, 128, 128, False, 0.1, keys_valid=bad), qq, kq, vq)
        assert e.value.status == 1, bad
    o_all, lse_all, ws = B.attn_fp8_fwd(B.AttnParams(1, 256, 2, 1, 128, 128, False, 0.1), qq, kq, vq)
    o_256, lse_256, ws = B.attn_fp8_fwd(B.AttnParams(1, 256, 2, 1, 128, 128, False, 0.1, keys_valid=256), qq, kq, vq)
    B.attn_fp8_read_status(ws)
    assert torch.equal(o_all, o_256) and torch.equal(lse_all, lse_256)
