"""attn_fp8_fwd_noalloc: the forward for call sites that cannot allocate device memory.

Some users of this library sit inside a framework that owns every byte of device memory, or in
a service whose memory was partitioned at start-up, and may not call cudaMalloc (or anything
that allocates) where they invoke attention.  For them the library carries a small built-in
scratch array and this one extra entry point.  The test drives it through the C ABI twice in a
row -- the second call finds the array as the first left it -- and requires the outputs to be
bit-identical to those of attn_fp8_fwd with a caller workspace (the same tolerance as the
reproducibility tests: none).  It is collected last so that a failure here cannot hide others.
"""
import pytest
import torch

from paper_2609_37852_b200 import workloads

pytestmark = pytest.mark.gpu


def test_noalloc_forward_matches_forward_twice():
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=4, heads_kv=2, seqlen=640)
    q, k, v, dO = workloads.make_inputs(w)
    params = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                          w.softmax_scale)
    qq = B.attn_fp8_quantize(q.cuda(), want_col=False)
    kq = B.attn_fp8_quantize(k.cuda(), want_col=False)
    vq = B.attn_fp8_quantize(v.cuda(), want_row=False)
    o_ref, lse_ref, ws = B.attn_fp8_fwd(params, qq, kq, vq)
    B.attn_fp8_read_status(ws)
    for call in range(2):
        o = torch.full_like(o_ref, float("nan"))
        lse = torch.full_like(lse_ref, float("nan"))
        B.attn_fp8_fwd_noalloc(params, qq, kq, vq, o, lse)
        torch.cuda.synchronize()
        assert torch.equal(o, o_ref), f"call {call}: O differs"
        assert torch.equal(lse, lse_ref), f"call {call}: LSE differs"


def test_noalloc_forward_validates_like_forward():
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=4, heads_kv=2, seqlen=256)
    params = B.AttnParams(w.batch, w.seqlen, 3, 2, w.head_dim_qk, w.head_dim_v, w.causal, w.softmax_scale)
    empty = B.QTensor(shape=(1, 1, 1, 1))
    with pytest.raises(B.AttnFp8Error) as e:
        B.attn_fp8_fwd_noalloc(params, empty, empty, empty, torch.empty(1, device="cuda"), torch.empty(1, device="cuda"))
    assert e.value.status == 1
