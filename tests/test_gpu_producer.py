"""attn_fp8_quantize_fused against the producer oracle (bit-exact) and end to end through attention."""
import numpy as np
import pytest
import torch

from oracle import attention as A
from oracle import mxfp8
from oracle import producer as P
from paper_2609_37852_b200 import workloads
from tests.util import rel_fro, to_np

pytestmark = pytest.mark.gpu


def _codes_match(qt, y, B, H, N, d):
    from paper_2609_37852_b200 import binding
    rc, rs = mxfp8.quantize(y, axis=-1)
    cc, cs = mxfp8.quantize(np.swapaxes(y, -1, -2), axis=-1)
    assert np.array_equal(qt.row_codes.cpu().numpy(), rc)
    assert np.array_equal(binding.unpack_scales(qt.row_scales, B, H, N, d).cpu().numpy(), rs)
    assert np.array_equal(qt.col_codes.cpu().numpy(), cc)
    assert np.array_equal(binding.unpack_scales(qt.col_scales, B, H, d, N).cpu().numpy(), cs)


@pytest.mark.parametrize("d", [64, 128, 192])
def test_fused_producer_bit_exact(d):
    from paper_2609_37852_b200 import binding
    B, H, N = 2, 3, 384
    g = torch.Generator().manual_seed(100 + d)
    x = (torch.randn((B, H, N, d), generator=g) + 0.75).to(torch.bfloat16)          # non-zero mean
    cos, sin = P.rope_tables(N, d)
    tc, ts = torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda()
    xn = to_np(x)
    tau = d ** -0.5
    # query side: rotary embedding + tau fold
    qt, mean = binding.attn_fp8_quantize_fused(x.cuda(), tc, ts, scale=tau)
    assert mean is None
    y, _ = P.fused_operand(xn, cos, sin, scale=np.float32(tau))
    _codes_match(qt, y, B, H, N, d)
    # key side: rotary embedding + centering
    kt, mean = binding.attn_fp8_quantize_fused(x.cuda(), tc, ts, center=True)
    y, m = P.fused_operand(xn, cos, sin, center=True)
    assert np.array_equal(to_np(mean), m)
    _codes_match(kt, y, B, H, N, d)
    # nothing requested: the plain quantiser
    pt, _ = binding.attn_fp8_quantize_fused(x.cuda())
    ref = binding.attn_fp8_quantize(x.cuda())
    for a, b in ((pt.row_codes, ref.row_codes), (pt.row_scales, ref.row_scales), (pt.col_codes, ref.col_codes),
                 (pt.col_scales, ref.col_scales)):
        assert torch.equal(a, b)


def test_attention_from_fused_operands():
    """q, k before rotary embedding -> fused producer (tau folded, keys centered) -> forward and
    backward with softmax_scale = 1, against the oracle run on the producer oracle's tensors."""
    from paper_2609_37852_b200 import binding as Bd
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=4, heads_kv=2, seqlen=512)
    q, k, v, dO = workloads.make_inputs(w)
    cos, sin = P.rope_tables(w.seqlen, w.head_dim_qk)
    tc, ts = torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda()
    tau = np.float32(w.softmax_scale)
    qq, _ = Bd.attn_fp8_quantize_fused(q.cuda(), tc, ts, scale=float(tau))
    kq, kmean = Bd.attn_fp8_quantize_fused(k.cuda(), tc, ts, center=True)
    vq, dOq = Bd.attn_fp8_quantize(v.cuda()), Bd.attn_fp8_quantize(dO.cuda())
    params = Bd.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal, 1.0)
    o, lse, ws = Bd.attn_fp8_fwd(params, qq, kq, vq)
    delta, ws = Bd.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, workspace=ws)
    dq, dk, dv, rs, ra, ws = Bd.attn_fp8_bwd(params, qq, kq, vq, dOq, lse, delta, diagnostics=True, workspace=ws)
    Bd.attn_fp8_read_status(ws)
    qy, _ = P.fused_operand(to_np(q), cos, sin, scale=tau)
    ky, _ = P.fused_operand(to_np(k), cos, sin, center=True)
    vn, dOn = to_np(v), to_np(dO)
    O, LSE = A.emu_forward(qy, ky, vn, 1.0, w.causal)
    assert rel_fro(to_np(o), O) <= 2e-3 and rel_fro(to_np(lse), LSE) <= 2e-3
    D = A.emu_delta(qy, ky, vn, dOn, to_np(lse), 1.0, w.causal)
    assert rel_fro(to_np(delta), D) <= 1e-4
    dQ, dK, dV, _, _ = A.emu_backward(qy, ky, vn, dOn, to_np(lse), to_np(delta), 1.0, w.causal)
    assert rel_fro(to_np(dq), dQ) <= 5e-3 and rel_fro(to_np(dk), dK) <= 5e-3 and rel_fro(to_np(dv), dV) <= 5e-3
    r_pre = A.residual_ratio(to_np(rs), to_np(ra))[..., 64:]
    assert np.nanmedian(r_pre) <= 1e-5


def test_fused_producer_rejects_bad_arguments():
    from paper_2609_37852_b200 import binding
    x = torch.randn((1, 1, 128, 64)).cuda()
    with pytest.raises(binding.AttnFp8Error) as e:                    # centering needs a BF16 source
        binding.attn_fp8_quantize_fused(x, center=True)
    assert e.value.status == 2
    with pytest.raises(binding.AttnFp8Error) as e:
        binding.attn_fp8_quantize_fused(x.to(torch.bfloat16), scale=0.0)
    assert e.value.status == 1
