"""The whole path under CUDA-graph capture.

Every entry point only enqueues work on the caller's stream (the one synchronising call is
attn_fp8_read_status), so a step -- batched quantiser, forward, row correction, gradient pass -- can be
captured once and replayed.  The test captures a step into a graph, replays it on two different
inputs written into the captured buffers and requires every output to be bit-identical to an
eager step on the same input.  The gradient pass launches its query-major kernel behind the
key-major one with programmatic stream serialisation: the capture covers that edge too.
"""
import pytest
import torch

from paper_2609_37852_b200 import workloads

pytestmark = pytest.mark.gpu


def _step(B, params, src, bufs):
    """One step into preallocated buffers (no allocation, no synchronisation)."""
    B.attn_fp8_quantize_batch(src, outs=bufs["operands"], workspace=bufs["ws"])
    qq, kq, vq, dOq = bufs["operands"]
    B.attn_fp8_fwd(params, qq, kq, vq, o=bufs["o"], lse=bufs["lse"], workspace=bufs["ws"])
    B.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, bufs["lse"], delta=bufs["delta"], workspace=bufs["ws"])
    B.attn_fp8_bwd(params, qq, kq, vq, dOq, bufs["lse"], bufs["delta"], dq=bufs["dq"], dk=bufs["dk"], dv=bufs["dv"],
                   workspace=bufs["ws"])


def _buffers(B, params, src):
    operands = [B.attn_fp8_quantize(x) for x in src]
    qq, kq, vq, dOq = operands
    o, lse, ws = B.attn_fp8_fwd(params, qq, kq, vq)
    ws = B.new_workspace(max(B.attn_fp8_workspace_bytes(params, i) for i in range(3)), "cuda")
    delta, _ = B.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, workspace=ws)
    dq, dk, dv, _, _, _ = B.attn_fp8_bwd(params, qq, kq, vq, dOq, lse, delta, workspace=ws)
    return dict(operands=operands, o=o, lse=lse, ws=ws, delta=delta, dq=dq, dk=dk, dv=dv)


@pytest.mark.parametrize("name,kw", [
    ("gqa8k_outlier", dict(heads_q=8, heads_kv=2, seqlen=1024)),
    ("mla8k", dict(heads_q=2, heads_kv=2, seqlen=512)),           # wide heads: two key-major passes ahead of the dQ kernel
])
def test_captured_step_replays_bit_identically(name, kw):
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS[name].scaled(**kw)
    params = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                          w.softmax_scale)
    inputs_a = [x.cuda() for x in workloads.make_inputs(w)]
    inputs_b = [x.cuda() for x in workloads.make_inputs(w.scaled(index=w.index + 40))]    # other seeds, same shape
    keys = ("o", "lse", "delta", "dq", "dk", "dv")

    eager = {}
    for tag, inp in (("a", inputs_a), ("b", inputs_b)):
        bufs = _buffers(B, params, inp)
        _step(B, params, inp, bufs)
        B.attn_fp8_read_status(bufs["ws"])
        eager[tag] = {k: bufs[k].clone() for k in keys}
    assert not torch.equal(eager["a"]["dq"], eager["b"]["dq"])

    static_in = [torch.empty_like(x) for x in inputs_a]
    bufs = _buffers(B, params, inputs_a)
    for k in keys:
        bufs[k].fill_(float("nan"))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        _step(B, params, inputs_a, bufs)                          # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        _step(B, params, static_in, bufs)
    for tag, inp in (("a", inputs_a), ("b", inputs_b), ("a", inputs_a)):
        for dst, x in zip(static_in, inp):
            dst.copy_(x)
        graph.replay()
        torch.cuda.synchronize()
        B.attn_fp8_read_status(bufs["ws"])
        for k in keys:
            assert torch.equal(bufs[k], eager[tag][k]), f"replay on input {tag}: {k} differs from the eager step"
