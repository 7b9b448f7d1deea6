"""Sequence shards: the rectangular causal problem a chunk of the queries runs against the keys it
can see (attn_params_t.seqlen_k / q_start), and the byte plumbing that assembles those keys from
per-chunk quantised shards.

One GPU stands in for the ranks: every chunk's problem is an independent set of launches, run one
after another.  What must hold:
  * quantising a chunk's tokens by themselves gives the bytes of the unsharded quantised tensor;
  * O, LSE, delta and dQ of a chunk are BIT-IDENTICAL to the same rows of the unsharded call;
  * the chunks' dK / dV contributions, summed in FP32, match the oracle's gradient of the
    unsharded problem within the gradient tolerance (each contribution is rounded to BF16 once).
"""
import numpy as np
import pytest
import torch

from oracle import attention as A
from paper_2609_37852_b200 import workloads
from tests.util import rel_fro, to_np, worst_row_error

pytestmark = pytest.mark.gpu


def _unsharded(B, params, prep, tensors):
    qq, kq, vq, dOq = (prep(x) for x in tensors)
    o, lse, ws = B.attn_fp8_fwd(params, qq, kq, vq)
    delta, ws = B.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, workspace=ws)
    dq, dk, dv, _, _, ws = B.attn_fp8_bwd(params, qq, kq, vq, dOq, lse, delta, workspace=ws)
    B.attn_fp8_read_status(ws)
    return dict(q=(qq, kq, vq, dOq), o=o, lse=lse, delta=delta, dq=dq, dk=dk, dv=dv)


@pytest.mark.parametrize("name,kw,n_chunks,bf16", [
    ("gqa4k", dict(batch=2, heads_q=4, heads_kv=2, seqlen=1024), 4, False),
    ("gqa8k_outlier", dict(heads_q=4, heads_kv=1, seqlen=768), 3, False),
    ("gqa8k_outlier", dict(heads_q=4, heads_kv=2, seqlen=768), 2, False),      # chunks of three tiles
    ("tiny", dict(seqlen=512, heads_q=2, heads_kv=1), 2, False),                # no mask: every chunk sees all keys
    ("mla8k", dict(heads_q=2, heads_kv=2, seqlen=512), 2, False),               # wide heads: dV / dK passes, dQ column tiles
    ("gqa8k_d256", dict(heads_q=2, heads_kv=1, seqlen=512), 4, False),
    ("gqa4k", dict(batch=1, heads_q=4, heads_kv=2, seqlen=768), 3, True),       # BF16 mode
])
def test_chunk_problems_reproduce_the_unsharded_rows(name, kw, n_chunks, bf16):
    from paper_2609_37852_b200 import binding as B
    from paper_2609_37852_b200 import sequence_parallel as SP
    w = workloads.WORKLOADS[name].scaled(**kw)
    tensors = [x.cuda() for x in workloads.make_inputs(w)]
    if bf16:
        tensors = [x.to(torch.bfloat16) for x in tensors]
    full = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                        w.softmax_scale, precision=B.ATTN_PREC_BF16 if bf16 else B.ATTN_PREC_MXFP8)
    prep = B.attn_fp8_prepare_bf16 if bf16 else B.attn_fp8_quantize
    ref = _unsharded(B, full, prep, tensors)
    L = w.seqlen // n_chunks
    cut = lambda x, c: x[:, :, c * L:(c + 1) * L].contiguous()
    # every chunk is quantised by its owner alone
    shards = [[prep(cut(x, c)) for x in tensors] for c in range(n_chunks)]
    if not bf16:
        for c in range(n_chunks):
            for t, whole in zip(shards[c], ref["q"]):
                want = SP.slice_chunk(whole, c, n_chunks)
                for f in ("row_codes", "row_scales", "col_codes", "col_scales"):
                    assert torch.equal(getattr(t, f).reshape(-1), getattr(want, f).reshape(-1)), (c, f)
    dk_sum = torch.zeros(ref["dk"].shape, dtype=torch.float32, device="cuda")
    dv_sum = torch.zeros(ref["dv"].shape, dtype=torch.float32, device="cuda")
    ws = None
    for c in range(n_chunks):
        p = SP.chunk_params(full, c, n_chunks)
        seen = c + 1 if w.causal else n_chunks
        if bf16:                                  # BF16 "quantised" tensors are the values and their transpose
            cat = lambda i: B.QTensor(shape=(w.batch, tensors[i].shape[1], seen * L, tensors[i].shape[3]),
                                      row_codes=torch.cat([shards[j][i].row_codes for j in range(seen)], dim=2).contiguous(),
                                      col_codes=torch.cat([shards[j][i].col_codes for j in range(seen)], dim=3).contiguous())
            kk, vv = cat(1), cat(2)
        else:
            kk = SP.concat_chunks([shards[j][1] for j in range(seen)])
            vv = SP.concat_chunks([shards[j][2] for j in range(seen)])
        qq, dOq = shards[c][0], shards[c][3]
        o, lse, ws = B.attn_fp8_fwd(p, qq, kk, vv, workspace=ws)
        delta, ws = B.attn_fp8_bwd_delta(p, qq, kk, vv, dOq, lse, workspace=ws)
        dq, dk, dv, _, _, ws = B.attn_fp8_bwd(p, qq, kk, vv, dOq, lse, delta, workspace=ws)
        B.attn_fp8_read_status(ws)
        assert dk.shape[2] == seen * L and dv.shape[2] == seen * L
        rows = slice(c * L, (c + 1) * L)
        assert torch.equal(o, ref["o"][:, :, rows]), f"chunk {c}: O"
        assert torch.equal(lse, ref["lse"][:, :, rows]), f"chunk {c}: LSE"
        assert torch.equal(delta, ref["delta"][:, :, rows]), f"chunk {c}: delta"
        assert torch.equal(dq, ref["dq"][:, :, rows]), f"chunk {c}: dQ"
        dk_sum[:, :, :seen * L] += dk.float()
        dv_sum[:, :, :seen * L] += dv.float()
    # the summed contributions against the unsharded kernel result and against the oracle
    assert rel_fro(to_np(dk_sum), to_np(ref["dk"])) <= 4e-3
    assert rel_fro(to_np(dv_sum), to_np(ref["dv"])) <= 4e-3
    qn, kn, vn, dOn = (to_np(x) for x in tensors)
    prec = "bf16" if bf16 else "mxfp8"
    _, dK, dV, _, _ = A.emu_backward(qn, kn, vn, dOn, to_np(ref["lse"]), to_np(ref["delta"]), w.softmax_scale, w.causal,
                                     prec=prec)
    for got, want, n_ in ((dk_sum, dK, "dk"), (dv_sum, dV, "dv")):
        assert rel_fro(to_np(got), want) <= 5e-3, n_
        assert worst_row_error(to_np(got), want) <= 5e-2, n_


def test_shard_parameters_are_validated():
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=2, heads_kv=1, seqlen=256)
    q, k, v, _ = (x.cuda() for x in workloads.make_inputs(w))
    qq, kq, vq = B.attn_fp8_quantize(q), B.attn_fp8_quantize(k), B.attn_fp8_quantize(v)
    base = dict(batch=1, seqlen=256, heads_q=2, heads_kv=1, head_dim_qk=128, head_dim_v=128, causal=True, softmax_scale=0.1)
    for bad, status in ((dict(seqlen_k=0, q_start=128), 1),          # q_start without seqlen_k
                        (dict(seqlen_k=512, q_start=128), 2),        # causal: seqlen_k != q_start + seqlen
                        (dict(seqlen_k=448, q_start=192), 2),        # not multiples of 128
                        (dict(seqlen_k=-128, q_start=0), 1)):
        with pytest.raises(B.AttnFp8Error) as e:
            B.attn_fp8_fwd(B.AttnParams(**base, **bad), qq, kq, vq)
        assert e.value.status == status, bad


def test_sharded_attention_on_a_one_rank_group():
    """The rank-level driver (quantise own chunks, exchange, per-chunk kernels, reduce key gradients)
    on a process group of one NCCL rank that owns both zig-zag chunks: the collectives run for real,
    and the results must be those of the unsharded call."""
    import torch.distributed as dist
    from paper_2609_37852_b200 import binding as B
    from paper_2609_37852_b200 import replicas
    from paper_2609_37852_b200 import sequence_parallel as SP
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=4, heads_kv=2, seqlen=1024)
    tensors = [x.cuda() for x in workloads.make_inputs(w)]
    full = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal, w.softmax_scale)
    ref = _unsharded(B, full, B.attn_fp8_quantize, tensors)
    started = not dist.is_initialized()
    if started:
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{replicas.free_port()}", rank=0, world_size=1)
    try:
        owners = SP.zigzag_chunks(1)                                   # [[0, 1]]
        L = w.seqlen // 2
        cut = lambda x: [x[:, :, c * L:(c + 1) * L].contiguous() for c in owners[0]]
        sa = SP.ShardedAttention(full, owners, rank=0)
        outs = sa.forward(cut(tensors[0]), cut(tensors[1]), cut(tensors[2]))
        grads = sa.backward(cut(tensors[3]))
        torch.cuda.synchronize()
    finally:
        if started:
            dist.destroy_process_group()
    n_el = w.batch * w.heads_kv * w.seqlen * w.head_dim_qk
    assert sa.fwd_exchange_bytes == 2 * n_el + 2 * n_el // 32 == sa.bwd_exchange_bytes
    for slot, c in enumerate(owners[0]):
        rows = slice(c * L, (c + 1) * L)
        o, lse = outs[slot]
        dq, dk, dv, delta = grads[slot]
        assert torch.equal(o, ref["o"][:, :, rows]) and torch.equal(lse, ref["lse"][:, :, rows])
        assert torch.equal(dq, ref["dq"][:, :, rows]) and torch.equal(delta, ref["delta"][:, :, rows])
        assert dk.dtype == torch.float32 and dk.shape == ref["dk"][:, :, rows].shape
        assert rel_fro(to_np(dk), to_np(ref["dk"][:, :, rows])) <= 4e-3
        assert rel_fro(to_np(dv), to_np(ref["dv"][:, :, rows])) <= 4e-3
