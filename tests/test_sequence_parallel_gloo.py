"""The exchange of the sequence-sharded path on CPU: two gloo ranks all-gather the bytes of their
quantised chunks and reduce the chunks' contributions to the key gradients.  No kernel runs here: the
tensors are random bytes / floats in the library's layouts, and what is checked is that every byte and
every partial sum ends up where the unsharded layout has it."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_37852_b200 import binding as B
from paper_2609_37852_b200 import sequence_parallel as SP


def _random_qtensor(Bn, H, N, d, seed):
    g = torch.Generator().manual_seed(seed)
    u8 = lambda n: torch.randint(0, 256, (n,), dtype=torch.uint8, generator=g)
    return B.QTensor(shape=(Bn, H, N, d),
                     row_codes=u8(Bn * H * N * d).view(Bn, H, N, d),
                     row_scales=u8(B.attn_fp8_scale_bytes(Bn, H, N, d)),
                     col_codes=u8(Bn * H * N * d).view(Bn, H, d, N),
                     col_scales=u8(B.attn_fp8_scale_bytes(Bn, H, d, N)))


def _same(a, b):
    return all(torch.equal(getattr(a, f).reshape(-1), getattr(b, f).reshape(-1))
               for f in ("row_codes", "row_scales", "col_codes", "col_scales"))


@pytest.mark.parametrize("d", [64, 128, 192, 256])
def test_slice_and_concat_are_inverse_and_follow_the_scale_layout(d):
    Bn, H, N, n_chunks = 2, 3, 1024, 4
    full = _random_qtensor(Bn, H, N, d, seed=d)
    parts = [SP.slice_chunk(full, c, n_chunks) for c in range(n_chunks)]
    assert _same(SP.concat_chunks(parts), full)
    # against the documented offset rule: the scale byte of (token, block) of chunk c is the scale byte
    # of (c * L + token, block) of the whole tensor, in both orientations
    L = N // n_chunks
    rs_full = B.unpack_scales(full.row_scales, Bn, H, N, d)              # [B, H, N, d/32]
    cs_full = B.unpack_scales(full.col_scales, Bn, H, d, N)              # [B, H, d, N/32]
    for c in (0, 2, 3):
        rs = B.unpack_scales(parts[c].row_scales, Bn, H, L, d)
        cs = B.unpack_scales(parts[c].col_scales, Bn, H, d, L)
        assert torch.equal(rs, rs_full[:, :, c * L:(c + 1) * L])
        assert torch.equal(cs, cs_full[:, :, :, c * L // 32:(c + 1) * L // 32])
        assert torch.equal(parts[c].row_codes, full.row_codes[:, :, c * L:(c + 1) * L])
        assert torch.equal(parts[c].col_codes, full.col_codes[:, :, :, c * L:(c + 1) * L])


def test_plans():
    assert SP.contiguous_chunks(3) == [[0], [1], [2]]
    assert SP.zigzag_chunks(2) == [[0, 3], [1, 2]]
    # zig-zag evens the causal work out; contiguous chunks do not
    t = 4
    zig = [SP.causal_tile_pairs(o, 8, t) for o in SP.zigzag_chunks(4)]
    con = [SP.causal_tile_pairs(o, 4, 2 * t) for o in SP.contiguous_chunks(4)]
    assert len(set(zig)) == 1 and sum(zig) == sum(con) == (8 * t) * (8 * t + 1) // 2
    assert con[-1] > 5 * con[0]
    full = B.AttnParams(1, 1024, 4, 2, 128, 128, True, 0.1)
    p = SP.chunk_params(full, 2, 4)
    assert (p.seqlen, p.seqlen_k, p.q_start) == (256, 768, 512)
    p = SP.chunk_params(B.AttnParams(1, 1024, 4, 2, 128, 128, False, 0.1), 2, 4)
    assert (p.seqlen, p.seqlen_k, p.q_start) == (256, 1024, 0)
    with pytest.raises(ValueError):
        SP.chunk_params(full, 0, 3)


def _worker(rank, world, port, zigzag, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    owners = SP.zigzag_chunks(world) if zigzag else SP.contiguous_chunks(world)
    n_chunks = sum(len(o) for o in owners)
    Bn, H, N, d = 1, 2, 128 * 2 * n_chunks, 128
    L = N // n_chunks
    full = _random_qtensor(Bn, H, N, d, seed=7)                       # every rank can rebuild the whole for the check
    mine = [SP.slice_chunk(full, c, n_chunks) for c in owners[rank]]
    # forward-style exchange: only the row copy travels; backward-style: only the col copy
    rows = SP.all_gather_chunks([SP.only(t, True, False) for t in mine], owners)
    cols = SP.all_gather_chunks([SP.only(t, False, True) for t in mine], owners)
    whole = SP.merged(SP.concat_chunks(rows), SP.concat_chunks(cols))
    ok_gather = _same(whole, full)
    sent = sum(SP.exchange_bytes(SP.only(t, True, False)) for t in mine)
    # key gradients: chunk c contributes to the keys of chunks 0..c (causal); owners get the sums
    g = torch.Generator().manual_seed(11)
    contrib = {c: torch.randn((Bn, H, (c + 1) * L, d), generator=g).to(torch.bfloat16) for c in range(n_chunks)}
    got = SP.reduce_scatter_key_grads([(c, contrib[c]) for c in owners[rank]], owners, rank, L)
    ok_sum = True
    for slot, c in enumerate(owners[rank]):
        want = sum(contrib[j].float()[:, :, c * L:(c + 1) * L] for j in range(c, n_chunks))
        ok_sum &= bool(torch.allclose(got[slot], want, rtol=0, atol=1e-5))
    out[rank] = (ok_gather, ok_sum, sent, len(mine) * Bn * H * L * d * (1 + 1 / 32))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("zigzag,port", [(False, 29651), (True, 29653)])
def test_two_ranks_exchange_fp8_chunks_and_reduce_key_gradients(zigzag, port):
    world = 2
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(world, port, zigzag, out), nprocs=world, join=True)
    for r in range(world):
        ok_gather, ok_sum, sent, expect = out[r]
        assert ok_gather and ok_sum, (r, ok_gather, ok_sum)
        assert sent == expect                                          # 1 + 1/32 bytes per element and orientation
