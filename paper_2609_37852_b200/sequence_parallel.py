"""Sequence-sharded (context-parallel) attention with an exchange of FP8 K / V.

The paper names the exchange of FP8 keys and values between sequence shards as the next engineering
step (Limitations); this module is that step for the kernels of this package.

Layout.  A sequence of N tokens is cut into chunks of L tokens (L a multiple of 128).  A rank owns one
or more chunks: its Q, K, V, dO rows for those tokens.  Every rank quantises its own tokens once (both
orientations; the 1x32 blocks never straddle a chunk because chunks are multiples of 128 tokens, so the
codes and scale bytes equal those of the unsharded tensor).  What crosses ranks is bytes:

  forward   all-gather of  K row codes + scales,  V col codes + scales            (1 + 1/32 B per element each)
  backward  all-gather of  V row codes + scales,  K col codes + scales            (the same again)
            reduce-scatter (sum) of the FP32 partial dK, dV of every chunk

against 2 B per element for BF16 K / V in each direction: half the bytes, and no rank re-quantises what
another rank owns.  Under the causal mask the chunk that starts at token s attends keys 0 .. s + L - 1;
the kernels take that rectangular problem directly (attn_params_t.seqlen_k / q_start), and its rows of
O, LSE, delta and dQ are bit-identical to the rows of the unsharded problem.  dK / dV of a chunk's
problem are that chunk's contribution to all keys it sees; the sum over chunks is the gradient.

Everything here is plumbing: tensor views, copies and torch.distributed collectives.  The functions
that only rearrange bytes work on CPU tensors too, which is how the exchange is tested without GPUs
(gloo, world size 2).  Balance: with one chunk per rank the last rank does (2R - 1) times the work of
the first; `zigzag_chunks` gives rank r the chunks r and 2R - 1 - r, which evens the causal work out.
"""
from dataclasses import replace
from typing import List, Optional, Sequence, Tuple

import torch

from . import binding as B


# --------------------------------------------------------------------------------------- planning

def contiguous_chunks(world: int) -> List[List[int]]:
    """One chunk per rank, in order: rank r owns chunk r of `world` chunks."""
    return [[r] for r in range(world)]


def zigzag_chunks(world: int) -> List[List[int]]:
    """Two chunks per rank out of 2 * world: rank r owns chunks r and 2 * world - 1 - r, so that every
    rank sees the same number of (query tile, key tile) pairs under the causal mask."""
    return [[r, 2 * world - 1 - r] for r in range(world)]


def chunk_params(full: B.AttnParams, chunk: int, n_chunks: int) -> B.AttnParams:
    """The problem chunk `chunk` of `n_chunks` runs: its own queries against the keys it can see."""
    if full.seqlen_k or full.q_start:
        raise ValueError("`full` must describe the unsharded problem")
    if full.seqlen % (128 * n_chunks):
        raise ValueError("seqlen must be a multiple of 128 * n_chunks")
    L = full.seqlen // n_chunks
    if full.causal:
        return replace(full, seqlen=L, seqlen_k=(chunk + 1) * L, q_start=chunk * L)
    return replace(full, seqlen=L, seqlen_k=full.seqlen, q_start=0)


def causal_tile_pairs(chunks: Sequence[int], n_chunks: int, tiles_per_chunk: int) -> int:
    """(query tile, key tile) pairs a rank that owns `chunks` executes under the causal mask."""
    t = tiles_per_chunk
    return sum(t * c * t + t * (t + 1) // 2 for c in chunks)


# ------------------------------------------------------------------------- byte layout of the shards

def _views(qt: B.QTensor):
    """The four byte tensors of a quantised [B, H, N, d] tensor, shaped so that the token dimension
    (in units of tokens or of 128-token tiles) is an explicit axis; entries are (tensor, token axis)."""
    Bn, H, N, d = qt.shape
    c = (d + 127) // 128
    out = {}
    if qt.row_codes is not None:
        out["row_codes"] = (qt.row_codes.view(Bn, H, N, d), 2)
    if qt.row_scales is not None:
        out["row_scales"] = (qt.row_scales.view(Bn, H, N // 128, c * 512), 2)
    if qt.col_codes is not None:
        out["col_codes"] = (qt.col_codes.view(Bn, H, d, N), 3)
    if qt.col_scales is not None:
        out["col_scales"] = (qt.col_scales.view(Bn, H, c, N // 128, 512), 3)
    return out


def concat_chunks(parts: Sequence[B.QTensor]) -> B.QTensor:
    """The quantised tensor of the concatenated tokens of `parts` (same batch, heads and head dim;
    the same orientations present in all).  A pure rearrangement of bytes."""
    Bn, H, _, d = parts[0].shape
    N = sum(p.shape[2] for p in parts)
    views = [_views(p) for p in parts]
    out = B.QTensor(shape=(Bn, H, N, d))
    for name in views[0]:
        axis = views[0][name][1]
        cat = torch.cat([v[name][0] for v in views], dim=axis).contiguous()
        setattr(out, name, cat if name.endswith("codes") else cat.reshape(-1))
    return out


def slice_chunk(qt: B.QTensor, chunk: int, n_chunks: int) -> B.QTensor:
    """The bytes of chunk `chunk` of a quantised tensor (the inverse of concat_chunks)."""
    Bn, H, N, d = qt.shape
    L = N // n_chunks
    out = B.QTensor(shape=(Bn, H, L, d))
    for name, (t, axis) in _views(qt).items():
        per = t.shape[axis] // n_chunks
        part = t.narrow(axis, chunk * per, per).contiguous()
        setattr(out, name, part if name.endswith("codes") else part.reshape(-1))
    return out


def only(qt: B.QTensor, row: bool, col: bool) -> B.QTensor:
    """`qt` restricted to the orientations asked for (what one exchange sends)."""
    return B.QTensor(shape=qt.shape, row_codes=qt.row_codes if row else None, row_scales=qt.row_scales if row else None,
                     col_codes=qt.col_codes if col else None, col_scales=qt.col_scales if col else None)


def merged(a: B.QTensor, b: B.QTensor) -> B.QTensor:
    """One tensor's orientations collected from two exchanges (row copy from one, col copy from the other)."""
    pick = lambda x, y: x if x is not None else y
    return B.QTensor(shape=a.shape, row_codes=pick(a.row_codes, b.row_codes), row_scales=pick(a.row_scales, b.row_scales),
                     col_codes=pick(a.col_codes, b.col_codes), col_scales=pick(a.col_scales, b.col_scales))


def exchange_bytes(qt: B.QTensor) -> int:
    """Bytes one rank contributes when `qt` is all-gathered."""
    return sum(t.numel() for t, _ in _views(qt).values())


# ------------------------------------------------------------------------------------- collectives

def all_gather_chunks(local: Sequence[B.QTensor], owners: Sequence[Sequence[int]], group=None) -> List[B.QTensor]:
    """All-gathers the quantised chunks every rank owns.  `local` are this rank's chunks in the order of
    owners[rank]; the result lists all chunks in token order.  One all_gather per byte tensor and local
    chunk (uint8: any backend)."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    n_chunks = sum(len(o) for o in owners)
    got: List[Optional[B.QTensor]] = [None] * n_chunks
    for slot, mine in enumerate(local):
        parts = [B.QTensor(shape=mine.shape) for _ in range(world)]
        for name, (t, _) in _views(mine).items():
            flat = t.contiguous().reshape(-1)
            outs = [torch.empty_like(flat) for _ in range(world)]
            dist.all_gather(outs, flat, group=group)
            for r in range(world):
                setattr(parts[r], name, outs[r].view(t.shape) if name.endswith("codes") else outs[r])
        for r in range(world):
            got[owners[r][slot]] = parts[r]
    return got  # type: ignore[return-value]


def reduce_scatter_key_grads(partials: Sequence[Tuple[int, torch.Tensor]], owners: Sequence[Sequence[int]], rank: int,
                             chunk_len: int, group=None) -> List[torch.Tensor]:
    """Sums the chunks' contributions to dK (or dV) and leaves every rank with the gradient of the
    chunks it owns.  `partials`: (chunk, tensor [B, Hkv, keys seen by that chunk, d]) for each of this
    rank's chunks.  The sum is formed in FP32 (the kernels round each contribution to BF16 once; the
    sum over chunks is rounded once more at the end by the caller if it wants BF16)."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    n_chunks = sum(len(o) for o in owners)
    ref = partials[0][1]
    Bn, H, _, d = ref.shape
    acc = torch.zeros((n_chunks, Bn, H, chunk_len, d), dtype=torch.float32, device=ref.device)
    for _, t in partials:
        seen = t.shape[2] // chunk_len
        acc[:seen] += t.float().view(Bn, H, seen, chunk_len, d).permute(2, 0, 1, 3, 4)
    out = []
    for slot in range(len(owners[rank])):
        # rank r receives the sum of everyone's contribution to its slot-th chunk
        send = [acc[owners[r][slot]].contiguous() for r in range(world)]
        recv = torch.empty_like(send[0])
        if dist.get_backend(group) == "gloo":                 # gloo has no reduce_scatter: reduce to each owner
            for r in range(world):
                buf = send[r].clone()
                dist.reduce(buf, dst=dist.get_global_rank(group, r) if group is not None else r, op=dist.ReduceOp.SUM,
                            group=group)
                if r == rank:
                    recv = buf
        else:
            dist.reduce_scatter(recv, send, op=dist.ReduceOp.SUM, group=group)
        out.append(recv)
    return out


# --------------------------------------------------------------------------- one rank's forward / backward

class ShardedAttention:
    """Forward and backward of one rank.  `full` describes the unsharded problem; `owners[r]` lists
    the chunks rank r owns (contiguous_chunks / zigzag_chunks).  Inputs are the rank's own tokens,
    one tensor per owned chunk, [B, H, L, d] BF16 or FP32 on the GPU."""

    def __init__(self, full: B.AttnParams, owners: Sequence[Sequence[int]], rank: int, group=None):
        self.full, self.owners, self.rank, self.group = full, [list(o) for o in owners], rank, group
        self.n_chunks = sum(len(o) for o in owners)
        self.L = full.seqlen // self.n_chunks
        self.mine = self.owners[rank]
        self.ws = None

    def _gather(self, local: Sequence[B.QTensor]) -> List[B.QTensor]:
        return all_gather_chunks(local, self.owners, self.group)

    def _keys_for(self, chunks_all: Sequence[B.QTensor], chunk: int) -> B.QTensor:
        seen = chunk + 1 if self.full.causal else self.n_chunks
        return concat_chunks(chunks_all[:seen])

    def forward(self, q: Sequence[torch.Tensor], k: Sequence[torch.Tensor], v: Sequence[torch.Tensor]):
        """Returns per owned chunk (O, LSE).  Keeps what the backward needs."""
        self.qq = [B.attn_fp8_quantize(x) for x in q]
        self.kq = [B.attn_fp8_quantize(x) for x in k]
        self.vq = [B.attn_fp8_quantize(x) for x in v]
        k_rows = self._gather([only(t, True, False) for t in self.kq])          # FP8 exchange of the forward
        v_cols = self._gather([only(t, False, True) for t in self.vq])
        self.fwd_exchange_bytes = sum(exchange_bytes(only(t, True, False)) for t in self.kq) + \
            sum(exchange_bytes(only(t, False, True)) for t in self.vq)
        self._k_rows, self._v_cols = k_rows, v_cols
        out = []
        self.lse = []
        for slot, chunk in enumerate(self.mine):
            p = chunk_params(self.full, chunk, self.n_chunks)
            o, lse, self.ws = B.attn_fp8_fwd(p, self.qq[slot], self._keys_for(k_rows, chunk), self._keys_for(v_cols, chunk),
                                             workspace=self.ws)
            self.lse.append(lse)
            out.append((o, lse))
        return out

    def backward(self, dO: Sequence[torch.Tensor]):
        """Returns per owned chunk (dQ, dK, dV, D); dK and dV are the FP32 sums over all chunks'
        contributions for the keys this rank owns."""
        dOq = [B.attn_fp8_quantize(x) for x in dO]
        v_rows = self._gather([only(t, True, False) for t in self.vq])          # FP8 exchange of the backward
        k_cols = self._gather([only(t, False, True) for t in self.kq])
        self.bwd_exchange_bytes = sum(exchange_bytes(only(t, True, False)) for t in self.vq) + \
            sum(exchange_bytes(only(t, False, True)) for t in self.kq)
        dqs, deltas, dk_parts, dv_parts = [], [], [], []
        for slot, chunk in enumerate(self.mine):
            p = chunk_params(self.full, chunk, self.n_chunks)
            kk = merged(self._keys_for(self._k_rows, chunk), self._keys_for(k_cols, chunk))
            vv = merged(self._keys_for(v_rows, chunk), self._keys_for(self._v_cols, chunk))
            delta, self.ws = B.attn_fp8_bwd_delta(p, self.qq[slot], kk, vv, dOq[slot], self.lse[slot], workspace=self.ws)
            dq, dk, dv, _, _, self.ws = B.attn_fp8_bwd(p, self.qq[slot], kk, vv, dOq[slot], self.lse[slot], delta,
                                                       workspace=self.ws)
            dqs.append(dq); deltas.append(delta)
            dk_parts.append((chunk, dk)); dv_parts.append((chunk, dv))
        B.attn_fp8_read_status(self.ws)
        dk_own = reduce_scatter_key_grads(dk_parts, self.owners, self.rank, self.L, self.group)
        dv_own = reduce_scatter_key_grads(dv_parts, self.owners, self.rank, self.L, self.group)
        return [(dqs[i], dk_own[i], dv_own[i], deltas[i]) for i in range(len(self.mine))]


# ------------------------------------------------------------------------------------------ timing

def _time_chunk_problems(seqlen: int, ranks: int, heads_q: int, heads_kv: int, steps: int = 5):
    """Per-rank time of one forward + correction + gradient pass over the rank's chunk problems, each
    rank's work run alone on the current GPU (no exchange: the collectives are not timed here)."""
    from . import workloads
    w = workloads.WORKLOADS["gqa8k_outlier"].scaled(seqlen=seqlen, heads_q=heads_q, heads_kv=heads_kv)
    tensors = [x.cuda() for x in workloads.make_inputs(w)]
    full = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, True, w.softmax_scale)

    def timed(step):
        for _ in range(3):
            step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    def one_pass(p, qq, kk, vv, dOq, state):
        o, lse, state["ws"] = B.attn_fp8_fwd(p, qq, kk, vv, workspace=state["ws"])
        delta, state["ws"] = B.attn_fp8_bwd_delta(p, qq, kk, vv, dOq, lse, workspace=state["ws"])
        B.attn_fp8_bwd(p, qq, kk, vv, dOq, lse, delta, workspace=state["ws"])

    def rank_ms(n_chunks, chunks):
        L = seqlen // n_chunks
        cut = lambda x, c: x[:, :, c * L:(c + 1) * L].contiguous()
        shards = {c: [B.attn_fp8_quantize(cut(x, c)) for x in tensors] for c in range(max(chunks) + 1)}
        total = 0.0
        for c in chunks:
            p = chunk_params(full, c, n_chunks)
            kk = concat_chunks([shards[j][1] for j in range(c + 1)])
            vv = concat_chunks([shards[j][2] for j in range(c + 1)])
            state = {"ws": None}
            total += timed(lambda: one_pass(p, shards[c][0], kk, vv, shards[c][3], state))
        return total

    con = [rank_ms(ranks, o) for o in contiguous_chunks(ranks)]
    zig = [rank_ms(2 * ranks, o) for o in zigzag_chunks(ranks)]
    q4 = [B.attn_fp8_quantize(x) for x in tensors]
    state = {"ws": None}
    whole = timed(lambda: one_pass(full, q4[0], q4[1], q4[2], q4[3], state))
    n_kv = w.batch * heads_kv * (seqlen // ranks) * w.head_dim_qk
    return dict(seqlen=seqlen, ranks=ranks, heads=(heads_q, heads_kv), contiguous_ms=con, zigzag_ms=zig, unsharded_ms=whole,
                exchange_bytes_per_rank_and_pass={"fp8": 2 * n_kv + 2 * n_kv // 32, "bf16": 4 * n_kv})


if __name__ == "__main__":
    import argparse
    import json
    ap = argparse.ArgumentParser(description="time the chunk problems of a sequence-sharded causal layer on one GPU")
    ap.add_argument("--seqlen", type=int, default=32768)
    ap.add_argument("--ranks", type=int, default=4)
    ap.add_argument("--heads-q", type=int, default=8)
    ap.add_argument("--heads-kv", type=int, default=2)
    a = ap.parse_args()
    print(json.dumps(_time_chunk_problems(a.seqlen, a.ranks, a.heads_q, a.heads_kv)))
