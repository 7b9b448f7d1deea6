"""Seeded synthetic attention inputs shaped like the paper's workloads.

The paper's kernel measurements use random-normal tensors (Appendix "Attention
Kernel Throughput") and its residual probe uses captured activations that are
not public; these generators stand in for both.  They hold none of the method's
arithmetic: they only draw Q, K, V, dO on the CPU from a seeded generator,
apply the input conditioning a workload names (QK RMS normalisation, rotary
embedding, outlier channels, heavy-tailed channel gains) and round to the
source dtype.  Both the CUDA tests and the CPU oracle tests consume them.
"""
from dataclasses import dataclass, replace
import math

import torch

SEED_BASE = 20260937852


@dataclass(frozen=True)
class Workload:
    name: str
    index: int            # position in the configuration list (seeds derive from it)
    batch: int
    heads_q: int
    heads_kv: int
    seqlen: int
    head_dim_qk: int
    head_dim_v: int
    causal: bool
    dtype: str            # "bf16" or "fp32": source dtype of Q, K, V, dO
    recipe: str           # "iid", "qknorm", "outlier_rope", "outlier_rope_aligned" (stress), "plain", "student_t"
    dO_std: float

    @property
    def softmax_scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim_qk)

    def credited_flops(self):
        """(forward, backward) FLOPs in the paper's convention: 2*B*Hq*N^2*d forward
        and 5*B*Hq*N^2*d backward for causal attention with one head dim; written
        per matmul so that unequal qk / v head dims are covered; doubled when not
        causal.  The row-correction pass earns no credit."""
        c = 1 if self.causal else 2
        base = c * self.batch * self.heads_q * self.seqlen * self.seqlen
        fwd = base * (self.head_dim_qk + self.head_dim_v)
        bwd = base * (3 * self.head_dim_qk + 2 * self.head_dim_v)
        return fwd, bwd

    def scaled(self, **kw):
        """Same recipe at another size (for parity tests the oracle can finish)."""
        return replace(self, **kw)


WORKLOADS = {
    w.name: w for w in [
        Workload("tiny", 1, 1, 1, 1, 256, 64, 64, False, "fp32", "iid", 1.0),
        Workload("gqa4k", 2, 2, 16, 4, 4096, 128, 128, True, "bf16", "qknorm", 1e-2),
        Workload("gqa8k_outlier", 3, 1, 32, 8, 8192, 128, 128, True, "bf16", "outlier_rope", 1e-2),
        Workload("mla8k", 4, 1, 16, 16, 8192, 192, 128, True, "bf16", "plain", 1e-2),
        Workload("gqa8k_d256", 6, 1, 8, 2, 8192, 256, 256, True, "bf16", "plain", 1e-2),
        Workload("long64k", 5, 1, 32, 8, 65536, 128, 128, True, "bf16", "student_t", 1e-3),
    ]
}


def _gen(w: Workload, tensor_index: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(SEED_BASE + 100 * w.index + tensor_index)
    return g


def _rope_half_split(x: torch.Tensor, base: float = 10000.0) -> torch.Tensor:
    """Rotary embedding over the whole head, channel c paired with c + d/2,
    positions 0..N-1, computed in FP32."""
    n, d = x.shape[-2], x.shape[-1]
    half = d // 2
    inv_freq = base ** (-torch.arange(half, dtype=torch.float32) / half)
    ang = torch.arange(n, dtype=torch.float32)[:, None] * inv_freq[None, :]
    cos, sin = ang.cos(), ang.sin()
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def _aligned_outlier_gain(w: Workload, heads: int, d: int) -> torch.Tensor:
    """Stress variant of the outlier recipe: a query head shares the four outlier channels of its
    KV head (scores then have a standard deviation of ~70 and rows are nearly one-hot)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(SEED_BASE + 100 * w.index + 50)
    per_kv = [torch.randperm(d, generator=g)[:4] for _ in range(w.heads_kv)]
    gain = torch.ones(heads, d)
    group = heads // w.heads_kv
    for h in range(heads):
        gain[h, per_kv[h // group]] = 20.0
    return gain


def _condition_qk(w: Workload, x: torch.Tensor, g: torch.Generator) -> torch.Tensor:
    if w.recipe == "qknorm":
        return x / torch.sqrt(x.pow(2).mean(dim=-1, keepdim=True) + 1e-6)
    if w.recipe == "outlier_rope":
        heads, d = x.shape[1], x.shape[-1]
        gain = torch.ones(heads, d)
        for h in range(heads):
            gain[h, torch.randperm(d, generator=g)[:4]] = 20.0
        return _rope_half_split(x * gain[None, :, None, :])
    if w.recipe == "outlier_rope_aligned":
        return _rope_half_split(x * _aligned_outlier_gain(w, x.shape[1], x.shape[-1])[None, :, None, :])
    if w.recipe == "student_t":
        heads, d = x.shape[1], x.shape[-1]
        z = torch.randn(heads, d, generator=g)
        chi2 = torch.randn(heads, d, 3, generator=g).pow(2).sum(-1)
        gain = (z / torch.sqrt(chi2 / 3.0)).abs()
        return x * gain[None, :, None, :]
    return x


def make_inputs(w: Workload):
    """Q [B,Hq,N,dqk], K [B,Hkv,N,dqk], V [B,Hkv,N,dv], dO [B,Hq,N,dv] on the CPU in
    the workload's source dtype (torch.bfloat16 or torch.float32)."""
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    out = []
    shapes = [
        (w.batch, w.heads_q, w.seqlen, w.head_dim_qk),
        (w.batch, w.heads_kv, w.seqlen, w.head_dim_qk),
        (w.batch, w.heads_kv, w.seqlen, w.head_dim_v),
        (w.batch, w.heads_q, w.seqlen, w.head_dim_v),
    ]
    for idx, shape in enumerate(shapes):
        g = _gen(w, idx)
        x = torch.randn(shape, generator=g, dtype=torch.float32)
        if idx < 2:
            x = _condition_qk(w, x, g)
        if idx == 3:
            x = x * w.dO_std
        out.append(x.to(dt).contiguous())
    return tuple(out)
