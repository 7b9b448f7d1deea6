"""Timing report over every workload and mode, in the paper's measurement protocol.

    python -m paper_2609_37852_b200.report [--workloads a,b,...] [--rounds 5] [--calls 20] [--out FILE]

For each workload (``workloads.WORKLOADS``) and each mode the library supports for it
(MXFP8 with the matched correction, MXFP8 with the stale correction, BF16 operands) the script
times the forward, the row correction and the gradient pass with CUDA events and prints one
markdown table row: milliseconds, TFLOP/s in the paper's FLOP convention, and the fraction of the
nominal dense tensor peak of the operand type.  Protocol (paper, Appendix "Attention Kernel
Throughput"): a few seconds of matmul warm-up, 5 warm-up calls, the median of 20 event timings
per round, 5 rounds interleaved over the modes, mean and standard error over the rounds.  The
operand preparation (quantiser, or the BF16 transposes) is timed separately and, as in the paper,
left out of the throughput columns.  Argument marshalling only: all work is done by the library.
"""
import argparse
import json
import math
import os
import statistics
import sys

import torch

from . import binding as B
from . import workloads

NOMINAL_TFLOPS = {"mxfp8": 4500.0, "bf16": 2250.0}


def measured_tflops():
    """Measured tensor peaks per operand type: the sustained BF16 GEMM figure of MEASURED_PEAKS.json at
    the repository root (an earlier measurement of the same pool where the file is absent), and twice
    that for FP8 (the nominal ratio)."""
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    bf16, source = 1400.0, "fallback"
    if os.path.exists(path):
        with open(path) as f:
            bf16, source = float(json.load(f)["bf16_tflops_sustained"]), "measured"
    return {"mxfp8": 2.0 * bf16, "bf16": bf16}, source


def _median_ms(fn, calls, stream):
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(calls)]
    for a, b in ev:
        a.record(stream)
        fn()
        b.record(stream)
    torch.cuda.synchronize()
    return statistics.median(a.elapsed_time(b) for a, b in ev)


class Case:
    """Device buffers and the three timed calls of one (workload, mode)."""

    def __init__(self, w, tensors, mode):
        self.w, self.mode = w, mode
        bf16 = mode == "bf16"
        self.prec = "bf16" if bf16 else "mxfp8"
        self.params = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                                   w.softmax_scale, precision=B.ATTN_PREC_BF16 if bf16 else B.ATTN_PREC_MXFP8,
                                   delta_mode=B.ATTN_DELTA_STALE if mode == "mxfp8-stale" else B.ATTN_DELTA_MATCHED)
        self.prepare = B.attn_fp8_prepare_bf16 if bf16 else B.attn_fp8_quantize
        self.src = tensors
        self.q, self.k, self.v, self.dO = (self.prepare(x) for x in tensors)
        self.dO_bf16 = tensors[3] if tensors[3].dtype == torch.bfloat16 else tensors[3].to(torch.bfloat16)
        self.o, self.lse, self.ws = B.attn_fp8_fwd(self.params, self.q, self.k, self.v)
        self.delta, _ = B.attn_fp8_bwd_delta(self.params, self.q, self.k, self.v, self.dO, self.lse,
                                             dO_bf16=self.dO_bf16, o_bf16=self.o, workspace=self.ws)
        self.dq, self.dk, self.dv, _, _, _ = B.attn_fp8_bwd(self.params, self.q, self.k, self.v, self.dO, self.lse,
                                                            self.delta, workspace=self.ws)
        B.attn_fp8_read_status(self.ws)

    def prep(self):
        if self.prec == "bf16":
            for x, t in zip(self.src, (self.q, self.k, self.v, self.dO)):
                self.prepare(x, out=t)
        else:                                            # the four operands in one quantiser launch
            B.attn_fp8_quantize_batch(self.src, outs=(self.q, self.k, self.v, self.dO), workspace=self.ws)

    def fwd(self):
        B.attn_fp8_fwd(self.params, self.q, self.k, self.v, o=self.o, lse=self.lse, workspace=self.ws)

    def corr(self):
        B.attn_fp8_bwd_delta(self.params, self.q, self.k, self.v, self.dO, self.lse, dO_bf16=self.dO_bf16,
                             o_bf16=self.o, delta=self.delta, workspace=self.ws)

    def grad(self):
        B.attn_fp8_bwd(self.params, self.q, self.k, self.v, self.dO, self.lse, self.delta, dq=self.dq, dk=self.dk,
                       dv=self.dv, workspace=self.ws)


def _modes_for(w):
    return ["mxfp8-matched", "mxfp8-stale", "bf16"]


def _mean_se(xs):
    m = statistics.mean(xs)
    se = statistics.stdev(xs) / math.sqrt(len(xs)) if len(xs) > 1 else 0.0
    return m, se


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workloads", default="tiny,gqa4k,gqa8k_outlier,mla8k,gqa8k_d256")
    ap.add_argument("--rounds", type=int, default=5)
    ap.add_argument("--calls", type=int, default=20)
    ap.add_argument("--warmup-seconds", type=float, default=3.0)
    ap.add_argument("--out", default=None)
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("the report needs a CUDA device: the attention path has no CPU fallback")
    dev = torch.device("cuda")
    stream = torch.cuda.current_stream()

    # matmul warm-up (clocks and power state)
    a = torch.randn((8192, 8192), device=dev, dtype=torch.bfloat16)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    while True:
        for _ in range(20):
            a @ a
        t1.record(); torch.cuda.synchronize()
        if t0.elapsed_time(t1) > args.warmup_seconds * 1e3:
            break
    del a

    measured, peak_source = measured_tflops()
    lines = [f"| workload | mode | prepare ms | fwd ms | correction ms | gradient ms | fwd TFLOP/s | bwd TFLOP/s | fwd+bwd TFLOP/s (+- SE) | with prepare | % of nominal peak | % of {peak_source} peak |",
             "|---|---|---|---|---|---|---|---|---|---|---|---|"]
    for name in args.workloads.split(","):
        w = workloads.WORKLOADS[name]
        tensors = [x.to(dev) for x in workloads.make_inputs(w)]
        cases = [Case(w, tensors, m) for m in _modes_for(w)]
        res = {c.mode: dict(prep=[], fwd=[], corr=[], grad=[]) for c in cases}
        for c in cases:
            for _ in range(5):
                c.prep(); c.fwd(); c.corr(); c.grad()
        torch.cuda.synchronize()
        for _ in range(args.rounds):                     # rounds interleaved over the modes
            for c in cases:
                for key, fn in (("prep", c.prep), ("fwd", c.fwd), ("corr", c.corr), ("grad", c.grad)):
                    res[c.mode][key].append(_median_ms(fn, args.calls, stream))
        for c in cases:
            B.attn_fp8_read_status(c.ws)
            r = res[c.mode]
            f_flops, b_flops = w.credited_flops()
            tot = [(f_flops + b_flops) / ((f + d + g) * 1e-3) / 1e12 for f, d, g in zip(r["fwd"], r["corr"], r["grad"])]
            m, se = _mean_se(tot)
            fwd_ms, corr_ms, grad_ms, prep_ms = (statistics.mean(r[k]) for k in ("fwd", "corr", "grad", "prep"))
            with_prep = (f_flops + b_flops) / ((fwd_ms + corr_ms + grad_ms + prep_ms) * 1e-3) / 1e12
            lines.append(f"| {name} (B={w.batch}, {w.heads_q}/{w.heads_kv} heads, N={w.seqlen}, d={w.head_dim_qk}/{w.head_dim_v}, "
                         f"{'causal' if w.causal else 'full'}) | {c.mode} | {prep_ms:.3f} | {fwd_ms:.3f} | {corr_ms:.3f} | {grad_ms:.3f} | "
                         f"{f_flops / (fwd_ms * 1e-3) / 1e12:.0f} | {b_flops / ((corr_ms + grad_ms) * 1e-3) / 1e12:.0f} | "
                         f"{m:.0f} +- {se:.1f} | {with_prep:.0f} | {100 * m / NOMINAL_TFLOPS[c.prec]:.1f} | "
                         f"{100 * m / measured[c.prec]:.1f} |")
        del cases, tensors
        torch.cuda.empty_cache()
    text = "\n".join(lines)
    print(text)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text + "\n")
    return 0


if __name__ == "__main__":
    sys.exit(main())
