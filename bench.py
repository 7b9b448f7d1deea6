#!/usr/bin/env python
"""Benchmark of the FP8 Delta-Matching attention path on B200.

A step is one pass of the whole hot path over one batch of synthetic input:
quantise Q, K, V, dO (both block orientations), forward, matched row
correction, gradient pass (dQ, then dK/dV).  The metric is causal-adjusted
TFLOP/s of forward + backward in the paper's FLOP convention (the correction
pass and the quantiser earn no credit).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  With N > 1 every rank runs an independent replica
of the workload on its own GPU -- the path has no exchange step -- and the value
is the aggregate over ranks.  ``--gpus N`` without a launcher around it (no
WORLD_SIZE in the environment) starts the N ranks itself.
``--impl reference`` times the CPU oracle on a bounded causal prefix of the
same workload instead (host cores; rank 0 only).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOAD = "gqa8k_outlier"          # B=1, Hq=32, Hkv=8, N=8192, d=128, causal: the configuration the metric is quoted on
METRIC = "fp8_attn_fwd_bwd_causal_tflops"
UNIT = "TFLOP/s"
NOMINAL_FP8_TFLOPS = 4500.0
FP8_OVER_BF16 = 2.0                 # nominal dense FP8 : BF16 tensor ratio on B200

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of each kernel on WORKLOAD, from
# the ncu captures summarised under profiles/; None where no capture has been taken.
NCU_TRAFFIC_BYTES = {"quantize": 288.9e6, "fwd": 73.5e6, "bwd_delta": 90.5e6, "bwd_dq": 126.2e6, "bwd_dkdv": 317.9e6}
MACS_PER_CLK_PER_SM_FP8 = 8192      # dense FP8 tensor rate of one SM (the nominal 4.5 PFLOP/s is this at ~1.86 GHz on 148 SMs)

# executed matmul products per kernel as (contractions or outputs of width dqk, of width dv): each is
# 2*width FLOPs per unmasked (i, j) pair and query head
PRODUCTS = {"fwd": (1, 1), "bwd_delta": (1, 1), "bwd_dq": (2, 1), "bwd_dkdv": (2, 2)}


def _measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"], hbm=p["hbm_gbs"],
                    source="measured")
    return dict(bf16_burst=1590.0, bf16_sustained=1400.0, hbm=6650.0, source="fallback")


class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons while the timed region runs: NVML
    read-only queries from a thread every few milliseconds; nvidia-smi in a loop where NVML cannot be
    loaded.  Nothing is set or reset."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    # NVML clock-event reason bits
    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None
        self.thread = None
        self.samples = []          # (sm MHz, reasons bit mask)
        self.max_mhz = None
        self._stop = False

    def _nvml_handle(self):
        import pynvml
        pynvml.nvmlInit()
        try:
            import torch
            uuid = str(torch.cuda.get_device_properties(self.gpu_index).uuid)
            return pynvml, pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
        except Exception:
            return pynvml, pynvml.nvmlDeviceGetHandleByIndex(self.gpu_index)

    def start(self):
        try:
            nv, h = self._nvml_handle()
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
            reasons_fn = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons

            def loop():
                import time
                while not self._stop:
                    try:
                        self.samples.append((float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)), int(reasons_fn(h))))
                    except Exception:
                        pass
                    time.sleep(0.004)
            import threading
            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.thread is not None:
            self._stop = True
            self.thread.join(timeout=2)
            if self.samples:
                mask = 0
                for _, m in self.samples:
                    mask |= m
                out.update(sm_mhz=statistics.median(x for x, _ in self.samples), sm_max_mhz=self.max_mhz,
                           samples=len(self.samples), source="nvml",
                           reasons=sorted(n for n, bit in self.REASONS.items() if mask & bit))
            return out
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm), source="nvidia-smi")
        out["reasons"] = sorted(reasons)
        return out


def oracle_step(w, sample_tokens, q, k, v, dO, prec="mxfp8"):
    """One pass of the oracle (forward, matched correction, gradient pass) on the causal prefix of
    ``sample_tokens`` tokens of one KV group.  Returns credited FLOPs."""
    import numpy as np
    from oracle import attention as A
    G = w.heads_q // w.heads_kv
    qs, ks, vs, dOs = (x[:1, :hh, :sample_tokens].float().numpy().astype(np.float64)
                       for x, hh in ((q, G), (k, 1), (v, 1), (dO, G)))
    O, LSE = A.emu_forward(qs, ks, vs, w.softmax_scale, w.causal, prec=prec)
    D = A.emu_delta(qs, ks, vs, dOs, LSE, w.softmax_scale, w.causal, prec=prec)
    A.emu_backward(qs, ks, vs, dOs, LSE, D, w.softmax_scale, w.causal, prec=prec)
    sub = w.scaled(batch=1, heads_q=G, heads_kv=1, seqlen=sample_tokens)
    return sum(sub.credited_flops())


def residual_statistics(rs, ra, ps, dk, lse=None, dust=None):
    """Row-sum residual statistics of the paper's Appendix "Row-Sum Residuals" / "dS Quantization
    Residuals" from the outputs of the instrumented dQ pass (rs = sum_j dS, ra = sum_j |dS| before the
    cast, ps = sum_j dS' after it; [B, Hq, N]) and the key gradient dk [B, Hkv, N, d]: rows i >= 64 with
    a non-zero denominator, as in the paper."""
    import torch
    extra = {}
    if lse is not None and dust is not None:
        # the per-row acceptance on EVERY row: 1e-5 of sum |dS| plus the dust the FP32 storage of LSE leaves of
        # delta_i (1 - sum_j P_ij), (ulp(LSE_i) + 2^-20) * sum_j P_ij |dP^_ij|
        a = lse.abs()
        ulp = (torch.nextafter(a, torch.full_like(a, float("inf"))) - a).double()
        keys = torch.arange(1, rs.shape[-1] + 1, device=rs.device, dtype=torch.float64)      # keys a causal row sees
        c = 2.0 ** -20 * torch.clamp(keys / 8192.0, min=1.0)                                 # FP32 summation over the row
        ok = rs.double().abs() <= 1e-5 * ra.double() + (ulp + c) * dust.double()
        extra = {"bound_with_lse_dust_ok_frac_all_rows": float(ok.double().mean()),
                 "bound_with_lse_dust_ok_frac_rows_ge_64": float(ok[..., 64:].double().mean()),
                 "bound_with_lse_dust": "|sum_j dS| <= 1e-5 sum_j |dS| + (ulp(LSE_i) + 2^-20 max(1, keys / 8192)) "
                                        "sum_j P |dP^|, every row"}
    rs, ra, ps = (t[..., 64:].double().flatten() for t in (rs, ra, ps))
    live = ra > 0
    r_pre = rs[live].abs() / ra[live]
    r_post = ps[live].abs() / ra[live]
    kappa = (ps[live] - rs[live]) / ra[live]
    dkf = dk.double()
    c_k = (dkf.sum(dim=2).norm(dim=-1) / dkf.pow(2).sum(dim=(2, 3)).sqrt()).flatten()
    def median(t):                                   # the mean of the two middle values when the count is even
        srt = t.sort().values
        n = srt.numel()
        return float(srt[(n - 1) // 2] + srt[n // 2]) / 2.0

    return {
        "rows": "query rows i >= 64 with a non-zero sum_j |dS_ij|",
        "r_pre_median": median(r_pre),
        "r_pre_p99": float(r_pre.sort().values[min(r_pre.numel() - 1, int(0.99 * r_pre.numel()))]),
        "strict_ok_frac": float((r_pre <= 1e-5).double().mean()),
        "strict_ok": "share of those rows with |sum_j dS| <= 1e-5 sum_j |dS|",
        "r_post_median": median(r_post),
        "kappa_mean": float(kappa.mean()),
        "key_common_mode_median": median(c_k),
        **extra,
    }


def roofline_peaks(stage_clocks, peaks, bf16_mode, sms):
    """Denominators of the tensor rooflines.  The kernels' durations come from the per-stage loop, so the
    measured cuBLAS BF16 figure that applies is the one that goes with the clock that loop ran at: the burst
    figure when the sampled SM clock stayed within 5 % of the maximum, the sustained one (taken under the
    power cap) otherwise; doubled for FP8 (nominal ratio).  Returns (peak TFLOP/s, "burst" | "sustained",
    clock-normalised peak or None, divisor that turns FP8 figures into those of the mode's dtype)."""
    sc = stage_clocks
    at_boost = bool(sc.get("sm_mhz") and sc.get("sm_max_mhz") and sc["sm_mhz"] >= 0.95 * sc["sm_max_mhz"])
    which = "burst" if at_boost else "sustained"
    ratio = 1.0 if bf16_mode else FP8_OVER_BF16
    peak = peaks["bf16_" + which] * ratio
    dtype_div = FP8_OVER_BF16 if bf16_mode else 1.0           # BF16 mode: half the FP8 rate
    clock_peak = (2.0 * MACS_PER_CLK_PER_SM_FP8 / dtype_div * sms * sc["sm_mhz"] * 1e6 / 1e12) if sc.get("sm_mhz") else None
    return peak, which, clock_peak, dtype_div


def _cores_used():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def run_reference(args, w):
    """--impl reference: the oracle, as it stands, on the host cores."""
    from paper_2609_37852_b200 import workloads
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample_tokens = 512
    small = w.scaled(heads_q=w.heads_q // w.heads_kv, heads_kv=1, seqlen=sample_tokens)
    q, k, v, dO = workloads.make_inputs(small)
    for _ in range(args.warmup):
        oracle_step(w, sample_tokens, q, k, v, dO, args.precision)
    t0 = time.perf_counter()
    flops = 0
    for _ in range(args.steps):
        flops += oracle_step(w, sample_tokens, q, k, v, dO, args.precision)
    dt = time.perf_counter() - t0
    value = flops / dt / 1e12
    sample = (f"causal prefix of {sample_tokens} tokens of one KV group ({small.heads_q} query heads) of {w.name}, "
              f"fwd + matched correction + gradient pass per step")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": _cores_used(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=WORKLOAD)
    ap.add_argument("--precision", default="mxfp8", choices=["mxfp8", "bf16"],
                    help="bf16: the same kernels with BF16 operands and no block scales (reference point)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="length of the extra back-to-back loop that shows the settled (power-capped) rate; 0 skips it")
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher around this process: start the N ranks (one per GPU) and let rank 0 print the line
        from paper_2609_37852_b200 import replicas
        raise SystemExit(replicas.launch_local(args.gpus, os.path.abspath(__file__), sys.argv[1:]))

    from paper_2609_37852_b200 import workloads
    w = workloads.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    from paper_2609_37852_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    bf16_mode = args.precision == "bf16"
    params = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                          w.softmax_scale, precision=B.ATTN_PREC_BF16 if bf16_mode else B.ATTN_PREC_MXFP8)
    # operand preparation: block-scaling quantiser, or (BF16 mode) the transposed BF16 copies
    prepare = B.attn_fp8_prepare_bf16 if bf16_mode else B.attn_fp8_quantize
    host = [x.pin_memory() for x in workloads.make_inputs(w)]
    q, k, v, dO = (x.to(dev, non_blocking=True) for x in host)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()

    # pre-allocated operands, outputs and workspaces (device memory is PyTorch's job; the path is the library's)
    qq, kq, vq, dOq = (prepare(x) for x in (q, k, v, dO))
    bf = dict(dtype=torch.bfloat16, device=dev)
    o = torch.empty((w.batch, w.heads_q, w.seqlen, w.head_dim_v), **bf)
    lse = torch.empty((w.batch, w.heads_q, w.seqlen), dtype=torch.float32, device=dev)
    delta = torch.empty_like(lse)
    dq = torch.empty((w.batch, w.heads_q, w.seqlen, w.head_dim_qk), **bf)
    dk = torch.empty((w.batch, w.heads_kv, w.seqlen, w.head_dim_qk), **bf)
    dv = torch.empty((w.batch, w.heads_kv, w.seqlen, w.head_dim_v), **bf)
    ws = B.new_workspace(max(B.attn_fp8_workspace_bytes(params, i) for i in range(3)), dev)

    def prepare_all(srcs):
        """Q, K, V, dO -> the operand buffers: one batched quantiser launch, or the four BF16 copies."""
        if bf16_mode:
            for x, t in zip(srcs, (qq, kq, vq, dOq)):
                prepare(x, out=t)
        else:
            B.attn_fp8_quantize_batch(srcs, outs=(qq, kq, vq, dOq), workspace=ws)


    def step(events=None, split=False):
        """One pass of the path.  ``events``: recorded at the stage boundaries.  ``split``: the two
        kernels of the gradient pass run once more as separate calls, for their own durations."""
        def mark(i):
            if events is not None:
                events[i].record(stream)
        mark(0)
        prepare_all((q, k, v, dO))
        mark(1)
        B.attn_fp8_fwd(params, qq, kq, vq, o=o, lse=lse, workspace=ws)
        mark(2)
        B.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, delta=delta, workspace=ws)
        mark(3)
        # the gradient pass as a user calls it: one call, the dQ kernel launched behind the dK/dV kernel
        # so that it fills that kernel's last wave
        B.attn_fp8_bwd(params, qq, kq, vq, dOq, lse, delta, dq=dq, dk=dk, dv=dv, workspace=ws)
        mark(4)
        if split:                                   # once more as two serialised calls, an event around each
            B.attn_fp8_bwd_dq(params, qq, kq, vq, dOq, lse, delta, dq=dq, workspace=ws)
            mark(5)
            B.attn_fp8_bwd_dkdv(params, qq, kq, vq, dOq, lse, delta, dk=dk, dv=dv, workspace=ws)
            mark(6)

    # one batched quantiser launch (BF16 mode: four operand-preparation launches) + fwd + delta + dQ + dK/dV
    # (two key-major passes when the qk head dim exceeds 128)
    kernels_per_step = (8 if bf16_mode else 5) + (1 if (not bf16_mode and w.head_dim_qk > 128) else 0)

    # ---- device-resident timing -------------------------------------------------------------
    for _ in range(warmup):
        step()
    B.attn_fp8_read_status(ws)
    sampler = ClockSampler(local_rank)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(7)] for _ in range(args.steps)]
    barrier()
    sampler.start()
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for i in range(args.steps):
        step()                                      # no event inside a step: each one costs a few microseconds
    t_end.record(stream)
    barrier()
    clocks = sampler.stop()
    B.attn_fp8_read_status(ws)
    total_ms = t_start.elapsed_time(t_end)
    # per-stage breakdown: the same steps once more with an event at every stage boundary, followed by
    # the two kernels of the gradient pass as separate (serialised) calls
    stage_sampler = ClockSampler(local_rank)
    stage_sampler.start()
    for i in range(args.steps):
        step(events[i], split=True)
    torch.cuda.synchronize()
    stage_clocks = stage_sampler.stop()
    B.attn_fp8_read_status(ws)
    stage_ms = {n: statistics.mean(ev[j].elapsed_time(ev[j + 1]) for ev in events)
                for j, n in enumerate(("quantize", "fwd", "bwd_delta", "bwd", "bwd_dq", "bwd_dkdv"))}

    # ---- the same step back to back for a couple of seconds: the rate the part settles to ------------
    sustained = None
    if args.sustained_seconds > 0:
        n_sus = max(args.steps, int(args.sustained_seconds * 1e3 / (total_ms / args.steps)))
        sus_sampler = ClockSampler(local_rank)
        barrier()
        sus_sampler.start()
        s0 = torch.cuda.Event(enable_timing=True); s1 = torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        for i in range(n_sus):
            step()
        s1.record(stream)
        barrier()
        sus_clocks = sus_sampler.stop()
        B.attn_fp8_read_status(ws)
        sustained = {"steps": n_sus, "ms_per_step": s0.elapsed_time(s1) / n_sus, "clocks": sus_clocks}

    # ---- the bare block-scaled FP8 MMA rate of this device (a few ms; see attn_fp8_measure_mma_peak) ----
    measured_fp8 = None if bf16_mode else B.attn_fp8_measure_mma_peak(ws)

    # ---- what the FP32 reduction of dQ alone would cost in a merged key-major gradient pass (see
    #      attn_fp8_measure_dq_reduction): a design question kept measurable, outside every timed region
    dq_reduction = None
    if not bf16_mode and rank == 0 and w.head_dim_qk <= 128:
        scratch = torch.empty((w.batch, w.heads_q, w.seqlen, w.head_dim_qk), dtype=torch.float32, device=dev)
        red_ms, red_bytes = B.attn_fp8_measure_dq_reduction(params, scratch)
        del scratch
        dq_reduction = {"ms": red_ms, "GB": red_bytes / 1e9, "TB_per_s": red_bytes / (red_ms * 1e-3) / 1e12,
                        "note": "FP32 adds a merged dQ/dK/dV pass would send to L2; compare stage_ms.bwd_dq"}

    # ---- end to end through the library with host buffers --------------------------------------
    # Host buffers in, host buffers out, every step: copies run on their own streams and overlap the
    # kernels of the neighbouring steps (three slots of device inputs / outputs), as a user pipeline would.
    # The first upload and the last download are inside the timed region and overlap nothing.
    n_slots = 3
    in_dev = [[torch.empty_like(x) for x in (q, k, v, dO)] for _ in range(n_slots)]
    out_dev = [[torch.empty_like(x) for x in (o, lse, dq, dk, dv)] for _ in range(n_slots)]
    outs_host = [[torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in (o, lse, dq, dk, dv)] for _ in range(n_slots)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_run(n):
        in_ready = [None] * n
        comp_done = [None] * n
        out_done = [None] * n
        first = torch.cuda.Event(enable_timing=True)
        last = torch.cuda.Event(enable_timing=True)
        first.record(s_in)
        for i in range(n):
            slot = i % n_slots
            with torch.cuda.stream(s_in):
                if i >= n_slots:
                    s_in.wait_event(comp_done[i - n_slots])          # inputs of that step fully consumed
                for src, dst in zip(host, in_dev[slot]):
                    dst.copy_(src, non_blocking=True)
                in_ready[i] = torch.cuda.Event(); in_ready[i].record(s_in)
            stream.wait_event(in_ready[i])
            if i >= n_slots:
                stream.wait_event(out_done[i - n_slots])             # outputs of that step already on the host
            qi, ki, vi, dOi = in_dev[slot]
            oo, ll, dqo, dko, dvo = out_dev[slot]
            prepare_all((qi, ki, vi, dOi))
            B.attn_fp8_fwd(params, qq, kq, vq, o=oo, lse=ll, workspace=ws)
            B.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, ll, delta=delta, workspace=ws)
            B.attn_fp8_bwd(params, qq, kq, vq, dOq, ll, delta, dq=dqo, dk=dko, dv=dvo, workspace=ws)
            comp_done[i] = torch.cuda.Event(); comp_done[i].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(comp_done[i])
                for src, dst in zip(out_dev[slot], outs_host[slot]):
                    dst.copy_(src, non_blocking=True)
                out_done[i] = torch.cuda.Event(); out_done[i].record(s_out)
        last.record(s_out)
        torch.cuda.synchronize()
        return first.elapsed_time(last)

    e2e_steps = 0 if args.no_e2e else max(4, args.steps)
    e2e_ms = 1e-9
    if e2e_steps:
        e2e_run(3)
        barrier()
        e2e_ms = e2e_run(e2e_steps)
        barrier()
        B.attn_fp8_read_status(ws)
    outs_host = outs_host[0]
    h2d = sum(t.numel() * t.element_size() for t in host)
    d2h = sum(t.numel() * t.element_size() for t in outs_host)

    # ---- max over ranks -----------------------------------------------------------------------
    from paper_2609_37852_b200 import replicas
    total_ms, e2e_ms = replicas.max_over_ranks([total_ms, e2e_ms], device=dev)
    if sustained is not None:
        sustained["ms_per_step"] = replicas.max_over_ranks([sustained["ms_per_step"]], device=dev)[0]

    fwd_flops, bwd_flops = w.credited_flops()
    credited = fwd_flops + bwd_flops
    value = replicas.aggregate_rate(credited * args.steps, world, total_ms * 1e-3) / 1e12
    e2e_value = replicas.aggregate_rate(credited * e2e_steps, world, e2e_ms * 1e-3) / 1e12 if e2e_steps else None

    step_ms = total_ms / args.steps
    # ---- roofline of the dominant kernel ------------------------------------------------------
    peaks = _measured_peaks()
    attn_stages = {n: stage_ms[n] for n in PRODUCTS}
    dominant = max(attn_stages, key=attn_stages.get)
    c = 1 if w.causal else 2
    pairs2 = c * w.batch * w.heads_q * w.seqlen * w.seqlen                          # 2 x (N^2 / 2) pairs per head
    n_qk, n_v = PRODUCTS[dominant]
    kernel_flops = pairs2 * (n_qk * w.head_dim_qk + n_v * w.head_dim_v)
    achieved = kernel_flops / (stage_ms[dominant] * 1e-3) / 1e12
    sc = stage_clocks
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    peak, which, clock_peak, dtype_div = roofline_peaks(sc, peaks, bf16_mode, sms)

    def tensor_roofline(a, name):
        return {"bound": "tensor", "achieved": a, "peak": peak, "unit": "TFLOP/s", "frac": a / peak,
                "frac_of_cublas_bf16_x2": a / peak,       # the same as frac, under the name of what the peak is
                "frac_of_nominal_peak": a / (NOMINAL_FP8_TFLOPS / dtype_div),
                "frac_of_clock_normalised_peak": a / clock_peak if clock_peak else None,
                "frac_of_measured_fp8_mma_rate": a / measured_fp8 if measured_fp8 else None,
                "traffic": NCU_TRAFFIC_BYTES.get(name) if (w.name == WORKLOAD and not bf16_mode) else None}
    roofline = dict(kernel=dominant, **tensor_roofline(achieved, dominant))
    roofline["peak_source"] = (f"{peaks['source']} {which} bf16 {peaks['bf16_' + which]} TFLOP/s"
                               + ("" if bf16_mode else f" x {FP8_OVER_BF16} (nominal fp8:bf16)")
                               + f"; stage loop ran at a median {sc.get('sm_mhz')} MHz of {sc.get('sm_max_mhz')} MHz")
    # the same figure for every kernel of the step (the operand preparation against the HBM copy bandwidth)
    rooflines = {}
    for name, (nq, nv) in PRODUCTS.items():
        a = pairs2 * (nq * w.head_dim_qk + nv * w.head_dim_v) / (stage_ms[name] * 1e-3) / 1e12
        rooflines[name] = tensor_roofline(a, name)
    n_el = w.batch * w.seqlen * (w.heads_q * (w.head_dim_qk + w.head_dim_v) + w.heads_kv * (w.head_dim_qk + w.head_dim_v))
    src_bytes = 2 if w.dtype == "bf16" else 4
    prep_bytes = n_el * (src_bytes + (2 * 2 if bf16_mode else 2 + 2.0 / 32))          # read once, two copies (+ their scale bytes)
    gbs = prep_bytes / (stage_ms["quantize"] * 1e-3) / 1e9
    rooflines["quantize"] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s", "frac": gbs / peaks["hbm"],
                             "traffic": NCU_TRAFFIC_BYTES.get("quantize") if (w.name == WORKLOAD and not bf16_mode) else None}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if bf16_mode else "fp8_e4m3", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.batch, "heads_q": w.heads_q, "heads_kv": w.heads_kv,
                   "seqlen": w.seqlen, "head_dim": w.head_dim_qk, "head_dim_v": w.head_dim_v, "causal": w.causal,
                   "delta_mode": "matched", "precision": args.precision,
                   "l2": "working set per step (>500 MB) exceeds the 126 MB L2", "parallelism": f"replicas x{world}",
                   "step": ("transposed BF16 copies of Q,K,V,dO" if bf16_mode else "quantize(Q,K,V,dO)")
                           + " + fwd + matched delta + dQ + dK/dV"},
        "pct_of_nominal_fp8_peak": 100.0 * value / world / NOMINAL_FP8_TFLOPS,
        "target": "north_star asks for >= 50 % of the nominal dense FP8 peak on this workload: not met",
        "measured_fp8_mma_tflops": measured_fp8,
        "merged_pass_dq_reduction": dq_reduction,
        "pct_of_measured_fp8_mma_rate": (100.0 * value / world / measured_fp8) if measured_fp8 else None,
        "sustained": (None if sustained is None else dict(
            sustained, value=replicas.aggregate_rate(credited, world, sustained["ms_per_step"] * 1e-3) / 1e12, unit=UNIT,
            note="the same step looped back to back for about --sustained-seconds: the rate under the power cap")),
        "pct_of_nominal_peak_of_dtype": 100.0 * value / world / (NOMINAL_FP8_TFLOPS / (FP8_OVER_BF16 if bf16_mode else 1.0)),
        "stage_ms": stage_ms,
        "stage_timing": "a second loop of the same steps, after the timed region, with an event at every stage boundary "
                        "(the timed region has none: an event costs a few microseconds); bwd = the overlapped gradient "
                        "call, bwd_dq and bwd_dkdv = its two kernels as separate, serialised calls; the rooflines use "
                        "these durations and the clocks sampled during this loop (stage_clocks)",
        "stage_clocks": stage_clocks,
        # the timed step less the operand preparation (the paper's accounting), and less the forward
        "attn_only_tflops": credited / ((step_ms - stage_ms["quantize"]) * 1e-3) / 1e12,
        "fwd_tflops": fwd_flops / (stage_ms["fwd"] * 1e-3) / 1e12,
        "bwd_tflops": bwd_flops / ((step_ms - stage_ms["quantize"] - stage_ms["fwd"]) * 1e-3) / 1e12,
        "bwd_tflops_serialised": bwd_flops / ((stage_ms["bwd_delta"] + stage_ms["bwd_dq"] + stage_ms["bwd_dkdv"]) * 1e-3) / 1e12,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / e2e_steps if e2e_steps else None},
        "gpu_launches": kernels_per_step * args.steps,
        "roofline": roofline,
        "rooflines": rooflines,
    }

    # ---- row-sum residual of dS (the metric's second half), from one untimed instrumented pass -------
    if rank == 0:
        _, rs, ra, ps, pa, _ = B.attn_fp8_bwd_dq_postcast(params, qq, kq, vq, dOq, lse, delta, dq=dq, workspace=ws)
        B.attn_fp8_read_status(ws)
        _, _, _, dust, _ = B.attn_fp8_bwd_dq_rowprobe(params, qq, kq, vq, dOq, lse, delta, dq=dq, workspace=ws)
        B.attn_fp8_read_status(ws)
        line["rowsum_ds_residual"] = dict(residual_statistics(rs, ra, ps, dk, lse=lse, dust=dust), delta_mode="matched")

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample_tokens = 2048
        small = w.scaled(heads_q=w.heads_q // w.heads_kv, heads_kv=1, seqlen=sample_tokens)
        sq, sk, sv, sdO = workloads.make_inputs(small)
        t0 = time.perf_counter()
        flops = oracle_step(w, sample_tokens, sq, sk, sv, sdO, args.precision)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {
            "value": flops / dt / 1e12, "unit": UNIT, "cores": _cores_used(), "kind": "oracle", "seconds": dt,
            "sample": f"causal prefix of {sample_tokens} tokens of one KV group ({small.heads_q} query heads) of {w.name}",
        }
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
