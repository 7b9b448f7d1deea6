"""Edge cases of the CUDA path: smallest shapes, head-group extremes, batches, argument errors on the device."""
import numpy as np
import pytest
import torch

from oracle import attention as A
from oracle import mxfp8
from paper_2609_37852_b200 import workloads
from tests.util import rel_fro, to_np, worst_row_error

pytestmark = pytest.mark.gpu


def _full_pass(w, tensors, bf16=False):
    from paper_2609_37852_b200 import binding as B
    params = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                          w.softmax_scale, precision=B.ATTN_PREC_BF16 if bf16 else B.ATTN_PREC_MXFP8)
    prep = B.attn_fp8_prepare_bf16 if bf16 else B.attn_fp8_quantize
    qq, kq, vq, dOq = (prep(x.cuda()) for x in tensors)
    o, lse, ws = B.attn_fp8_fwd(params, qq, kq, vq)
    delta, ws = B.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, workspace=ws)
    dq, dk, dv, rs, ra, ws = B.attn_fp8_bwd(params, qq, kq, vq, dOq, lse, delta, diagnostics=True, workspace=ws)
    B.attn_fp8_read_status(ws)
    return dict(o=o, lse=lse, delta=delta, dq=dq, dk=dk, dv=dv, rs=rs, ra=ra)


def _check(w, tensors, got, prec="mxfp8"):
    qn, kn, vn, dOn = (to_np(x) for x in tensors)
    O, LSE = A.emu_forward(qn, kn, vn, w.softmax_scale, w.causal, prec=prec)
    assert rel_fro(to_np(got["o"]), O) <= 2e-3
    assert rel_fro(to_np(got["lse"]), LSE) <= 2e-3
    lse, delta = to_np(got["lse"]), to_np(got["delta"])
    D = A.emu_delta(qn, kn, vn, dOn, lse, w.softmax_scale, w.causal, prec=prec)
    assert rel_fro(delta, D) <= 1e-4
    dQ, dK, dV, rs, ra = A.emu_backward(qn, kn, vn, dOn, lse, delta, w.softmax_scale, w.causal, prec=prec)
    assert rel_fro(to_np(got["dq"]), dQ) <= 5e-3
    assert rel_fro(to_np(got["dk"]), dK) <= 5e-3
    assert rel_fro(to_np(got["dv"]), dV) <= 5e-3
    assert worst_row_error(to_np(got["o"]), O) <= 2e-2
    for n_, ref in (("dq", dQ), ("dk", dK), ("dv", dV)):
        assert worst_row_error(to_np(got[n_]), ref) <= 5e-2, n_


@pytest.mark.parametrize("name,kw", [
    ("tiny", dict(seqlen=128)),                                         # one tile, non-causal, d = 64
    ("tiny", dict(seqlen=128, causal=True)),                            # one (diagonal) tile
    ("gqa4k", dict(batch=1, heads_q=1, heads_kv=1, seqlen=128)),        # one tile, d = 128
    ("gqa4k", dict(batch=1, heads_q=2, heads_kv=2, seqlen=256, causal=False)),   # non-causal at d = 128, one head per group
    ("gqa4k", dict(batch=3, heads_q=8, heads_kv=1, seqlen=256)),        # batch of 3, one KV head for eight query heads
    ("gqa8k_outlier", dict(batch=2, heads_q=2, heads_kv=1, seqlen=384)),
])
def test_small_and_extreme_shapes(name, kw):
    w = workloads.WORKLOADS[name].scaled(**kw)
    tensors = workloads.make_inputs(w)
    _check(w, tensors, _full_pass(w, tensors))


@pytest.mark.parametrize("name,kw,bf16", [
    ("mla8k", dict(heads_q=2, heads_kv=2, seqlen=384, causal=False), False),        # wide heads without the causal mask
    ("mla8k", dict(heads_q=4, heads_kv=1, seqlen=256, causal=False), False),
    ("gqa8k_d256", dict(heads_q=2, heads_kv=1, seqlen=384, causal=False), False),
    ("gqa8k_d256", dict(batch=2, heads_q=4, heads_kv=2, seqlen=256), False),         # d = 256 with a batch
    ("gqa4k", dict(batch=1, heads_q=4, heads_kv=2, seqlen=384, causal=False), True),  # BF16 mode, non-causal
    ("tiny", dict(seqlen=384, heads_q=3, heads_kv=3, batch=2), False),               # odd head count, d = 64, FP32 source
    ("tiny", dict(seqlen=384, heads_q=6, heads_kv=2, causal=True), True),            # BF16 mode at d = 64, groups of 3
    ("long64k", dict(heads_q=2, heads_kv=1, seqlen=1152), False),                    # heavy-tailed channel gains, 9 tiles
    ("gqa8k_outlier", dict(batch=3, heads_q=16, heads_kv=1, seqlen=256), False),     # 16 query heads on one KV head
    ("gqa8k_outlier", dict(batch=3, heads_q=6, heads_kv=3, seqlen=640), True),       # BF16 mode, outlier scores: far-key
                                                                                      # probabilities below the BF16 range
    ("mla8k", dict(batch=2, heads_q=6, heads_kv=3, seqlen=384), True),               # BF16 mode at (192, 128)
    ("mla8k", dict(heads_q=2, heads_kv=1, seqlen=256, causal=False), True),
    ("gqa8k_d256", dict(batch=2, heads_q=4, heads_kv=2, seqlen=384), True),          # BF16 mode at (256, 256)
])
def test_shape_and_mode_combinations(name, kw, bf16):
    w = workloads.WORKLOADS[name].scaled(**kw)
    tensors = workloads.make_inputs(w)
    if bf16 and w.dtype != "bf16":
        tensors = tuple(x.to(torch.bfloat16) for x in tensors)
    _check(w, tensors, _full_pass(w, tensors, bf16=bf16), prec="bf16" if bf16 else "mxfp8")


def test_nearly_one_hot_rows_stress():
    """Outlier channels shared by a query head and its KV head: scores with a standard deviation of
    ~70, rows nearly one-hot, the running shift raised (and the output accumulator rescaled) often."""
    w = workloads.WORKLOADS["gqa8k_outlier"].scaled(heads_q=4, heads_kv=2, seqlen=640, recipe="outlier_rope_aligned")
    tensors = workloads.make_inputs(w)
    got = _full_pass(w, tensors)
    qn, kn = to_np(tensors[0]), to_np(tensors[1])
    s = w.softmax_scale * qn[0, 0] @ kn[0, 0].T
    assert s.std() > 30                                                 # the recipe does what it says
    qn, kn, vn, dOn = (to_np(x) for x in tensors)
    O, LSE = A.emu_forward(qn, kn, vn, w.softmax_scale, w.causal)
    assert rel_fro(to_np(got["o"]), O) <= 2e-3 and rel_fro(to_np(got["lse"]), LSE) <= 2e-3
    assert torch.isfinite(got["o"].float()).all() and torch.isfinite(got["lse"]).all()
    lse, delta = to_np(got["lse"]), to_np(got["delta"])
    assert rel_fro(delta, A.emu_delta(qn, kn, vn, dOn, lse, w.softmax_scale, w.causal)) <= 1e-4
    # Nearly every row is one-hot to ~1e-5 and has a vanishing dS, so a head's whole gradient sits in
    # a handful of rows and elements; where the largest of them lies on an E4M3 rounding tie (here
    # one does, 5e-7 away), the float64 oracle and the FP32 kernel round it to neighbouring codes and
    # that single step is percents of dQ.  dQ is therefore bounded loosely as a whole and by the usual
    # tolerance once the single worst row of each head is set aside.
    dQ, dK, dV, _, _ = A.emu_backward(qn, kn, vn, dOn, lse, delta, w.softmax_scale, w.causal)
    errs = {n: rel_fro(to_np(got[n]), r) for n, r in (("dq", dQ), ("dk", dK), ("dv", dV))}
    dq_gpu = to_np(got["dq"])
    row_err = np.linalg.norm(dq_gpu - dQ, axis=-1)                      # [B, Hq, N]
    keep = np.ones_like(row_err, dtype=bool)
    np.put_along_axis(keep, row_err.argmax(axis=-1)[..., None], False, axis=-1)
    errs["dq_without_worst_row"] = float(np.linalg.norm((dq_gpu - dQ)[keep]) / np.linalg.norm(dQ[keep]))
    print("\nstress errors", errs)
    assert errs["dv"] <= 5e-3 and errs["dk"] <= 5e-3
    assert errs["dq"] <= 2e-2 and errs["dq_without_worst_row"] <= 5e-3


def test_first_row_sees_one_key():
    """Causal row 0 attends to key 0 only: P = 1 up to the rounding of LSE, so dS_0 and dQ_0 vanish
    (to FP32 rounding level), and O_0 is V^c_0 times the ratio of the cast probability to the exact one."""
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=2, heads_kv=1, seqlen=256)
    tensors = workloads.make_inputs(w)
    got = _full_pass(w, tensors)
    qn, kn, vn = (to_np(x) for x in tensors[:3])
    O0, _ = A.emu_forward(qn, kn, vn, w.softmax_scale, w.causal, rows=[0])
    assert np.abs(to_np(got["o"][0, :, 0]) - O0[0, :, 0]).max() <= 2.0 ** -7 * np.abs(O0).max()
    v_c = mxfp8.fake_quant(vn[0, 0], 0)                                 # blocks along tokens
    ratio = to_np(got["o"][0, 0, 0]) / np.where(v_c[0] == 0, 1.0, v_c[0])
    assert np.all(np.abs(ratio[v_c[0] != 0] - 1.0) <= 2.0 ** -4 + 2.0 ** -7)      # one E4M3 half-ulp and the BF16 store
    assert float(got["dq"][0, :, 0].float().abs().max()) <= 1e-5 * float(got["dq"].float().abs().max())
    assert float(got["rs"][0, :, 0].abs().max()) <= 1e-6 * float(got["ra"].abs().max())


def test_zero_output_gradient_gives_zero_gradients():
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=2, heads_kv=1, seqlen=256)
    q, k, v, dO = workloads.make_inputs(w)
    got = _full_pass(w, (q, k, v, torch.zeros_like(dO)))
    for key in ("delta", "dq", "dk", "dv", "rs", "ra"):
        assert float(got[key].float().abs().max()) == 0.0, key


@pytest.mark.parametrize("name,kw,bf16", [
    ("gqa4k", dict(batch=2, heads_q=4, heads_kv=2, seqlen=384), False),
    ("gqa4k", dict(batch=1, heads_q=2, heads_kv=1, seqlen=256), True),
    ("mla8k", dict(heads_q=2, heads_kv=2, seqlen=256), False),
    ("gqa8k_d256", dict(heads_q=2, heads_kv=1, seqlen=256), False),
    ("mla8k", dict(heads_q=2, heads_kv=2, seqlen=256), True),
    ("gqa8k_d256", dict(heads_q=2, heads_kv=1, seqlen=256), True),
])
def test_every_output_element_is_written(name, kw, bf16):
    """Outputs pre-filled with NaN: a region no CTA writes would survive the call."""
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS[name].scaled(**kw)
    tensors = [x.cuda() for x in workloads.make_inputs(w)]
    params = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, w.head_dim_qk, w.head_dim_v, w.causal,
                          w.softmax_scale, precision=B.ATTN_PREC_BF16 if bf16 else B.ATTN_PREC_MXFP8)
    prep = B.attn_fp8_prepare_bf16 if bf16 else B.attn_fp8_quantize
    qq, kq, vq, dOq = (prep(x) for x in tensors)
    nan = lambda shape, dt: torch.full(shape, float("nan"), dtype=dt, device="cuda")
    Bn, Hq, Hkv, N = w.batch, w.heads_q, w.heads_kv, w.seqlen
    o, lse = nan((Bn, Hq, N, w.head_dim_v), torch.bfloat16), nan((Bn, Hq, N), torch.float32)
    _, _, ws = B.attn_fp8_fwd(params, qq, kq, vq, o=o, lse=lse)
    delta = nan((Bn, Hq, N), torch.float32)
    B.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, delta=delta, workspace=ws)
    dq, dk, dv = (nan((Bn, h, N, d), torch.bfloat16) for h, d in ((Hq, w.head_dim_qk), (Hkv, w.head_dim_qk), (Hkv, w.head_dim_v)))
    stats = [nan((Bn, Hq, N), torch.float32) for _ in range(4)]
    B.attn_fp8_bwd_dkdv(params, qq, kq, vq, dOq, lse, delta, dk=dk, dv=dv, workspace=ws)
    c = params.c_struct()
    import ctypes
    B._check(B._lib.attn_fp8_bwd_dq_postcast(ctypes.byref(c), qq.c_struct(), kq.c_struct(), vq.c_struct(), dOq.c_struct(),
                                             B._ptr(lse), B._ptr(delta), B._ptr(dq), *(B._ptr(t) for t in stats),
                                             B._ptr(ws), ws.numel(), B._stream(None)))
    B.attn_fp8_read_status(ws)
    for nm, t in dict(o=o, lse=lse, delta=delta, dq=dq, dk=dk, dv=dv, rs=stats[0], ra=stats[1], ps=stats[2], pa=stats[3]).items():
        assert not torch.isnan(t.float()).any(), nm


def test_argument_errors_on_the_device():
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=2, heads_kv=1, seqlen=256)
    q, k, v, dO = (x.cuda() for x in workloads.make_inputs(w))
    qq, kq, vq = (B.attn_fp8_quantize(x) for x in (q, k, v))
    ok = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, 128, 128, True, w.softmax_scale)
    # workspace too small
    with pytest.raises(B.AttnFp8Error) as e:
        B.attn_fp8_fwd(ok, qq, kq, vq, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4
    # missing orientation: the forward needs the column copy of V
    v_rows_only = B.attn_fp8_quantize(v, want_col=False)
    with pytest.raises(B.AttnFp8Error) as e:
        B.attn_fp8_fwd(ok, qq, kq, v_rows_only)
    assert e.value.status == 1 and "v.col_codes" in str(e.value)
    # unsupported head dims, unknown precision, unknown delta mode
    for bad, status in ((B.AttnParams(1, 256, 2, 1, 96, 96, True, 0.1), 2),
                        (B.AttnParams(1, 256, 2, 1, 128, 128, True, 0.1, precision=7), 1),
                        (B.AttnParams(1, 200, 2, 1, 128, 128, True, 0.1), 2)):
        with pytest.raises(B.AttnFp8Error) as e:
            B.attn_fp8_fwd(bad, qq, kq, vq)
        assert e.value.status == status
    o, lse, ws = B.attn_fp8_fwd(ok, qq, kq, vq)
    dOq = B.attn_fp8_quantize(dO)
    bad_mode = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, 128, 128, True, w.softmax_scale, delta_mode=9)
    with pytest.raises(B.AttnFp8Error) as e:
        B.attn_fp8_bwd_delta(bad_mode, qq, kq, vq, dOq, lse)
    assert e.value.status == 1
    # misaligned output pointer
    o_mis = torch.empty(o.numel() + 8, dtype=torch.bfloat16, device="cuda")[1:1 + o.numel()].view_as(o)
    with pytest.raises(B.AttnFp8Error) as e:
        B.attn_fp8_fwd(ok, qq, kq, vq, o=o_mis)
    assert e.value.status == 3
    # the context is still usable
    o2, lse2, ws = B.attn_fp8_fwd(ok, qq, kq, vq)
    B.attn_fp8_read_status(ws)
    assert torch.equal(o, o2) and torch.equal(lse, lse2)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_prepare_bf16_is_an_exact_rounding_and_transpose(dtype):
    from paper_2609_37852_b200 import binding as B
    g = torch.Generator().manual_seed(5)
    x = torch.randn((2, 3, 256, 128), generator=g).to(dtype).cuda()
    t = B.attn_fp8_prepare_bf16(x)
    want = x.to(torch.bfloat16)
    assert torch.equal(t.row_codes, want)
    assert torch.equal(t.col_codes, want.transpose(2, 3).contiguous())


@pytest.mark.parametrize("d", [192, 256])
def test_quantize_wide_heads_bit_exact(d):
    """Two 512-byte scale tiles per 128-row tile in both orientations."""
    from paper_2609_37852_b200 import binding as B
    g = torch.Generator().manual_seed(d)
    x = (torch.randn((1, 2, 256, d), generator=g) * torch.exp2(torch.randint(-6, 6, (1, 2, 256, 1), generator=g).float())
         ).to(torch.bfloat16)
    t = B.attn_fp8_quantize(x.cuda())
    xn = to_np(x)
    for axis, codes, scales, rows, cols in ((-1, t.row_codes, t.row_scales, 256, d), (-2, t.col_codes, t.col_scales, d, 256)):
        c_or, e_or = mxfp8.quantize(xn if axis == -1 else np.swapaxes(xn, -1, -2), axis=-1)
        assert np.array_equal(codes.cpu().numpy(), c_or)
        got_e = B.unpack_scales(scales, 1, 2, rows, cols).cpu().numpy()
        assert np.array_equal(got_e, e_or)


def test_expired_wait_is_reported_and_the_context_survives():
    """A bounded device-side wait that runs out (a barrier nothing completes, ~2 ms limit) sets the
    workspace status word; read_status reports ATTN_ERR_TIMEOUT; later calls work as before."""
    import time
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=2, heads_kv=1, seqlen=256)
    q, k, v, dO = (x.cuda() for x in workloads.make_inputs(w))
    qq, kq, vq = (B.attn_fp8_quantize(x) for x in (q, k, v))
    params = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, 128, 128, True, w.softmax_scale)
    o, lse, ws = B.attn_fp8_fwd(params, qq, kq, vq)
    B.attn_fp8_read_status(ws)
    t0 = time.perf_counter()
    B.attn_fp8_selftest_timeout(ws)
    with pytest.raises(B.AttnFp8Error) as e:
        B.attn_fp8_read_status(ws)
    assert e.value.status == 7
    assert time.perf_counter() - t0 < 1.0                              # it gave up within its limit
    B.attn_fp8_read_status(ws)                                         # reported once: the read cleared it
    # the status is sticky across calls: a failure is still reported after later, healthy calls
    B.attn_fp8_selftest_timeout(ws)
    o2, lse2, ws = B.attn_fp8_fwd(params, qq, kq, vq, workspace=ws)
    with pytest.raises(B.AttnFp8Error) as e:
        B.attn_fp8_read_status(ws)
    assert e.value.status == 7
    assert torch.equal(o, o2) and torch.equal(lse, lse2)               # the forward itself was healthy
    o3, lse3, ws = B.attn_fp8_fwd(params, qq, kq, vq, workspace=ws)
    B.attn_fp8_read_status(ws)
    assert torch.equal(o, o3) and torch.equal(lse, lse3)
    # a workspace the caller made has to be initialised once: garbage in the status word reads as an error
    raw = torch.full((B.attn_fp8_workspace_bytes(params, 0),), 0xFF, dtype=torch.uint8, device="cuda")
    B.attn_fp8_workspace_init(raw)
    B.attn_fp8_fwd(params, qq, kq, vq, workspace=raw)
    B.attn_fp8_read_status(raw)


def test_header_counters_are_cleared_by_the_call_that_uses_them():
    """Beyond the status word the workspace header holds the ticket counter of the persistent dQ
    kernel; the gradient call clears it itself, so whatever an earlier user left there is harmless."""
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS["gqa4k"].scaled(batch=1, heads_q=4, heads_kv=2, seqlen=512)
    tensors = [x.cuda() for x in workloads.make_inputs(w)]
    params = B.AttnParams(w.batch, w.seqlen, w.heads_q, w.heads_kv, 128, 128, True, w.softmax_scale)
    (qq, kq, vq, dOq), _ = B.attn_fp8_quantize_batch(tensors)
    o, lse, ws = B.attn_fp8_fwd(params, qq, kq, vq)
    delta, ws = B.attn_fp8_bwd_delta(params, qq, kq, vq, dOq, lse, workspace=ws)
    ref = B.attn_fp8_bwd(params, qq, kq, vq, dOq, lse, delta, workspace=ws)
    B.attn_fp8_read_status(ws)
    dirty = torch.full((ws.numel(),), 0x5A, dtype=torch.uint8, device="cuda")
    dirty[:4] = 0                                                       # the status word alone is initialised
    for call in range(2):
        got = B.attn_fp8_bwd(params, qq, kq, vq, dOq, lse, delta, workspace=dirty)
        B.attn_fp8_read_status(dirty)
        for a, b in zip(got[:3], ref[:3]):
            assert torch.equal(a, b), f"call {call}"
        dq_only = B.attn_fp8_bwd_dq(params, qq, kq, vq, dOq, lse, delta, workspace=dirty)
        assert torch.equal(dq_only[0], ref[0])


def test_random_shapes_and_modes():
    """A seeded sweep over batch, head grouping, sequence length, mask, recipe and operand mode, every
    case checked against the oracle: the net under the persistent / ticket-scheduled kernels, whose
    item lists depend on all of these."""
    import random
    rnd = random.Random(20260937852)
    done = 0
    while done < 16:
        base = rnd.choice(["tiny", "gqa4k", "gqa8k_outlier", "mla8k", "gqa8k_d256", "long64k"])
        hkv = rnd.choice([1, 2, 3])
        kw = dict(batch=rnd.choice([1, 1, 2, 3]), heads_kv=hkv, heads_q=hkv * rnd.choice([1, 2, 4, 5]),
                  seqlen=128 * rnd.choice([1, 2, 3, 4, 5, 6]), causal=rnd.choice([True, True, False]))
        w = workloads.WORKLOADS[base].scaled(**kw)
        if w.batch * w.heads_q * w.seqlen * w.seqlen > 2 * 8 * 768 * 768:
            continue                                                    # keep the oracle's share to seconds
        bf16 = rnd.random() < 0.25
        tensors = workloads.make_inputs(w)
        if bf16 and w.dtype != "bf16":
            tensors = tuple(x.to(torch.bfloat16) for x in tensors)
        try:
            _check(w, tensors, _full_pass(w, tensors, bf16=bf16), prec="bf16" if bf16 else "mxfp8")
        except AssertionError as e:
            raise AssertionError(f"{base} {kw} bf16={bf16}") from e
        done += 1


def test_measurement_aids():
    """The two measurement entry points of the benchmark: the bare block-scaled MMA rate (a plausible
    number, status word clean) and the dQ-reduction probe (its adds land where they should)."""
    from paper_2609_37852_b200 import binding as B
    ws = B.new_workspace(256, torch.device("cuda"))
    tflops = B.attn_fp8_measure_mma_peak(ws)
    B.attn_fp8_read_status(ws)
    assert 1000.0 < tflops < 6000.0, tflops
    params = B.AttnParams(1, 1024, 4, 2, 128, 128, True, 0.1)
    dq = torch.empty((1, 4, 1024, 128), dtype=torch.float32, device="cuda")
    ms, nbytes = B.attn_fp8_measure_dq_reduction(params, dq)
    assert ms > 0 and nbytes == 4 * (8 * 9 // 2) * 2 * 64 * 128 * 4
    want = (torch.arange(1024, device="cuda") // 128 + 1).float()          # key tiles a causal row sees
    assert torch.equal(dq, want[None, None, :, None].expand_as(dq))
