"""attn_fp8_quantize against the oracle quantiser: codes and scale bytes bit for bit."""
import numpy as np
import pytest
import torch

from oracle import mxfp8
from paper_2609_37852_b200 import workloads
from tests.util import to_np

pytestmark = pytest.mark.gpu


def _check(x: torch.Tensor):
    from paper_2609_37852_b200 import binding
    B, H, N, d = x.shape
    qt = binding.attn_fp8_quantize(x.cuda())
    torch.cuda.synchronize()
    xn = to_np(x)
    rc, rs = mxfp8.quantize(xn, axis=-1)
    cc, cs = mxfp8.quantize(xn, axis=-2)
    assert np.array_equal(qt.row_codes.cpu().numpy(), rc)
    assert np.array_equal(binding.unpack_scales(qt.row_scales, B, H, N, d).cpu().numpy(), rs)
    assert np.array_equal(qt.col_codes.cpu().numpy(), np.swapaxes(cc, -1, -2))
    assert np.array_equal(binding.unpack_scales(qt.col_scales, B, H, d, N).cpu().numpy(), np.swapaxes(cs, -1, -2))
    # padding bytes of the scale tiles are zero
    total = int(qt.row_scales.to(torch.int64).sum()) - int(rs.astype(np.int64).sum())
    assert total == 0
    total = int(qt.col_scales.to(torch.int64).sum()) - int(cs.astype(np.int64).sum())
    assert total == 0


@pytest.mark.parametrize("name,N", [("tiny", 256), ("gqa4k", 384), ("gqa8k_outlier", 256), ("mla8k", 256),
                                    ("gqa8k_d256", 128), ("long64k", 256)])
def test_quantize_workload_inputs_bit_exact(name, N):
    w = workloads.WORKLOADS[name].scaled(seqlen=N, heads_q=min(4, workloads.WORKLOADS[name].heads_q),
                                         heads_kv=min(2, workloads.WORKLOADS[name].heads_kv))
    for x in workloads.make_inputs(w):
        _check(x)


def test_quantize_edge_values():
    g = torch.Generator().manual_seed(7)
    x = torch.randn(1, 2, 128, 64, generator=g)
    x[0, 0, :32, :32] = 0.0                       # all-zero row and column blocks
    x[0, 0, 5, 40] = -0.0
    x[0, 1, 3, :] *= 2.0 ** 60                    # huge and tiny blocks
    x[0, 1, 4, :] *= 2.0 ** -70
    x[0, 1, 64:96, 7] = 448.0                     # exactly on the saturation edge
    x[0, 1, 96:128, 9] = 1.75                     # mantissa exactly 1.75: no bump
    x[0, 1, 96, 10] = 1.7500001
    _check(x)
    _check(x.to(torch.bfloat16))


def test_quantize_single_orientation_and_errors():
    from paper_2609_37852_b200 import binding
    x = torch.randn(1, 1, 128, 96, device="cuda", dtype=torch.bfloat16)
    full = binding.attn_fp8_quantize(x)
    only_row = binding.attn_fp8_quantize(x, want_col=False)
    only_col = binding.attn_fp8_quantize(x, want_row=False)
    torch.cuda.synchronize()
    assert only_row.col_codes is None and torch.equal(only_row.row_codes, full.row_codes)
    assert only_col.row_codes is None and torch.equal(only_col.col_codes, full.col_codes)
    assert torch.equal(only_col.col_scales, full.col_scales)
    with pytest.raises(binding.AttnFp8Error) as e:
        binding.attn_fp8_quantize(torch.randn(1, 1, 100, 64, device="cuda"))
    assert e.value.status == 2


def _same(a, b):
    for f in ("row_codes", "row_scales", "col_codes", "col_scales"):
        x, y = getattr(a, f), getattr(b, f)
        assert (x is None) == (y is None), f
        if x is not None:
            assert torch.equal(x, y), f


@pytest.mark.parametrize("name,kw", [
    ("gqa8k_outlier", dict(heads_q=8, heads_kv=2, seqlen=1024)),        # d = 128, more tiles than resident CTAs
    ("tiny", dict(seqlen=256)),                                          # FP32 source, d = 64, two tiles per tensor
    ("mla8k", dict(heads_q=2, heads_kv=2, seqlen=384)),                  # head dims 192 and 128 in one launch
    ("gqa8k_d256", dict(heads_q=2, heads_kv=1, seqlen=256)),             # d = 256
])
def test_quantize_batch_is_bit_identical_to_single_calls(name, kw):
    """The persistent multi-tensor launch against the oracle (through the single-tensor check) and
    against attn_fp8_quantize on each tensor, orientations as the attention calls need them."""
    from paper_2609_37852_b200 import binding as B
    w = workloads.WORKLOADS[name].scaled(**kw)
    srcs = [x.cuda() for x in workloads.make_inputs(w)]
    want = [(True, True), (True, True), (True, True), (True, True)]
    outs, ws = B.attn_fp8_quantize_batch(srcs, want=want)
    B.attn_fp8_read_status(ws)
    for x, q in zip(srcs, outs):
        _same(q, B.attn_fp8_quantize(x))
    # against the oracle directly, first tensor
    xn = to_np(srcs[0]); Bn, H, N, d = srcs[0].shape
    rc, rs = mxfp8.quantize(xn, axis=-1)
    assert np.array_equal(outs[0].row_codes.cpu().numpy(), rc)
    assert np.array_equal(B.unpack_scales(outs[0].row_scales, Bn, H, N, d).cpu().numpy(), rs)
    # single orientations, outputs prefilled: only what was asked for is written, and all of it
    want = [(True, False), (False, True), (True, True), (False, True)]
    outs2, _ = B.attn_fp8_quantize_batch(srcs, want=want, workspace=ws)
    for q in outs2:
        for f in ("row_codes", "row_scales", "col_codes", "col_scales"):
            if getattr(q, f) is not None:
                getattr(q, f).fill_(0xAB)
    outs2, _ = B.attn_fp8_quantize_batch(srcs, outs=outs2, workspace=ws)
    B.attn_fp8_read_status(ws)
    for (wr, wc), q, full in zip(want, outs2, outs):
        assert (q.row_codes is not None) == wr and (q.col_codes is not None) == wc
        if wr:
            assert torch.equal(q.row_codes, full.row_codes) and torch.equal(q.row_scales, full.row_scales)
        if wc:
            assert torch.equal(q.col_codes, full.col_codes) and torch.equal(q.col_scales, full.col_scales)


def test_quantize_batch_single_tile_ring_and_errors():
    from paper_2609_37852_b200 import binding as B
    g = torch.Generator().manual_seed(5)
    # FP32 source with d = 256: two source tiles do not fit in shared memory, the ring holds one
    xs = [torch.randn((1, 2, 256, 256), generator=g).cuda(), torch.randn((1, 1, 128, 256), generator=g).cuda()]
    outs, ws = B.attn_fp8_quantize_batch(xs)
    B.attn_fp8_read_status(ws)
    for x, q in zip(xs, outs):
        _same(q, B.attn_fp8_quantize(x))
    with pytest.raises(B.AttnFp8Error) as e:                               # mixed source dtypes
        B.attn_fp8_quantize_batch([xs[0], xs[1].to(torch.bfloat16)])
    assert e.value.status == 1
    with pytest.raises(B.AttnFp8Error) as e:                               # too many tensors
        B.attn_fp8_quantize_batch([xs[1]] * 9)
    assert e.value.status == 1
    with pytest.raises(B.AttnFp8Error) as e:                               # status workspace too small
        B.attn_fp8_quantize_batch([xs[1]], workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4


def test_quantize_batch_random_job_mixes_bit_exact():
    """Seeded mixes of one to eight tensors with head dims 32 ... 256 (those without a compile-time
    instance included), both source dtypes, zero columns and random orientations: codes, scale
    bytes and the zero padding of the scale tiles against the oracle, bit for bit."""
    import random
    from paper_2609_37852_b200 import binding as B
    rnd = random.Random(3)
    g = torch.Generator().manual_seed(11)
    for trial in range(8):
        dt = rnd.choice([torch.bfloat16, torch.float32])
        xs = []
        for j in range(rnd.choice([1, 2, 3, 5, 8])):
            shape = (rnd.choice([1, 2]), rnd.choice([1, 3]), 128 * rnd.choice([1, 2, 3]), 32 * rnd.choice([1, 2, 3, 4, 5, 6, 7, 8]))
            x = torch.randn(shape, generator=g) * (10.0 ** rnd.uniform(-3, 3))
            if rnd.random() < 0.3:
                x[..., ::7] = 0
            xs.append(x.to(dt).cuda())
        want = [(rnd.random() < 0.8, True) if rnd.random() < 0.5 else (True, rnd.random() < 0.8) for _ in xs]
        outs, ws = B.attn_fp8_quantize_batch(xs, want=want)
        B.attn_fp8_read_status(ws)
        for x, q, (wr, wc) in zip(xs, outs, want):
            Bn, H, N, d = x.shape
            xn = to_np(x)
            if wr:
                rc, rs = mxfp8.quantize(xn, axis=-1)
                assert np.array_equal(q.row_codes.cpu().numpy(), rc), (trial, x.shape)
                assert np.array_equal(B.unpack_scales(q.row_scales, Bn, H, N, d).cpu().numpy(), rs), (trial, x.shape)
                assert int(q.row_scales.to(torch.int64).sum()) == int(rs.astype(np.int64).sum())
            else:
                assert q.row_codes is None
            if wc:
                cc, cs = mxfp8.quantize(xn, axis=-2)
                assert np.array_equal(q.col_codes.cpu().numpy(), np.swapaxes(cc, -1, -2)), (trial, x.shape)
                assert np.array_equal(B.unpack_scales(q.col_scales, Bn, H, d, N).cpu().numpy(), np.swapaxes(cs, -1, -2)), (trial, x.shape)
                assert int(q.col_scales.to(torch.int64).sum()) == int(cs.astype(np.int64).sum())
            else:
                assert q.col_codes is None
