"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "attn_fp8.h")


@pytest.fixture(scope="module")
def lib_path():
    from paper_2609_37852_b200 import build
    return build.build()


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(attn_fp8_\w+)\s*\(", text)))


def test_header_declares_the_four_entry_points():
    names = _declared_functions()
    for n in ("attn_fp8_quantize", "attn_fp8_fwd", "attn_fp8_bwd_delta", "attn_fp8_bwd"):
        assert n in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in _declared_functions():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols(lib_path):
    from paper_2609_37852_b200 import binding
    assert sorted(binding.EXPORTED_SYMBOLS) == _declared_functions()


def test_scale_offset_rule(lib_path):
    from paper_2609_37852_b200 import binding
    for n_blocks in (2, 4, 6, 8, 64):
        seen = set()
        for row in range(0, 256):
            for blk in range(n_blocks):
                want = ((row // 128) * ((n_blocks + 3) // 4) + blk // 4) * 512 + (row % 32) * 16 \
                    + ((row % 128) // 32) * 4 + blk % 4
                got = binding.attn_fp8_scale_offset(row, blk, n_blocks)
                assert got == want
                seen.add(got)
        assert len(seen) == 256 * n_blocks                      # a permutation: no two scales collide
    assert binding.attn_fp8_scale_bytes(2, 3, 256, 128) == 2 * 3 * 2 * 1 * 512
    assert binding.attn_fp8_scale_bytes(1, 1, 64, 256) == 1 * 2 * 512
    assert binding.attn_fp8_scale_bytes(1, 1, 192, 128) == 2 * 512


def test_unpack_scales_inverts_the_tiling(lib_path):
    import torch
    from paper_2609_37852_b200 import binding
    B, H, rows, cols = 1, 2, 256, 192
    nbytes = binding.attn_fp8_scale_bytes(B, H, rows, cols)
    flat = torch.zeros(nbytes, dtype=torch.uint8)
    plain = torch.randint(1, 255, (B, H, rows, cols // 32), dtype=torch.uint8)
    slab = nbytes // (B * H)
    for s in range(B * H):
        for r in range(rows):
            for k in range(cols // 32):
                flat[s * slab + binding.attn_fp8_scale_offset(r, k, cols // 32)] = plain[s // H, s % H, r, k]
    assert torch.equal(binding.unpack_scales(flat, B, H, rows, cols), plain)


def test_validation_errors_without_touching_a_gpu(lib_path):
    from paper_2609_37852_b200 import binding
    st = binding._lib.attn_fp8_quantize(None, 0, 1, 1, 128, 128, binding._QTensor(), None)
    assert st == 1 and "src" in binding.attn_fp8_last_error()
    st = binding._lib.attn_fp8_quantize(ctypes.c_void_p(16), 0, 1, 1, 100, 128, binding._QTensor(), None)
    assert st == 2
    st = binding._lib.attn_fp8_quantize(ctypes.c_void_p(8), 0, 1, 1, 128, 128, binding._QTensor(), None)
    assert st == 3
    p = binding.AttnParams(1, 128, 3, 2, 128, 128, True, 0.1).c_struct()
    q = binding._QTensor()
    st = binding._lib.attn_fp8_fwd(ctypes.byref(p), q, q, q, None, None, None, 0, None)
    assert st == 1 and "heads_q" in binding.attn_fp8_last_error()
    p = binding.AttnParams(1, 128, 4, 2, 96, 96, True, 0.1).c_struct()
    st = binding._lib.attn_fp8_fwd(ctypes.byref(p), q, q, q, None, None, None, 0, None)
    assert st == 2
    # more rows than the kernels' 32-bit row coordinates reach: refused before any launch
    p = binding.AttnParams(64, 1 << 20, 64, 8, 128, 128, True, 0.1).c_struct()
    st = binding._lib.attn_fp8_fwd(ctypes.byref(p), q, q, q, None, None, None, 0, None)
    assert st == 2 and "2^31" in binding.attn_fp8_last_error()


def test_batched_quantiser_and_workspace_validation_without_a_gpu(lib_path):
    """Argument checks of attn_fp8_quantize_batch and attn_fp8_workspace_init run before any device call."""
    from paper_2609_37852_b200 import binding
    lib = binding._lib
    fake = ctypes.c_void_p(4096)                                   # aligned, never dereferenced on these paths
    out = binding._QTensor(fake, fake, fake, fake)
    ok = binding._QuantizeJob(fake, binding.ATTN_SRC_BF16, 1, 1, 128, 128, out)
    jobs = (binding._QuantizeJob * 2)(ok, ok)
    assert lib.attn_fp8_quantize_batch(None, 1, fake, 256, None) == 1
    assert lib.attn_fp8_quantize_batch(jobs, 0, fake, 256, None) == 1
    assert lib.attn_fp8_quantize_batch(jobs, binding.ATTN_QUANTIZE_MAX_JOBS + 1, fake, 256, None) == 1
    jobs[1] = binding._QuantizeJob(fake, binding.ATTN_SRC_FP32, 1, 1, 128, 128, out)
    assert lib.attn_fp8_quantize_batch(jobs, 2, fake, 256, None) == 1 and "src_dtype" in binding.attn_fp8_last_error()
    jobs[1] = binding._QuantizeJob(fake, binding.ATTN_SRC_BF16, 1, 1, 192, 128, out)      # N not a multiple of 128
    assert lib.attn_fp8_quantize_batch(jobs, 2, fake, 256, None) == 2
    jobs[1] = binding._QuantizeJob(fake, binding.ATTN_SRC_BF16, 1, 1, 128, 128, binding._QTensor(fake, None, None, None))
    assert lib.attn_fp8_quantize_batch(jobs, 2, fake, 256, None) == 1      # codes without their scales
    assert lib.attn_fp8_workspace_init(None, 256, None) == 4
    assert lib.attn_fp8_workspace_init(fake, 16, None) == 4
    assert lib.attn_fp8_workspace_init(ctypes.c_void_p(4100), 256, None) == 3
    # a NULL workspace means the built-in scratch array of the current device: without a device the call
    # stops at the device check (ATTN_ERR_CUDA), with one it reads that array's status word
    import torch
    if not torch.cuda.is_available():
        assert lib.attn_fp8_read_status(None, None) == 6
