"""ctypes binding of ``libattnfp8.so`` -- same entry-point names as ``include/attn_fp8.h``.

Argument marshalling only: tensors are torch CUDA tensors whose device pointers
are handed to the C ABI; every step of the attention path runs in the
library's kernels.  Importing this module fails loudly when the library has
not been built (``python -m paper_2609_37852_b200.build``): there is no
fallback path.
"""
import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libattnfp8.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build the CUDA library first (python -m paper_2609_37852_b200.build); "
        "this package has no CPU or eager fallback")
_lib = ctypes.CDLL(LIB_PATH)

ATTN_OK = 0
STATUS_NAMES = {0: "ATTN_OK", 1: "ATTN_ERR_INVALID_ARG", 2: "ATTN_ERR_UNSUPPORTED", 3: "ATTN_ERR_ALIGNMENT",
                4: "ATTN_ERR_WORKSPACE", 5: "ATTN_ERR_ARCH", 6: "ATTN_ERR_CUDA", 7: "ATTN_ERR_TIMEOUT"}
ATTN_PREC_MXFP8, ATTN_PREC_BF16, ATTN_PREC_MXFP8_PROTECTED_DP = 0, 1, 2
ATTN_DELTA_MATCHED, ATTN_DELTA_STALE, ATTN_DELTA_CONSISTENT_DO = 0, 1, 2
ATTN_SRC_BF16, ATTN_SRC_FP32 = 0, 1
ATTN_WS_FWD, ATTN_WS_BWD_DELTA, ATTN_WS_BWD = 0, 1, 2

EXPORTED_SYMBOLS = (
    "attn_fp8_scale_offset", "attn_fp8_scale_bytes", "attn_fp8_quantize", "attn_fp8_quantize_fused", "attn_fp8_prepare_bf16", "attn_fp8_fwd", "attn_fp8_bwd_delta",
    "attn_fp8_bwd", "attn_fp8_bwd_dq", "attn_fp8_bwd_dq_postcast", "attn_fp8_bwd_dkdv", "attn_fp8_fwd_noalloc",
    "attn_fp8_quantize_batch", "attn_fp8_workspace_bytes", "attn_fp8_workspace_init", "attn_fp8_read_status", "attn_fp8_last_error", "attn_fp8_selftest_timeout",
    "attn_fp8_measure_mma_peak", "attn_fp8_bwd_dq_rowprobe",
    "attn_fp8_measure_dq_reduction",
)


class AttnFp8Error(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class _Params(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("seqlen", ctypes.c_int32), ("heads_q", ctypes.c_int32),
                ("heads_kv", ctypes.c_int32), ("head_dim_qk", ctypes.c_int32), ("head_dim_v", ctypes.c_int32),
                ("causal", ctypes.c_int32), ("softmax_scale", ctypes.c_float), ("precision", ctypes.c_int32),
                ("delta_mode", ctypes.c_int32), ("seqlen_k", ctypes.c_int32), ("q_start", ctypes.c_int32),
                ("keys_valid", ctypes.c_int32)]


class _QTensor(ctypes.Structure):
    _fields_ = [("row_codes", ctypes.c_void_p), ("row_scales", ctypes.c_void_p),
                ("col_codes", ctypes.c_void_p), ("col_scales", ctypes.c_void_p)]


_vp, _i32, _sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
_lib.attn_fp8_scale_offset.restype = _sz
_lib.attn_fp8_scale_offset.argtypes = [ctypes.c_int64] * 3
_lib.attn_fp8_scale_bytes.restype = _sz
_lib.attn_fp8_scale_bytes.argtypes = [ctypes.c_int64] * 4
_lib.attn_fp8_quantize.restype = _i32
_lib.attn_fp8_quantize.argtypes = [_vp, _i32, _i32, _i32, _i32, _i32, _QTensor, _vp]
_lib.attn_fp8_prepare_bf16.restype = _i32
_lib.attn_fp8_prepare_bf16.argtypes = [_vp, _i32, _i32, _i32, _i32, _i32, _QTensor, _vp]
_lib.attn_fp8_fwd.restype = _i32
_lib.attn_fp8_fwd.argtypes = [ctypes.POINTER(_Params), _QTensor, _QTensor, _QTensor, _vp, _vp, _vp, _sz, _vp]
_lib.attn_fp8_bwd_delta.restype = _i32
_lib.attn_fp8_bwd_delta.argtypes = [ctypes.POINTER(_Params), _QTensor, _QTensor, _QTensor, _QTensor, _vp, _vp, _vp,
                                    _vp, _vp, _sz, _vp]
_lib.attn_fp8_bwd.restype = _i32
_lib.attn_fp8_bwd.argtypes = [ctypes.POINTER(_Params), _QTensor, _QTensor, _QTensor, _QTensor, _vp, _vp, _vp, _vp,
                              _vp, _vp, _vp, _vp, _sz, _vp]
_lib.attn_fp8_bwd_dq.restype = _i32
_lib.attn_fp8_bwd_dq.argtypes = [ctypes.POINTER(_Params), _QTensor, _QTensor, _QTensor, _QTensor, _vp, _vp, _vp, _vp,
                                 _vp, _vp, _sz, _vp]
_lib.attn_fp8_bwd_dkdv.restype = _i32
_lib.attn_fp8_bwd_dkdv.argtypes = [ctypes.POINTER(_Params), _QTensor, _QTensor, _QTensor, _QTensor, _vp, _vp, _vp,
                                   _vp, _vp, _sz, _vp]
_lib.attn_fp8_workspace_bytes.restype = _sz
_lib.attn_fp8_workspace_bytes.argtypes = [ctypes.POINTER(_Params), _i32]
_lib.attn_fp8_read_status.restype = _i32
_lib.attn_fp8_read_status.argtypes = [_vp, _vp]
_lib.attn_fp8_last_error.restype = ctypes.c_char_p
_lib.attn_fp8_last_error.argtypes = []


def attn_fp8_last_error() -> str:
    return _lib.attn_fp8_last_error().decode()


def _check(status):
    if status != ATTN_OK:
        raise AttnFp8Error(status, attn_fp8_last_error())


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


@dataclass
class AttnParams:
    batch: int
    seqlen: int
    heads_q: int
    heads_kv: int
    head_dim_qk: int
    head_dim_v: int
    causal: bool
    softmax_scale: float
    precision: int = ATTN_PREC_MXFP8
    delta_mode: int = ATTN_DELTA_MATCHED
    seqlen_k: int = 0            # keys; 0 = seqlen (square problem)
    q_start: int = 0             # position of query row 0 in the key sequence (a shard of the queries)
    keys_valid: int = 0          # real keys among the allocated ones (zero-padded ragged sequence); 0 = all

    @property
    def keys(self) -> int:
        return self.seqlen_k or self.seqlen

    def c_struct(self) -> _Params:
        return _Params(self.batch, self.seqlen, self.heads_q, self.heads_kv, self.head_dim_qk, self.head_dim_v,
                       int(self.causal), float(self.softmax_scale), self.precision, self.delta_mode, self.seqlen_k,
                       self.q_start, self.keys_valid)


@dataclass
class QTensor:
    """Device buffers of one quantised tensor [B, H, N, d] (see attn_qtensor_t)."""
    shape: tuple
    row_codes: Optional[torch.Tensor] = None
    row_scales: Optional[torch.Tensor] = None
    col_codes: Optional[torch.Tensor] = None
    col_scales: Optional[torch.Tensor] = None

    def c_struct(self) -> _QTensor:
        return _QTensor(*(None if t is None else t.data_ptr()
                          for t in (self.row_codes, self.row_scales, self.col_codes, self.col_scales)))


def protect_dp_operand(qt: QTensor, src_bf16: torch.Tensor) -> QTensor:
    """Operand of the protected-dP precision: ``qt`` with its row copy replaced by the BF16 tensor
    itself (dO or V); the column copy stays FP8."""
    if src_bf16.dtype != torch.bfloat16 or not src_bf16.is_contiguous() or tuple(src_bf16.shape) != tuple(qt.shape):
        raise ValueError("src_bf16 must be a contiguous bfloat16 tensor of the operand's shape")
    return QTensor(shape=qt.shape, row_codes=src_bf16, row_scales=None, col_codes=qt.col_codes, col_scales=qt.col_scales)


def pad_tokens(x: torch.Tensor, multiple: int = 128) -> torch.Tensor:
    """``x`` [B, H, N, d] with zero rows appended up to the next multiple of ``multiple`` tokens (the form in
    which a ragged sequence is handed to the library; see attn_params_t.keys_valid)."""
    n = x.shape[2]
    pad = (-n) % multiple
    if pad == 0:
        return x.contiguous()
    out = torch.zeros((x.shape[0], x.shape[1], n + pad, x.shape[3]), dtype=x.dtype, device=x.device)
    out[:, :, :n] = x
    return out


def attn_fp8_scale_offset(row: int, block: int, n_blocks: int) -> int:
    return int(_lib.attn_fp8_scale_offset(row, block, n_blocks))


def attn_fp8_scale_bytes(B: int, H: int, rows: int, cols: int) -> int:
    return int(_lib.attn_fp8_scale_bytes(B, H, rows, cols))


def unpack_scales(scales: torch.Tensor, B: int, H: int, rows: int, cols: int) -> torch.Tensor:
    """Reorders a tiled scale tensor into plain [B, H, rows, cols/32] (a pure index permutation,
    the inverse of the offset rule documented for attn_qtensor_t)."""
    nb = cols // 32
    r = np.arange(rows)[:, None]
    k = np.arange(nb)[None, :]
    off = ((r // 128) * ((nb + 3) // 4) + k // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + (k % 4)
    idx = torch.from_numpy(off.reshape(-1)).to(scales.device)
    slab = scales.reshape(B * H, -1)
    return slab[:, idx].reshape(B, H, rows, nb)


def attn_fp8_quantize(src: torch.Tensor, want_row: bool = True, want_col: bool = True, stream=None,
                      out: Optional[QTensor] = None) -> QTensor:
    """Quantise ``src`` [B, H, N, d] (BF16 or FP32, CUDA, contiguous) into the requested orientations.
    ``out`` reuses the buffers of an earlier call of the same shape (its non-None orientations are written)."""
    if not src.is_cuda or not src.is_contiguous() or src.dim() != 4:
        raise ValueError("src must be a contiguous CUDA tensor [B, H, N, d]")
    if src.dtype == torch.bfloat16:
        dt = ATTN_SRC_BF16
    elif src.dtype == torch.float32:
        dt = ATTN_SRC_FP32
    else:
        raise ValueError("src must be bfloat16 or float32")
    B, H, N, d = src.shape
    if out is None:
        out = QTensor(shape=(B, H, N, d))
        u8 = dict(dtype=torch.uint8, device=src.device)
        if want_row:
            out.row_codes = torch.empty((B, H, N, d), **u8)
            out.row_scales = torch.empty(attn_fp8_scale_bytes(B, H, N, d), **u8)
        if want_col:
            out.col_codes = torch.empty((B, H, d, N), **u8)
            out.col_scales = torch.empty(attn_fp8_scale_bytes(B, H, d, N), **u8)
    elif tuple(out.shape) != (B, H, N, d):
        raise ValueError("out was allocated for another shape")
    _check(_lib.attn_fp8_quantize(_ptr(src), dt, B, H, N, d, out.c_struct(), _stream(stream)))
    return out


class _QuantizeJob(ctypes.Structure):
    _fields_ = [("src", _vp), ("src_dtype", _i32), ("B", _i32), ("H", _i32), ("N", _i32), ("d", _i32),
                ("out", _QTensor)]


ATTN_QUANTIZE_MAX_JOBS = 8
ATTN_STATUS_WORKSPACE_BYTES = 256
_lib.attn_fp8_quantize_batch.restype = _i32
_lib.attn_fp8_quantize_batch.argtypes = [ctypes.POINTER(_QuantizeJob), _i32, _vp, _sz, _vp]


def attn_fp8_quantize_batch(srcs, outs=None, want=None, workspace=None, stream=None):
    """attn_fp8_quantize of several tensors (each [B, H, N, d], one dtype) in one launch.
    ``outs``: QTensors of earlier calls to reuse; ``want``: per tensor (want_row, want_col) when
    ``outs`` is None.  Returns (list of QTensor, workspace)."""
    srcs = list(srcs)
    if outs is None:
        want = want or [(True, True)] * len(srcs)
        outs = []
        for x, (wr, wc) in zip(srcs, want):
            B, H, N, d = x.shape
            q = QTensor(shape=(B, H, N, d))
            u8 = dict(dtype=torch.uint8, device=x.device)
            if wr:
                q.row_codes = torch.empty((B, H, N, d), **u8)
                q.row_scales = torch.empty(attn_fp8_scale_bytes(B, H, N, d), **u8)
            if wc:
                q.col_codes = torch.empty((B, H, d, N), **u8)
                q.col_scales = torch.empty(attn_fp8_scale_bytes(B, H, d, N), **u8)
            outs.append(q)
    jobs = (_QuantizeJob * len(srcs))()
    for j, (x, q) in enumerate(zip(srcs, outs)):
        if not x.is_cuda or not x.is_contiguous() or x.dim() != 4:
            raise ValueError("every source must be a contiguous CUDA tensor [B, H, N, d]")
        if x.dtype not in (torch.bfloat16, torch.float32):
            raise ValueError("sources must be bfloat16 or float32")
        if tuple(q.shape) != tuple(x.shape):
            raise ValueError("an output was allocated for another shape")
        B, H, N, d = x.shape
        jobs[j] = _QuantizeJob(_ptr(x), ATTN_SRC_BF16 if x.dtype == torch.bfloat16 else ATTN_SRC_FP32, B, H, N, d,
                               q.c_struct())
    if workspace is None:
        workspace = new_workspace(ATTN_STATUS_WORKSPACE_BYTES, srcs[0].device)
    _check(_lib.attn_fp8_quantize_batch(jobs, len(srcs), _ptr(workspace), workspace.numel(), _stream(stream)))
    return list(outs), workspace


_lib.attn_fp8_quantize_fused.restype = _i32
_lib.attn_fp8_quantize_fused.argtypes = [_vp, _i32, _i32, _i32, _i32, _i32, _vp, _vp, ctypes.c_float, _vp, _QTensor, _vp]


def attn_fp8_quantize_fused(src: torch.Tensor, rope_cos: Optional[torch.Tensor] = None,
                            rope_sin: Optional[torch.Tensor] = None, scale: float = 1.0, center: bool = False,
                            want_row: bool = True, want_col: bool = True, stream=None):
    """Quantiser with the producer fused in front: optional rotary embedding (FP32 tables [N, d/2]),
    optional key centering, optional FP32 scale.  Returns (QTensor, mean [B, H, d] fp32 or None)."""
    if not src.is_cuda or not src.is_contiguous() or src.dim() != 4:
        raise ValueError("src must be a contiguous CUDA tensor [B, H, N, d]")
    if src.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("src must be bfloat16 or float32")
    dt = ATTN_SRC_BF16 if src.dtype == torch.bfloat16 else ATTN_SRC_FP32
    B, H, N, d = src.shape
    out = QTensor(shape=(B, H, N, d))
    u8 = dict(dtype=torch.uint8, device=src.device)
    if want_row:
        out.row_codes = torch.empty((B, H, N, d), **u8)
        out.row_scales = torch.empty(attn_fp8_scale_bytes(B, H, N, d), **u8)
    if want_col:
        out.col_codes = torch.empty((B, H, d, N), **u8)
        out.col_scales = torch.empty(attn_fp8_scale_bytes(B, H, d, N), **u8)
    mean = torch.empty((B, H, d), dtype=torch.float32, device=src.device) if center else None
    for t in (rope_cos, rope_sin):
        if t is not None and (t.dtype != torch.float32 or not t.is_contiguous() or tuple(t.shape) != (N, d // 2)):
            raise ValueError("rotary tables must be contiguous float32 [N, d/2]")
    _check(_lib.attn_fp8_quantize_fused(_ptr(src), dt, B, H, N, d, _ptr(rope_cos), _ptr(rope_sin), float(scale),
                                        _ptr(mean), out.c_struct(), _stream(stream)))
    return out, mean


def attn_fp8_prepare_bf16(src: torch.Tensor, want_row: bool = True, want_col: bool = True, stream=None,
                          out: Optional[QTensor] = None) -> QTensor:
    """BF16-mode operands of ``src`` [B, H, N, d]: ``row_codes`` = BF16 [B, H, N, d] (``src`` itself when
    it already is BF16), ``col_codes`` = BF16 [B, H, d, N]; no scales.  ``out`` reuses the buffers of an
    earlier call of the same shape."""
    if not src.is_cuda or not src.is_contiguous() or src.dim() != 4:
        raise ValueError("src must be a contiguous CUDA tensor [B, H, N, d]")
    if src.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("src must be bfloat16 or float32")
    dt = ATTN_SRC_BF16 if src.dtype == torch.bfloat16 else ATTN_SRC_FP32
    B, H, N, d = src.shape
    alias_row = src.dtype == torch.bfloat16      # the row operand is the source itself
    if out is None:
        out = QTensor(shape=(B, H, N, d))
        bf = dict(dtype=torch.bfloat16, device=src.device)
        if want_row and not alias_row:
            out.row_codes = torch.empty((B, H, N, d), **bf)
        if want_col:
            out.col_codes = torch.empty((B, H, d, N), **bf)
    elif tuple(out.shape) != (B, H, N, d):
        raise ValueError("out was allocated for another shape")
    row_buf = None if alias_row else out.row_codes
    if row_buf is not None or out.col_codes is not None:
        c = _QTensor(None if row_buf is None else row_buf.data_ptr(), None,
                     None if out.col_codes is None else out.col_codes.data_ptr(), None)
        _check(_lib.attn_fp8_prepare_bf16(_ptr(src), dt, B, H, N, d, c, _stream(stream)))
    if alias_row and (want_row or out.row_codes is not None):
        out.row_codes = src
    return out


def attn_fp8_workspace_bytes(params: AttnParams, which: int) -> int:
    c = params.c_struct()
    return int(_lib.attn_fp8_workspace_bytes(ctypes.byref(c), which))


_lib.attn_fp8_workspace_init.restype = _i32
_lib.attn_fp8_workspace_init.argtypes = [_vp, _sz, _vp]


def attn_fp8_workspace_init(workspace: torch.Tensor, stream=None) -> torch.Tensor:
    """Clears the status header of a caller-made workspace (once, before its first use)."""
    _check(_lib.attn_fp8_workspace_init(_ptr(workspace), workspace.numel(), _stream(stream)))
    return workspace


def new_workspace(nbytes: int, device, stream=None) -> torch.Tensor:
    """A workspace of ``nbytes`` (at least the status header) with its status word cleared."""
    ws = torch.empty(max(int(nbytes), ATTN_STATUS_WORKSPACE_BYTES), dtype=torch.uint8, device=device)
    return attn_fp8_workspace_init(ws, stream)


def _workspace(params, which, workspace, device):
    if workspace is None:
        workspace = new_workspace(attn_fp8_workspace_bytes(params, which), device)
    return workspace


_lib.attn_fp8_selftest_timeout.restype = _i32
_lib.attn_fp8_selftest_timeout.argtypes = [_vp, _sz, _vp]


def attn_fp8_selftest_timeout(workspace: Optional[torch.Tensor], stream=None) -> None:
    """Enqueues the bounded-wait self-test: the next attn_fp8_read_status(workspace) raises ATTN_ERR_TIMEOUT.
    ``workspace=None`` targets the library's built-in scratch array on the current device."""
    _check(_lib.attn_fp8_selftest_timeout(_ptr(workspace), 0 if workspace is None else workspace.numel(), _stream(stream)))


def attn_fp8_read_status(workspace: Optional[torch.Tensor], stream=None) -> None:
    """Synchronises ``stream`` and raises if a kernel of the last call reported a timeout.
    ``workspace=None`` reads the built-in scratch array (attn_fp8_quantize, attn_fp8_fwd_noalloc)."""
    _check(_lib.attn_fp8_read_status(_ptr(workspace), _stream(stream)))


_lib.attn_fp8_measure_mma_peak.restype = _i32
_lib.attn_fp8_measure_mma_peak.argtypes = [ctypes.POINTER(ctypes.c_double), _vp, _sz, _vp]


_lib.attn_fp8_measure_dq_reduction.restype = _i32
_lib.attn_fp8_measure_dq_reduction.argtypes = [ctypes.POINTER(_Params), _vp, _sz, ctypes.POINTER(ctypes.c_double),
                                               ctypes.POINTER(ctypes.c_double), _vp]


def attn_fp8_measure_dq_reduction(params: "AttnParams", dq_f32: torch.Tensor, stream=None):
    """(milliseconds, bytes added) of the FP32 dQ reduction a merged key-major gradient pass would issue
    for ``params``; ``dq_f32`` is an FP32 [B, Hq, N, dqk] device tensor (overwritten).  Synchronises."""
    ms, nbytes = ctypes.c_double(0.0), ctypes.c_double(0.0)
    c = params.c_struct()
    _check(_lib.attn_fp8_measure_dq_reduction(ctypes.byref(c), _ptr(dq_f32), dq_f32.numel() * dq_f32.element_size(),
                                              ctypes.byref(ms), ctypes.byref(nbytes), _stream(stream)))
    return ms.value, nbytes.value


def attn_fp8_measure_mma_peak(workspace: torch.Tensor, stream=None) -> float:
    """TFLOP/s of the bare block-scaled FP8 tensor-core instruction on this device (synchronises)."""
    out = ctypes.c_double(0.0)
    _check(_lib.attn_fp8_measure_mma_peak(ctypes.byref(out), _ptr(workspace), workspace.numel(), _stream(stream)))
    return out.value


def attn_fp8_fwd(params: AttnParams, q: QTensor, k: QTensor, v: QTensor, o=None, lse=None, workspace=None,
                 stream=None):
    """Returns (O [B,Hq,N,dv] bf16, LSE [B,Hq,N] fp32, workspace)."""
    dev = q.row_codes.device
    if o is None:
        o = torch.empty((params.batch, params.heads_q, params.seqlen, params.head_dim_v), dtype=torch.bfloat16, device=dev)
    if lse is None:
        lse = torch.empty((params.batch, params.heads_q, params.seqlen), dtype=torch.float32, device=dev)
    workspace = _workspace(params, ATTN_WS_FWD, workspace, dev)
    c = params.c_struct()
    _check(_lib.attn_fp8_fwd(ctypes.byref(c), q.c_struct(), k.c_struct(), v.c_struct(), _ptr(o), _ptr(lse),
                             _ptr(workspace), workspace.numel(), _stream(stream)))
    return o, lse, workspace


def attn_fp8_bwd_delta(params: AttnParams, q: QTensor, k: QTensor, v: QTensor, dO: QTensor, lse, dO_bf16=None,
                       o_bf16=None, delta=None, workspace=None, stream=None):
    """Returns (delta [B,Hq,N] fp32, workspace).  ``params.delta_mode`` selects matched / stale."""
    dev = lse.device
    if delta is None:
        delta = torch.empty((params.batch, params.heads_q, params.seqlen), dtype=torch.float32, device=dev)
    workspace = _workspace(params, ATTN_WS_BWD_DELTA, workspace, dev)
    c = params.c_struct()
    _check(_lib.attn_fp8_bwd_delta(ctypes.byref(c), q.c_struct(), k.c_struct(), v.c_struct(), dO.c_struct(),
                                   _ptr(dO_bf16), _ptr(o_bf16), _ptr(lse), _ptr(delta), _ptr(workspace),
                                   workspace.numel(), _stream(stream)))
    return delta, workspace


def attn_fp8_bwd(params: AttnParams, q: QTensor, k: QTensor, v: QTensor, dO: QTensor, lse, delta, dq=None, dk=None,
                 dv=None, diagnostics: bool = False, workspace=None, stream=None):
    """Returns (dQ, dK, dV, rowsum_dS or None, rowsum_abs_dS or None, workspace)."""
    dev = lse.device
    bf = dict(dtype=torch.bfloat16, device=dev)
    B, N = params.batch, params.seqlen
    if dq is None:
        dq = torch.empty((B, params.heads_q, N, params.head_dim_qk), **bf)
    if dk is None:
        dk = torch.empty((B, params.heads_kv, params.keys, params.head_dim_qk), **bf)
    if dv is None:
        dv = torch.empty((B, params.heads_kv, params.keys, params.head_dim_v), **bf)
    rs = ra = None
    if diagnostics:
        rs = torch.empty((B, params.heads_q, N), dtype=torch.float32, device=dev)
        ra = torch.empty((B, params.heads_q, N), dtype=torch.float32, device=dev)
    workspace = _workspace(params, ATTN_WS_BWD, workspace, dev)
    c = params.c_struct()
    _check(_lib.attn_fp8_bwd(ctypes.byref(c), q.c_struct(), k.c_struct(), v.c_struct(), dO.c_struct(), _ptr(lse),
                             _ptr(delta), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(rs), _ptr(ra), _ptr(workspace),
                             workspace.numel(), _stream(stream)))
    return dq, dk, dv, rs, ra, workspace


def attn_fp8_bwd_dq(params: AttnParams, q: QTensor, k: QTensor, v: QTensor, dO: QTensor, lse, delta, dq=None,
                    diagnostics: bool = False, workspace=None, stream=None):
    """Query-major half of the gradient pass.  Returns (dQ, rowsum_dS or None, rowsum_abs_dS or None, workspace)."""
    dev = lse.device
    B, N = params.batch, params.seqlen
    if dq is None:
        dq = torch.empty((B, params.heads_q, N, params.head_dim_qk), dtype=torch.bfloat16, device=dev)
    rs = ra = None
    if diagnostics:
        rs = torch.empty((B, params.heads_q, N), dtype=torch.float32, device=dev)
        ra = torch.empty((B, params.heads_q, N), dtype=torch.float32, device=dev)
    workspace = _workspace(params, ATTN_WS_BWD, workspace, dev)
    c = params.c_struct()
    _check(_lib.attn_fp8_bwd_dq(ctypes.byref(c), q.c_struct(), k.c_struct(), v.c_struct(), dO.c_struct(), _ptr(lse),
                                _ptr(delta), _ptr(dq), _ptr(rs), _ptr(ra), _ptr(workspace), workspace.numel(),
                                _stream(stream)))
    return dq, rs, ra, workspace


_lib.attn_fp8_bwd_dq_postcast.restype = _i32
_lib.attn_fp8_bwd_dq_postcast.argtypes = [ctypes.POINTER(_Params), _QTensor, _QTensor, _QTensor, _QTensor, _vp, _vp, _vp,
                                          _vp, _vp, _vp, _vp, _vp, _sz, _vp]


def attn_fp8_bwd_dq_postcast(params: AttnParams, q: QTensor, k: QTensor, v: QTensor, dO: QTensor, lse, delta, dq=None,
                             workspace=None, stream=None):
    """dQ plus the pre- and post-cast row statistics of dS.  Returns
    (dQ, rowsum_dS, rowsum_abs_dS, rowsum_dS_cast, rowsum_abs_dS_cast, workspace)."""
    dev = lse.device
    B, N = params.batch, params.seqlen
    if dq is None:
        dq = torch.empty((B, params.heads_q, N, params.head_dim_qk), dtype=torch.bfloat16, device=dev)
    stats = [torch.empty((B, params.heads_q, N), dtype=torch.float32, device=dev) for _ in range(4)]
    workspace = _workspace(params, ATTN_WS_BWD, workspace, dev)
    c = params.c_struct()
    _check(_lib.attn_fp8_bwd_dq_postcast(ctypes.byref(c), q.c_struct(), k.c_struct(), v.c_struct(), dO.c_struct(),
                                         _ptr(lse), _ptr(delta), _ptr(dq), *(_ptr(t) for t in stats), _ptr(workspace),
                                         workspace.numel(), _stream(stream)))
    return (dq, *stats, workspace)


_lib.attn_fp8_bwd_dq_rowprobe.restype = _i32
_lib.attn_fp8_bwd_dq_rowprobe.argtypes = [ctypes.POINTER(_Params), _QTensor, _QTensor, _QTensor, _QTensor, _vp, _vp, _vp,
                                          _vp, _vp, _vp, _vp, _sz, _vp]


def attn_fp8_bwd_dq_rowprobe(params: AttnParams, q: QTensor, k: QTensor, v: QTensor, dO: QTensor, lse, delta, dq=None,
                             workspace=None, stream=None):
    """dQ plus what the per-row acceptance of the zero-row-sum invariant needs.  Returns
    (dQ, rowsum_dS, rowsum_abs_dS, rowsum_P_abs_dP, workspace)."""
    dev = lse.device
    B, N = params.batch, params.seqlen
    if dq is None:
        dq = torch.empty((B, params.heads_q, N, params.head_dim_qk), dtype=torch.bfloat16, device=dev)
    stats = [torch.empty((B, params.heads_q, N), dtype=torch.float32, device=dev) for _ in range(3)]
    workspace = _workspace(params, ATTN_WS_BWD, workspace, dev)
    c = params.c_struct()
    _check(_lib.attn_fp8_bwd_dq_rowprobe(ctypes.byref(c), q.c_struct(), k.c_struct(), v.c_struct(), dO.c_struct(),
                                         _ptr(lse), _ptr(delta), _ptr(dq), *(_ptr(t) for t in stats), _ptr(workspace),
                                         workspace.numel(), _stream(stream)))
    return (dq, *stats, workspace)


def attn_fp8_bwd_dkdv(params: AttnParams, q: QTensor, k: QTensor, v: QTensor, dO: QTensor, lse, delta, dk=None,
                      dv=None, workspace=None, stream=None):
    """Key-major half of the gradient pass.  Returns (dK, dV, workspace)."""
    dev = lse.device
    bf = dict(dtype=torch.bfloat16, device=dev)
    B, N = params.batch, params.seqlen
    if dk is None:
        dk = torch.empty((B, params.heads_kv, params.keys, params.head_dim_qk), **bf)
    if dv is None:
        dv = torch.empty((B, params.heads_kv, params.keys, params.head_dim_v), **bf)
    workspace = _workspace(params, ATTN_WS_BWD, workspace, dev)
    c = params.c_struct()
    _check(_lib.attn_fp8_bwd_dkdv(ctypes.byref(c), q.c_struct(), k.c_struct(), v.c_struct(), dO.c_struct(),
                                  _ptr(lse), _ptr(delta), _ptr(dk), _ptr(dv), _ptr(workspace), workspace.numel(),
                                  _stream(stream)))
    return dk, dv, workspace


_lib.attn_fp8_fwd_noalloc.restype = _i32
_lib.attn_fp8_fwd_noalloc.argtypes = [ctypes.POINTER(_Params), _QTensor, _QTensor, _QTensor, _vp, _vp, _vp]


def attn_fp8_fwd_noalloc(params: AttnParams, q: QTensor, k: QTensor, v: QTensor, o: torch.Tensor, lse: torch.Tensor,
                         stream=None) -> None:
    """Forward for call sites that may not allocate: the caller passes the outputs ``o`` and ``lse``
    (already allocated, like the inputs) and no workspace; the library uses its built-in 4096-byte
    scratch array.  This wrapper allocates nothing either.  Calls that overlap on the GPU share that
    array and race; see the header for the remaining rules."""
    c = params.c_struct()
    _check(_lib.attn_fp8_fwd_noalloc(ctypes.byref(c), q.c_struct(), k.c_struct(), v.c_struct(), _ptr(o), _ptr(lse),
                                     _stream(stream)))
