"""FP8 Delta-Matching attention for NVIDIA B200 (sm_100a).

The compute path lives in a C-ABI shared library built from ``csrc/``;
``binding`` wraps it with the same entry-point names (argument marshalling
only) and raises at import when the library has not been built.
``workloads`` holds the seeded synthetic input generators and imports nothing
from the compute path.
"""
_EXPORTS = (
    "attn_fp8_quantize", "attn_fp8_fwd", "attn_fp8_bwd_delta", "attn_fp8_bwd", "attn_fp8_bwd_dq", "attn_fp8_bwd_dkdv", "attn_fp8_fwd_noalloc",
    "attn_fp8_workspace_bytes", "attn_fp8_last_error", "QTensor", "AttnParams",
)


def __getattr__(name):
    if name in _EXPORTS:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
