"""Helpers shared by the GPU parity tests (no method arithmetic)."""
import numpy as np
import torch


def to_np(t: torch.Tensor) -> np.ndarray:
    """Exact float64 copy of a (bf16 / fp32) tensor on the host."""
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def rel_fro(got, want) -> float:
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


def worst_row_error(got, want) -> float:
    """Largest relative error of a single row (a vector along the last axis) among the rows whose
    reference norm is at least the median row norm of the tensor: the companion of a whole-tensor
    Frobenius bound, which one badly wrong row in a few thousand would pass."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = np.linalg.norm(got - want, axis=-1)
    ref = np.linalg.norm(want, axis=-1)
    sel = ref >= np.median(ref)
    if not sel.any() or ref[sel].max() == 0.0:
        return 0.0
    sel &= ref > 0
    return float((err[sel] / ref[sel]).max())
