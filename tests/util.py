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
