"""Shared test helpers: bf16 <-> numpy conversions and cache (de)paging for the oracle side."""
import numpy as np
import torch


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 torch tensor -> uint16 numpy bit patterns (host)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def from_f64(a: np.ndarray) -> torch.Tensor:
    """float64 values -> bf16 tensor (round to nearest even, via fp32)."""
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def row_rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max over rows of  max_c |got - ref| / max_c |ref|  (rows = all leading dims)."""
    g = got.reshape(-1, got.shape[-1])
    r = ref.reshape(-1, ref.shape[-1])
    num = np.abs(g - r).max(axis=1)
    den = np.abs(r).max(axis=1)
    return float((num / np.maximum(den, 1e-300)).max())
