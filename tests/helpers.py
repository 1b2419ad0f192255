"""Shared helpers for the parity tests (no method arithmetic lives here)."""
import numpy as np
import torch


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def bf16_round(a: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).float().numpy().astype(np.float64)


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max-abs-error / RMS(reference): the tolerance metric for bf16 outputs."""
    rms = float(np.sqrt(np.mean(ref * ref)))
    return float(np.abs(got - ref).max() / max(rms, 1e-30))


def bf16_bound(ref: np.ndarray, tol: float = 1e-2) -> float:
    """Tolerance for a bf16 output: the stated 1e-2, or - where merely rounding the exact
    result to bf16 already exceeds it on heavy-tailed entries - that rounding floor plus
    2e-3."""
    floor = rel_err(bf16_round(ref), ref)
    return max(tol, floor + 2e-3)
