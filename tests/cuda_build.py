"""Test-side names for the library's level builders, plus the error measures the parity tests use."""
import numpy as np
import torch

from paper_2207_02849_b200.problems import (  # noqa: F401
    correct_reweight_levels, dev, logreg_levels, quadratic_levels, reweight_levels, three_levels,
)


def _np(a):
    return a.detach().double().cpu().numpy() if isinstance(a, torch.Tensor) else np.asarray(a, np.float64)


def rel_l2(got, ref):
    got, ref = _np(got), _np(ref)
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))


def rel_max(got, ref):
    """Largest element error over the largest reference magnitude: catches one wrong component of a short
    vector that a whole-vector norm would let through."""
    got, ref = _np(got), _np(ref)
    return float(np.max(np.abs(got - ref)) / max(np.max(np.abs(ref)), 1e-300)) if ref.size else 0.0
