"""Helpers shared by the GPU parity tests: moving seeded workloads to either side and error metrics.

No arithmetic of the layer lives here: the CUDA side is reached only through the C-ABI binding and the
reference side only through the oracle package.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle.adapters import bits_or_f32, f32, oracle_inputs, shape_of  # noqa: F401


def clear_gap_tokens(logits: np.ndarray, k: int, gap: float = 1e-3) -> np.ndarray:
    """Tokens whose K+1 largest logits are pairwise separated by more than `gap`: their top-K list (members and
    order) cannot depend on rounding below that size."""
    srt = -np.sort(-logits.astype(np.float64), axis=1)
    top = srt[:, :min(k + 1, logits.shape[1])]
    return np.all(top[:, :-1] - top[:, 1:] > gap, axis=1) if top.shape[1] > 1 else np.ones(len(logits), bool)


def rel_err_per_token(y: np.ndarray, ref: np.ndarray) -> float:
    """max over tokens of |y_t - ref_t|_inf / max(|ref_t|_inf, 1e-6 |ref|_inf)."""
    y, ref = y.astype(np.float64), ref.astype(np.float64)
    if ref.size == 0:
        return 0.0
    row = np.abs(ref).max(axis=1)
    floor = 1e-6 * max(float(np.abs(ref).max()), 1e-30)
    return float((np.abs(y - ref).max(axis=1) / np.maximum(row, floor)).max())


def max_abs(y: np.ndarray, ref: np.ndarray) -> float:
    return float(np.abs(y.astype(np.float64) - ref.astype(np.float64)).max()) if ref.size else 0.0


def sample_tokens(idx: np.ndarray, n_experts: int, n: int, seed: int = 0) -> np.ndarray:
    """A token sample that hits every expert that is hit at all, plus random tokens up to n."""
    rng = np.random.default_rng(seed)
    chosen = []
    for e in range(n_experts):
        hit = np.nonzero((idx == e).any(axis=1))[0]
        if len(hit):
            chosen.extend(rng.choice(hit, size=min(2, len(hit)), replace=False).tolist())
    rest = rng.choice(idx.shape[0], size=min(n, idx.shape[0]), replace=False).tolist()
    out = list(dict.fromkeys(chosen + rest))[:max(n, len(chosen))]
    return np.array(sorted(out), np.int32)
