"""Acceptance rules that compare a candidate result with the oracle.  TEST INFRASTRUCTURE ONLY.

Floating-point scores from a GPU differ from fp64 by rounding, so exact index
equality cannot be demanded where two keys' scores straddle the k-th value by
less than the rounding error.  The rules (tolerance tol_t = 1e-3 * RMS of row
t's visible scores, RMS taken from the oracle):

  scores  |I_gpu - I_oracle| <= tol_t for every visible pair that is checked;
  indices the selected sets are equal, except for keys in the symmetric
          difference whose oracle scores all lie within tol_t of the oracle's
          k-th score (a legal swap at the boundary);
  order   a candidate's output must be sorted by (score descending, index
          ascending) in its own scores, with distinct in-range indices.
"""
from __future__ import annotations

import numpy as np

REL_TOL = 1e-3


def check_row_indices(cand_idx: np.ndarray, oracle_idx: np.ndarray, oracle_full: np.ndarray,
                      kth: float, tol: float) -> tuple[bool, str]:
    """Index rule for one row.  `oracle_full` holds the oracle's fp64 score of every visible key."""
    n_vis = oracle_full.shape[0]
    a = cand_idx[cand_idx >= 0]
    b = oracle_idx[oracle_idx >= 0]
    if a.shape[0] != b.shape[0]:
        return False, f"selected {a.shape[0]} keys, oracle selected {b.shape[0]}"
    if np.unique(a).shape[0] != a.shape[0]:
        return False, "duplicate indices"
    if a.size and (a.min() < 0 or a.max() >= n_vis):
        return False, "index outside the causal bound"
    if np.any(cand_idx[a.shape[0]:] != -1):
        return False, "padding is not -1"
    extra = np.setdiff1d(a, b)
    missing = np.setdiff1d(b, a)
    for name, keys in (("extra", extra), ("missing", missing)):
        if keys.size:
            dev = np.abs(oracle_full[keys] - kth).max()
            if dev > tol:
                return False, f"{name} keys {keys[:4]} differ from the k-th score by {dev:.3e} > tol {tol:.3e}"
    return True, f"{extra.size} boundary swaps"


def check_row_scores(cand_score_row: np.ndarray, oracle_full: np.ndarray, tol: float) -> tuple[bool, float]:
    """Score rule for one dense row: visible keys within tol, masked keys are -inf."""
    n_vis = oracle_full.shape[0]
    err = np.abs(cand_score_row[:n_vis].astype(np.float64) - oracle_full).max() if n_vis else 0.0
    masked_ok = bool(np.all(np.isneginf(cand_score_row[n_vis:])))
    return bool(err <= tol) and masked_ok, float(err)


def canonical_topk_of(scores_row: np.ndarray, n_vis: int, topk: int) -> tuple[np.ndarray, np.ndarray]:
    """Independent selector used to verify that a candidate's indices are exactly the top-k of
    its OWN dumped scores: stable argsort of the visible prefix (ties keep the lower index)."""
    s = np.asarray(scores_row[:n_vis])
    order = np.argsort(-s.astype(np.float64), kind="stable")[:topk]
    idx = np.full(topk, -1, dtype=np.int64)
    val = np.full(topk, -np.inf, dtype=np.float32)
    idx[: order.shape[0]] = order
    val[: order.shape[0]] = s[order]
    return idx, val
