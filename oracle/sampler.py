"""CPU oracle for the previous-chunk sampler.  TEST INFRASTRUCTURE ONLY.

Paper Sec. 3.2 "Sampling": for sparse attention the sample of the current chunk
is "the k' tokens (k' = 3k for DSA) that occur most frequently in the top-k
results of the previous chunk".  Written out, with the tie rule the paper leaves
open (reading: the lower position wins, as everywhere else in this build):

    count[p] = number of (row, slot) pairs of the previous chunk's top-k index
               matrix that hold position p          (entries < 0 are padding)
    result   = the k' positions with the largest (count, then smaller position),
               in that order; positions nobody selected (count 0) fill the tail
               in ascending order if fewer than k' distinct positions occur.

The definition is a histogram followed by a sort, and that is all this module
does (numpy bincount + lexsort).  It shares no code with the CUDA library and may
be imported only by tests, the smoke check and the benchmark's CPU leg.

Parity pins (tests/test_oracle_pins.py): a pure-Python Counter brute force on tiny
inputs, closed-form constructed inputs, and invariants (distinct positions,
counts non-increasing, permutation invariance in rows and slots).
"""
from __future__ import annotations

import numpy as np


def position_counts(idx: np.ndarray, N: int) -> np.ndarray:
    """count[p] over an index matrix (any shape); negative entries are padding and ignored."""
    flat = np.asarray(idx).reshape(-1).astype(np.int64)
    flat = flat[flat >= 0]
    if flat.size and flat.max() >= N:
        raise ValueError("index outside [0, N)")
    return np.bincount(flat, minlength=N).astype(np.int64)


def frequent_positions(idx: np.ndarray, N: int, n_out: int) -> tuple[np.ndarray, np.ndarray]:
    """(positions, counts) of the n_out most frequent positions, count descending, position ascending."""
    if not 0 < n_out <= N:
        raise ValueError("need 0 < n_out <= N")
    count = position_counts(idx, N)
    order = np.lexsort((np.arange(N, dtype=np.int64), -count))  # primary: -count, secondary: position
    pos = order[:n_out]
    return pos.astype(np.int64), count[pos]
