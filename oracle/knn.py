"""CPU oracle for the k-NN (inner-product) variant.  TEST INFRASTRUCTURE ONLY.

Paper Sec. 3.1 "Problem Definition" (Eq. 2) with the scoring function of the
retrieval workload (Sec. 4.1 "Large-Scale Retrieval Benchmark"): every query of a
batch is scored against every vector of the corpus,

    f(q, x) = q . x                                   (inner product, D = 768)
    TopK(q) = arg-top-k over the whole corpus of f(q, x)   (no causal mask)

and the k best are returned in (score descending, index ascending) order.  The
definition written out in fp64 with numpy: decode the bf16 storage, one matmul,
one sort per row.  It shares no code with the CUDA library.

Parity pins (tests/test_oracle_pins.py): exact-rational brute force on tiny
inputs; agreement with the indexer oracle for H = 1, w = 1 on inputs whose dot
products are all non-negative (there the ReLU of Eq. 1 is the identity);
invariance of the selected set under a common positive scaling of the queries.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np

from .indexer_topk import decode_bf16, select_topk


def knn_scores(q_bits: np.ndarray, x_bits: np.ndarray, rows: Optional[Sequence[int]] = None) -> np.ndarray:
    """fp64 inner products of the bf16-coded queries (rows) with every bf16-coded corpus vector."""
    q = decode_bf16(q_bits).astype(np.float64)
    x = decode_bf16(x_bits).astype(np.float64)
    if rows is not None:
        q = q[np.asarray(rows, dtype=np.int64)]
    return q @ x.T


def knn_topk(q_bits: np.ndarray, x_bits: np.ndarray, topk: int, rows: Optional[Sequence[int]] = None):
    """(idx [R, topk] int64, score [R, topk] fp64, rms [R], full scores [R, N])."""
    s = knn_scores(q_bits, x_bits, rows)
    idx = np.empty((s.shape[0], topk), dtype=np.int64)
    val = np.empty((s.shape[0], topk), dtype=np.float64)
    for r in range(s.shape[0]):
        idx[r], val[r] = select_topk(s[r], topk)
    rms = np.sqrt(np.mean(s * s, axis=1))
    return idx, val, rms, s
