"""CPU oracle for the DSA indexer top-k.  TEST INFRASTRUCTURE ONLY.

This is the plain definition, written out in fp64 with numpy, of what the fused
GPU path must return.  It is slow on purpose, shares no code with the CUDA
library, and may be imported only by the tests, the smoke check and the
benchmark's CPU-baseline leg.  Nothing in the product path may call it.

What it computes (paper section and equation in brackets):

  index score  [Sec. 2 "Sparse Attention", Eq. 1]
      I[t, s] = sum_j  w[t, j] * ReLU( q[t, j] . k[s] )
  exact top-k  [Sec. 3.1 "Problem Definition", Eq. 2]
      TopK(t) = arg-top-k over the candidate keys s of I[t, s]

The fused method (sample, bin, online threshold, filtered write-back, tail
select; Sec. 3.2) is stated to preserve exact top-k correctness, so the oracle
is the definition itself, not the filter: score every visible key, sort, take k.

Readings where the paper is silent (all listed in the design notes too):
  * ReLU acts on the per-head dot product (Eq. 1; Eq. 3's print is garbled).
  * w may have either sign; any other scalar factor is pre-folded into w.
  * fp8 inputs are e4m3 codes times one fp32 scale per token; the key's scale
    multiplies the head sum (scale >= 0), the query's scale is pre-folded into w.
  * causal rule: the query at row t sits at position causal_offset + t and sees
    keys 0 .. causal_offset + t inclusive (clipped to N).
  * ties: the lower key index wins; output order is (score descending, index
    ascending); rows with fewer than k visible keys are padded with (-1, -inf).
  * -0.0 and +0.0 compare equal (a tie).

Parity pins (tests/test_oracle_pins.py): storage-format facts, a pure-Python
brute force with exact rationals on tiny inputs, constructed inputs whose score
order is known in closed form, and invariants / metamorphic relations.
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Sequence

import numpy as np

# ----------------------------------------------------------------------------
# storage-format decoding (exact in fp64)
# ----------------------------------------------------------------------------


def decode_bf16(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> fp64.  A bf16 is the upper half of an IEEE fp32."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def _e4m3_table() -> np.ndarray:
    """All 256 e4m3 ("fn" flavour) values: 1 sign, 4 exponent (bias 7), 3 mantissa bits.
    Exponent field 0 is subnormal (m/8 * 2^-6); there is no infinity; 0x7F / 0xFF are NaN."""
    tab = np.empty(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e = (code >> 3) & 0xF
        m = code & 0x7
        if e == 0xF and m == 0x7:
            val = np.nan
        elif e == 0:
            val = (m / 8.0) * 2.0 ** -6
        else:
            val = (1.0 + m / 8.0) * 2.0 ** (e - 7)
        tab[code] = sign * val
    return tab


_E4M3 = _e4m3_table()


def decode_e4m3(codes: np.ndarray) -> np.ndarray:
    return _E4M3[np.asarray(codes, dtype=np.uint8)]


def decode(arr: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return np.asarray(arr, dtype=np.float32).astype(np.float64)
    if dtype == "bf16":
        return decode_bf16(arr)
    if dtype == "e4m3":
        return decode_e4m3(arr)
    raise ValueError(f"unknown dtype {dtype!r}")


# ----------------------------------------------------------------------------
# scores (Eq. 1) and exact selection (Eq. 2)
# ----------------------------------------------------------------------------


def visible_keys(t: int, N: int, causal_offset: int) -> int:
    """Row t sees keys 0 .. causal_offset + t inclusive."""
    return int(min(N, max(0, causal_offset + t + 1)))


def score_row(q_t: np.ndarray, w_t: np.ndarray, k_vis: np.ndarray, k_scale_vis: Optional[np.ndarray]) -> np.ndarray:
    """Eq. 1 for one query against its visible keys, all in fp64.

    q_t [H, D], w_t [H], k_vis [n, D], k_scale_vis [n] or None -> I [n]."""
    dots = k_vis @ q_t.T  # [n, H]: q[t, j] . k[s]
    relu = np.maximum(dots, 0.0)
    score = relu @ w_t  # sum over heads of w[t, j] * ReLU(.)
    if k_scale_vis is not None:
        score = score * k_scale_vis
    return score


def select_topk(score: np.ndarray, topk: int) -> tuple[np.ndarray, np.ndarray]:
    """Eq. 2 by full sort: order keys by (score descending, index ascending), keep the first k.
    Short rows are padded with index -1 / score -inf."""
    n = score.shape[0]
    idx = np.arange(n, dtype=np.int64)
    order = np.lexsort((idx, -score))  # last key is primary; -(-0.0) == -(0.0) so signed zeros tie
    keep = order[:topk]
    out_idx = np.full(topk, -1, dtype=np.int64)
    out_score = np.full(topk, -np.inf, dtype=np.float64)
    out_idx[: keep.shape[0]] = keep
    out_score[: keep.shape[0]] = score[keep]
    return out_idx, out_score


@dataclasses.dataclass
class OracleResult:
    rows: np.ndarray  # [R] row numbers t
    idx: np.ndarray  # [R, k] int64, -1 padded
    score: np.ndarray  # [R, k] fp64, -inf padded
    rms: np.ndarray  # [R] sqrt(mean over visible keys of I^2)
    kth: np.ndarray  # [R] the k-th (last selected) score
    full: Optional[list]  # per row: fp64 scores of all visible keys (if requested)


def indexer_topk(q: np.ndarray, w: np.ndarray, k: np.ndarray, k_scale: Optional[np.ndarray], dtype: str,
                 topk: int, causal_offset: int, rows: Optional[Sequence[int]] = None,
                 keep_scores: bool = False) -> OracleResult:
    """Exact per-row top-k of the index score for the chosen rows (default: all rows)."""
    T = q.shape[0]
    N = k.shape[0]
    rows = np.arange(T) if rows is None else np.asarray(list(rows), dtype=np.int64)
    kd = decode(k, dtype)
    ks = None if k_scale is None else np.asarray(k_scale, dtype=np.float32).astype(np.float64)
    wd = np.asarray(w, dtype=np.float32).astype(np.float64)
    R = rows.shape[0]
    out_idx = np.empty((R, topk), dtype=np.int64)
    out_score = np.empty((R, topk), dtype=np.float64)
    rms = np.zeros(R)
    kth = np.full(R, -np.inf)
    full = [] if keep_scores else None
    for r, t in enumerate(rows):
        n = visible_keys(int(t), N, causal_offset)
        qd = decode(q[t], dtype)
        s = score_row(qd, wd[t], kd[:n], None if ks is None else ks[:n])
        out_idx[r], out_score[r] = select_topk(s, topk)
        if n > 0:
            rms[r] = np.sqrt(np.mean(s * s))
            kth[r] = out_score[r, min(n, topk) - 1]
        if keep_scores:
            full.append(s)
    return OracleResult(rows=rows, idx=out_idx, score=out_score, rms=rms, kth=kth, full=full)


def indexer_scores(q, w, k, k_scale, dtype: str, causal_offset: int, rows: Sequence[int]) -> np.ndarray:
    """Dense [len(rows), N] fp64 score rows; keys a row may not see hold -inf."""
    N = k.shape[0]
    kd = decode(k, dtype)
    ks = None if k_scale is None else np.asarray(k_scale, dtype=np.float32).astype(np.float64)
    wd = np.asarray(w, dtype=np.float32).astype(np.float64)
    out = np.full((len(rows), N), -np.inf)
    for r, t in enumerate(rows):
        n = visible_keys(int(t), N, causal_offset)
        out[r, :n] = score_row(decode(q[t], dtype), wd[t], kd[:n], None if ks is None else ks[:n])
    return out


def oracle_topk(inp, rows: Optional[Sequence[int]] = None, keep_scores: bool = False) -> OracleResult:
    """Convenience wrapper for an object with q, w, k, k_scale, dtype, topk, causal_offset fields."""
    return indexer_topk(inp.q, inp.w, inp.k, inp.k_scale, inp.dtype, inp.topk, inp.causal_offset,
                        rows=rows, keep_scores=keep_scores)
