"""CPU oracle for the LiteDSA union list and membership masks.  TEST INFRASTRUCTURE ONLY.

Paper Sec. 3.3 "LiteDSA": adjacent query tokens are grouped; the group's selected
key positions are deduplicated into ONE explicit list shared by all tokens of the
group (a bitmap over the position space is filled with atomic ORs and then swept,
so the list comes out in ascending position order), and every query of the group
gets a bitmask over the slots of that list saying which entries belong to its own
top-k set.  Written out as set operations (numpy unique + isin):

    union[g]   = sorted( U_{t in group g}  { idx[t, j] : idx[t, j] >= 0 } )
    mask[t][s] = 1  iff  union[g(t)][s] is one of idx[t, :]

Readings where the paper is silent: groups are consecutive blocks of `group` rows
(the last one may be shorter); the list order is ascending position (what a bitmap
sweep yields); negative entries are padding; bit s of a row's mask is bit (s % 32)
of 32-bit word s // 32.

Parity pins (tests/test_oracle_pins.py): a pure-Python set brute force on tiny
inputs and invariants (strictly ascending union, mask population = the row's
distinct entries, decoding a mask gives back the row's set, union = OR of masks).
"""
from __future__ import annotations

import numpy as np


def union_and_masks(idx: np.ndarray, N: int, group: int):
    """Returns (unions, masks): unions[g] = int64 array (ascending positions), masks[t] = bool array over unions[g(t)]."""
    idx = np.asarray(idx)
    if idx.ndim != 2 or group <= 0:
        raise ValueError("idx must be [T, k] and group positive")
    T = idx.shape[0]
    unions, masks = [], []
    for g0 in range(0, T, group):
        rows = idx[g0:g0 + group].astype(np.int64)
        valid = rows[rows >= 0]
        if valid.size and valid.max() >= N:
            raise ValueError("index outside [0, N)")
        u = np.unique(valid)
        unions.append(u)
        for r in rows:
            masks.append(np.isin(u, r[r >= 0]))
    return unions, masks


def pack_mask_words(mask: np.ndarray, n_words: int) -> np.ndarray:
    """Bit s of the mask -> bit (s % 32) of uint32 word s // 32, zero padded to n_words words."""
    bits = np.zeros(n_words * 32, dtype=np.uint8)
    bits[:mask.shape[0]] = mask
    return np.packbits(bits.reshape(n_words, 32), axis=1, bitorder="little").view("<u4").reshape(n_words)
