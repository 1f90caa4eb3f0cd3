"""Pins for the arbiter of every parity test (oracle/acceptance.py) and for the dense-score oracle.

The acceptance rules decide whether a GPU result passes, so a mistake in them (a tolerance compared the wrong way
round, `extra` and `missing` swapped, a skipped padding check) would make the index rule vacuous without any test
failing.  Each rule is therefore driven with hand-made rows whose outcome is known from the rule's definition:
legal boundary swaps must pass, every kind of illegal result must fail.  `indexer_scores`, the reference of every
dense-score parity check, is compared value by value with the exact-rational brute force.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import indexer_scores, indexer_topk
from oracle.acceptance import REL_TOL, canonical_topk_of, check_row_indices, check_row_scores
from workloads import bf16_encode, quantize_e4m3_per_token
from oracle import decode_bf16, decode_e4m3

from test_oracle_pins import _brute_force, _to_frac


def _row():
    """Ten visible keys, k = 4.  Scores: key 7 and key 2 sit 0.0005 below / at the k-th score."""
    full = np.array([0.10, 0.90, 0.5000, 0.80, 0.20, 0.70, 0.30, 0.4995, 0.00, -0.40])
    oracle_idx = np.array([1, 3, 5, 2])  # 0.90, 0.80, 0.70, 0.50
    kth = 0.5
    return full, oracle_idx, kth


def test_rel_tol_is_the_north_star_value():
    assert REL_TOL == 1e-3


def test_index_rule_accepts_the_oracle_itself_in_any_order():
    full, oracle_idx, kth = _row()
    ok, msg = check_row_indices(oracle_idx.copy(), oracle_idx, full, kth, tol=1e-6)
    assert ok and msg.startswith("0 ")
    ok, _ = check_row_indices(oracle_idx[::-1].copy(), oracle_idx, full, kth, tol=1e-6)  # a set rule: order is checked elsewhere
    assert ok


def test_index_rule_accepts_a_swap_inside_the_tolerance_only():
    full, oracle_idx, kth = _row()
    swapped = np.array([1, 3, 5, 7])  # key 7 (0.4995) instead of key 2 (0.5000): 5e-4 from the k-th score
    ok, msg = check_row_indices(swapped, oracle_idx, full, kth, tol=6e-4)
    assert ok and msg.startswith("1 ")
    ok, msg = check_row_indices(swapped, oracle_idx, full, kth, tol=4e-4)
    assert not ok and "extra" in msg


def test_index_rule_rejects_a_missing_key_far_above_the_kth_score():
    full, oracle_idx, kth = _row()
    # key 7 is within tolerance of the k-th score, but the key it displaced (key 1, score 0.90) is not:
    # the `missing` side must be checked too, not only the `extra` side
    cand = np.array([7, 3, 5, 2])
    ok, msg = check_row_indices(cand, oracle_idx, full, kth, tol=6e-4)
    assert not ok and "missing" in msg


def test_index_rule_rejects_an_extra_key_far_below_the_kth_score():
    full, oracle_idx, kth = _row()
    cand = np.array([1, 3, 5, 4])  # key 4 scores 0.20; the displaced key 2 is the k-th itself, so only `extra` can catch it
    ok, msg = check_row_indices(cand, oracle_idx, full, kth, tol=6e-4)
    assert not ok and "extra" in msg


def test_index_rule_rejects_duplicates_wrong_counts_out_of_range_and_bad_padding():
    full, oracle_idx, kth = _row()
    tol = 1e-3
    assert not check_row_indices(np.array([1, 3, 5, 5]), oracle_idx, full, kth, tol)[0]        # duplicate
    assert not check_row_indices(np.array([1, 3, 5, -1]), oracle_idx, full, kth, tol)[0]       # one key short
    assert not check_row_indices(np.array([1, 3, 5, 10]), oracle_idx, full, kth, tol)[0]       # index = vis(t): outside
    assert not check_row_indices(np.array([1, 3, 5, 12]), oracle_idx, full, kth, tol)[0]       # further outside
    # short row: 3 visible keys, k = 5 -> exactly three indices, then -1 padding
    full3 = np.array([0.3, 0.1, 0.2])
    o3 = np.array([0, 2, 1, -1, -1])
    assert check_row_indices(np.array([0, 2, 1, -1, -1]), o3, full3, 0.1, tol)[0]
    assert not check_row_indices(np.array([0, 2, 1, -1, -7]), o3, full3, 0.1, tol)[0]          # padding must be -1
    assert not check_row_indices(np.array([0, 2, -1, -1, -1]), o3, full3, 0.1, tol)[0]         # a key is missing
    assert not check_row_indices(np.array([0, 2, 1, 1, -1]), o3, full3, 0.1, tol)[0]           # more keys than visible


def test_score_rule_bounds_the_error_and_wants_masked_keys_at_minus_infinity():
    full = np.array([1.0, -2.0, 0.5])
    good = np.array([1.0004, -2.0004, 0.4996, -np.inf, -np.inf], dtype=np.float32)
    ok, err = check_row_scores(good, full, tol=5e-4)
    assert ok and 3e-4 < err < 5e-4
    ok, err = check_row_scores(good, full, tol=3e-4)
    assert not ok                                                          # tolerance the right way round
    leaky = good.copy()
    leaky[3] = 0.0
    assert not check_row_scores(leaky, full, tol=5e-4)[0]                  # a masked key with a finite score
    nan_row = good.copy()
    nan_row[1] = np.nan
    assert not check_row_scores(nan_row, full, tol=5e-4)[0]


def _argmax_select(scores, n_vis, topk):
    """Repeated argmax with strict '>' in ascending index order: the lowest index wins ties."""
    taken, out = [False] * n_vis, []
    for _ in range(min(topk, n_vis)):
        best = None
        for s in range(n_vis):
            if not taken[s] and (best is None or scores[s] > scores[best]):
                best = s
        taken[best] = True
        out.append(best)
    return out + [-1] * (topk - len(out))


def test_canonical_selector_against_repeated_argmax():
    rng = np.random.default_rng(3)
    for trial in range(20):
        n, n_vis, topk = 40, int(rng.integers(0, 41)), int(rng.integers(1, 12))
        row = rng.integers(-3, 4, n).astype(np.float32) / 4  # few levels: many exact ties
        row[rng.integers(0, n, 5)] = -0.0                     # signed zeros among them
        idx, val = canonical_topk_of(row, n_vis, topk)
        want = _argmax_select([float(v) for v in row], n_vis, topk)
        assert idx.tolist() == want
        m = min(topk, n_vis)
        assert np.array_equal(val[:m], row[want[:m]]) and np.isneginf(val[m:]).all()
    # -0.0 and +0.0 are one value: the lower index wins whichever sign it carries
    idx, _ = canonical_topk_of(np.array([-0.0, 0.0, -0.0, 1.0], dtype=np.float32), 4, 3)
    assert idx.tolist() == [3, 0, 1]
    # keys beyond the visible prefix never appear, however large
    idx, _ = canonical_topk_of(np.array([0.1, 0.2, 9.0, 9.0], dtype=np.float32), 2, 3)
    assert idx.tolist() == [1, 0, -1]


@pytest.mark.parametrize("dtype", ["f32", "bf16", "e4m3"])
def test_dense_scores_equal_the_exact_rational_brute_force(dtype):
    """Values (not just the -inf pattern) of indexer_scores for a row subset that does not start at row 0."""
    rng = np.random.default_rng(41)
    T, N, H, D, topk, co = 5, 20, 3, 4, 4, 13
    q = rng.standard_normal((T, H, D)).astype(np.float32)
    k = rng.standard_normal((N, D)).astype(np.float32)
    w = rng.standard_normal((T, H)).astype(np.float32)
    ks = None
    if dtype == "bf16":
        q, k = bf16_encode(q), bf16_encode(k)
        qv, kv = decode_bf16(q), decode_bf16(k)
    elif dtype == "e4m3":
        q, _ = quantize_e4m3_per_token(q)
        k, ks = quantize_e4m3_per_token(k)
        qv, kv = decode_e4m3(q), decode_e4m3(k)
    else:
        qv, kv = q.astype(np.float64), k.astype(np.float64)
    ref = _brute_force(_to_frac(qv), _to_frac(w.astype(np.float64)), _to_frac(kv),
                       [Fraction(1)] * N if ks is None else _to_frac(ks.astype(np.float64)), topk, co)
    rows = [3, 1, 4]
    dense = indexer_scores(q, w, k, ks, dtype, co, rows=rows)
    assert dense.shape == (3, N)
    for r, t in enumerate(rows):
        want = [float(v) for v in ref[t][1]]
        n_vis = len(want)
        assert n_vis == co + t + 1
        assert np.allclose(dense[r, :n_vis], want, rtol=1e-12, atol=1e-15)
        assert np.isneginf(dense[r, n_vis:]).all()


def test_kth_score_of_a_short_row_is_its_last_real_entry():
    """A row that sees fewer than k keys: kth is the score of its last selected key, not padding."""
    rng = np.random.default_rng(8)
    T, N, H, D, topk, co = 3, 10, 2, 3, 6, 2  # rows see 3, 4, 5 keys: all fewer than k = 6
    q = rng.standard_normal((T, H, D)).astype(np.float32)
    k = rng.standard_normal((N, D)).astype(np.float32)
    w = rng.standard_normal((T, H)).astype(np.float32)
    res = indexer_topk(q, w, k, None, "f32", topk, co, keep_scores=True)
    for t in range(T):
        n_vis = co + t + 1
        assert (res.idx[t] >= 0).sum() == n_vis and np.isneginf(res.score[t, n_vis:]).all()
        assert res.kth[t] == res.score[t, n_vis - 1] == res.full[t].min()
        assert np.isfinite(res.kth[t])
