"""Pins for the CPU oracle: things the paper and the mathematics fix, none of which
is the oracle's own formula re-typed.

  * storage-format facts (e4m3 / bf16 bit patterns with known values)
  * a brute force in exact rational arithmetic with a repeated-argmax selector
  * constructed inputs whose score order follows in closed form from Eq. 1
  * invariants and metamorphic relations of Eq. 2
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import decode_bf16, decode_e4m3, indexer_scores, indexer_topk, select_topk, visible_keys
from workloads import bf16_encode, e4m3_encode, make_inputs, quantize_e4m3_per_token

# ----------------------------------------------------------------------------
# storage formats
# ----------------------------------------------------------------------------


def test_e4m3_known_codes():
    # 1-4-3 layout, bias 7, no infinity: these values are fixed by the format definition
    known = {0x00: 0.0, 0x38: 1.0, 0x40: 2.0, 0x7E: 448.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9,
             0x08: 2.0 ** -6, 0x3C: 1.5, 0xB8: -1.0, 0xFE: -448.0, 0x30: 0.5, 0x77: 240.0}
    got = decode_e4m3(np.array(list(known.keys()), dtype=np.uint8))
    assert got.tolist() == list(known.values())
    assert np.isnan(decode_e4m3(np.array([0x7F, 0xFF], dtype=np.uint8))).all()
    # strictly increasing over the positive finite codes (a wrong subnormal rule breaks this at 0x07 -> 0x08)
    pos = decode_e4m3(np.arange(0x7F, dtype=np.uint8))
    assert np.all(np.diff(pos) > 0)


def test_bf16_known_codes():
    known = {0x3F80: 1.0, 0xBF80: -1.0, 0x4000: 2.0, 0x3F00: 0.5, 0x3FC0: 1.5, 0x0000: 0.0, 0x4049: 3.140625}
    got = decode_bf16(np.array(list(known.keys()), dtype=np.uint16))
    assert got.tolist() == list(known.values())


def test_encode_decode_round_trip():
    rng = np.random.default_rng(0)
    # every finite e4m3 code survives decode -> encode
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    back = e4m3_encode(decode_e4m3(codes).astype(np.float32))
    nz = (codes & 0x7F) != 0
    assert np.array_equal(back[nz], codes[nz])
    # nearest rounding: relative error <= 2^-4 for normals, saturation at 448
    x = rng.standard_normal(20000).astype(np.float32) * 50
    d = decode_e4m3(e4m3_encode(x))
    normal = np.abs(x) >= 2.0 ** -6
    assert np.all(np.abs(d[normal] - np.clip(x[normal], -448, 448)) <= np.abs(np.clip(x[normal], -448, 448)) * 2.0 ** -4)
    assert decode_e4m3(e4m3_encode(np.array([1e6, -1e6], dtype=np.float32))).tolist() == [448.0, -448.0]
    # ties to even: 1.0625 is halfway between 1.0 (even mantissa) and 1.125
    assert decode_e4m3(e4m3_encode(np.array([1.0625, 1.1875], dtype=np.float32))).tolist() == [1.0, 1.25]
    # bf16 (7 stored mantissa bits): relative error <= 2^-8, ties to even
    y = rng.standard_normal(20000).astype(np.float32)
    assert np.all(np.abs(decode_bf16(bf16_encode(y)) - y) <= np.abs(y) * 2.0 ** -8)
    assert decode_bf16(bf16_encode(np.array([1.00390625, 1.01171875], dtype=np.float32))).tolist() == [1.0, 1.015625]


def test_per_token_quantisation():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 3, 16)).astype(np.float32)
    x[2] = 0
    codes, scale = quantize_e4m3_per_token(x)
    assert scale[2] == 1.0 and not codes[2].any()
    absmax = np.abs(x.reshape(5, -1)).max(axis=1)
    live = [0, 1, 3, 4]
    assert np.allclose(scale[live], absmax[live] / 448.0, rtol=1e-6)
    # the largest element of each token maps to +-448 exactly
    assert np.all(np.abs(decode_e4m3(codes)).reshape(5, -1).max(axis=1)[live] == 448.0)


# ----------------------------------------------------------------------------
# brute force in exact arithmetic
# ----------------------------------------------------------------------------


def _brute_force(qf, wf, kf, ksf, topk, causal_offset):
    """Eq. 1 / Eq. 2 with Python loops, exact rationals and a repeated-argmax selector."""
    T, H, D = len(qf), len(qf[0]), len(qf[0][0])
    N = len(kf)
    out = []
    for t in range(T):
        n = min(N, max(0, causal_offset + t + 1))
        scores = []
        for s in range(n):
            tot = Fraction(0)
            for j in range(H):
                dot = sum((qf[t][j][d] * kf[s][d] for d in range(D)), Fraction(0))
                if dot > 0:
                    tot += wf[t][j] * dot
            scores.append(tot * ksf[s])
        chosen = []
        taken = [False] * n
        for _ in range(min(topk, n)):
            best = None
            for s in range(n):  # ascending s and strict '>' keeps the lowest index on ties
                if not taken[s] and (best is None or scores[s] > scores[best]):
                    best = s
            taken[best] = True
            chosen.append(best)
        out.append((chosen + [-1] * (topk - len(chosen)), scores))
    return out


def _to_frac(a):
    return [[[Fraction(float(v)) for v in row] for row in m] for m in a] if a.ndim == 3 else (
        [[Fraction(float(v)) for v in row] for row in a] if a.ndim == 2 else [Fraction(float(v)) for v in a])


@pytest.mark.parametrize("dtype", ["f32", "bf16", "e4m3"])
@pytest.mark.parametrize("seed", [0, 1])
def test_brute_force_tiny(dtype, seed):
    rng = np.random.default_rng(100 + seed)
    T, N, H, D, topk, co = 4, 24, 3, 4, 5, 17  # rows see 18..21 keys; N=24 leaves masked keys
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
    res = indexer_topk(q, w, k, ks, dtype, topk, co, keep_scores=True)
    for t in range(T):
        want_idx, want_scores = ref[t]
        assert res.idx[t].tolist() == want_idx
        assert np.allclose(res.full[t], [float(v) for v in want_scores], rtol=1e-12, atol=1e-15)
        assert np.allclose(res.score[t], [float(want_scores[i]) for i in want_idx], rtol=1e-12, atol=1e-15)
        n = len(want_scores)
        assert np.isclose(res.rms[t], np.sqrt(sum(float(v) ** 2 for v in want_scores) / n), rtol=1e-12)
        assert res.kth[t] == res.score[t, topk - 1]


def test_brute_force_with_ties_and_short_rows():
    # integer-valued inputs: many exact ties; causal_offset = 1 makes rows shorter than k
    rng = np.random.default_rng(7)
    T, N, H, D, topk, co = 5, 12, 2, 3, 4, 1
    q = rng.integers(-1, 2, (T, H, D)).astype(np.float32)
    k = rng.integers(-1, 2, (N, D)).astype(np.float32)
    w = rng.integers(-1, 2, (T, H)).astype(np.float32)
    ref = _brute_force(_to_frac(q), _to_frac(w), _to_frac(k), [Fraction(1)] * N, topk, co)
    res = indexer_topk(q, w, k, None, "f32", topk, co)
    for t in range(T):
        assert res.idx[t].tolist() == ref[t][0]
    assert res.idx[0].tolist()[2:] == [-1, -1] and np.isneginf(res.score[0, 2:]).all()  # row 0 sees keys 0, 1 only


# ----------------------------------------------------------------------------
# closed forms: score order known by construction
# ----------------------------------------------------------------------------


def _axis_problem(a, T=3, H=1, topk=4, co=None, w=None, qsign=None):
    """q[t, j] = qsign[j] * e0, k[s] = a[s] * e0, so q.k = qsign[j] * a[s]."""
    N = len(a)
    D = 4
    q = np.zeros((T, H, D), np.float32)
    q[:, :, 0] = 1.0 if qsign is None else np.asarray(qsign, np.float32)[None, :]
    k = np.zeros((N, D), np.float32)
    k[:, 0] = a
    w = np.ones((T, H), np.float32) if w is None else np.broadcast_to(np.asarray(w, np.float32), (T, H)).copy()
    return q, w, k, (N - T if co is None else co), topk


def test_closed_form_increasing_and_decreasing():
    N = 40
    q, w, k, co, topk = _axis_problem(np.arange(1, N + 1, dtype=np.float32))
    res = indexer_topk(q, w, k, None, "f32", topk, co)
    for t in range(3):  # score = a[s] increasing: the newest visible keys win
        p = co + t
        assert res.idx[t].tolist() == [p, p - 1, p - 2, p - 3]
        assert res.score[t].tolist() == [p + 1.0, p + 0.0, p - 1.0, p - 2.0]
    q, w, k, co, topk = _axis_problem(np.arange(N, 0, -1, dtype=np.float32))
    res = indexer_topk(q, w, k, None, "f32", topk, co)
    for t in range(3):
        assert res.idx[t].tolist() == [0, 1, 2, 3]


def test_closed_form_two_heads_relu_branches():
    # heads +e0 and -e0 with weights (1, 2): score = a if a > 0 else 2|a|
    a = np.array([3, -1, 0.5, -4, 2, -0.25, 0, 1], np.float32)
    q, w, k, co, topk = _axis_problem(a, T=1, H=2, topk=8, co=7, w=[1, 2], qsign=[1, -1])
    res = indexer_topk(q, w, k, None, "f32", topk, co)
    want = np.where(a > 0, a, 2 * np.abs(a))
    assert want.tolist() == [3, 2, 0.5, 8, 2, 0.5, 0, 1]
    assert res.idx[0].tolist() == [3, 0, 1, 4, 7, 2, 5, 6]  # ties (2,2) and (.5,.5) by lower index
    assert res.score[0].tolist() == [8, 3, 2, 2, 1, 0.5, 0.5, 0]


def test_closed_form_negative_weight_reverses_and_zero_scores_tie():
    # w < 0: positive dots are ranked in reverse; non-positive dots score exactly 0 and beat them
    a = np.array([2, -1, 5, -3, 1, 0], np.float32)
    q, w, k, co, topk = _axis_problem(a, T=1, topk=6, co=5, w=[-1])
    res = indexer_topk(q, w, k, None, "f32", topk, co)
    assert res.idx[0].tolist() == [1, 3, 5, 4, 0, 2]
    assert res.score[0].tolist() == [0, 0, 0, -1, -2, -5]


def test_closed_form_identical_keys_and_permutation():
    rng = np.random.default_rng(3)
    N, T, topk = 50, 2, 7
    k = np.tile(rng.standard_normal((1, 8)).astype(np.float32), (N, 1))
    q = rng.standard_normal((T, 3, 8)).astype(np.float32)
    w = rng.standard_normal((T, 3)).astype(np.float32)
    res = indexer_topk(q, w, k, None, "f32", topk, N - T)
    assert all(res.idx[t].tolist() == list(range(topk)) for t in range(T))
    # k[s] = pi(s)/N * e0 for a permutation pi: the winners are the positions of the largest visible pi
    pi = rng.permutation(N).astype(np.float32)
    q, w, k, co, topk = _axis_problem(pi / N, T=3, topk=5)
    res = indexer_topk(q, w, k, None, "f32", topk, co)
    for t in range(3):
        vis = co + t + 1
        want = sorted(range(vis), key=lambda s: -pi[s])[:topk]
        assert res.idx[t].tolist() == want


def test_closed_form_fp8_order_follows_key_scale():
    # identical key codes, varying per-key scale: the order is the scale's order
    N, D = 16, 4
    k = np.full((N, D), 0x38, np.uint8)  # every coordinate 1.0
    q = np.full((1, 2, D), 0x38, np.uint8)
    w = np.array([[0.5, 0.25]], np.float32)
    ks = np.array([3, 1, 4, 1, 5, 9, 2, 6, 5, 3, 5, 8, 9, 7, 9, 3], np.float32)
    res = indexer_topk(q, w, k, ks, "e4m3", 6, N - 1)
    assert res.idx[0].tolist() == [5, 12, 14, 11, 13, 7]
    assert res.score[0].tolist() == [27.0, 27.0, 27.0, 24.0, 21.0, 18.0]  # (0.5 + 0.25) * 4 * scale


def test_closed_form_planted_keys_win():
    rng = np.random.default_rng(5)
    T, N, H, D, topk = 3, 200, 4, 16, 10
    q = rng.standard_normal((T, H, D)).astype(np.float32) / 4
    w = np.abs(rng.standard_normal((T, H))).astype(np.float32)
    k = rng.standard_normal((N, D)).astype(np.float32) / 4
    planted = rng.permutation(N - T)[:topk]
    k[planted] = 10 * q[:, 0, :].mean(axis=0)  # huge along a direction every row's head 0 likes
    k[planted] += 10 * q[:, 1, :].mean(axis=0)
    res = indexer_topk(q, w, k, None, "f32", topk, N - T)
    for t in range(T):
        assert sorted(res.idx[t].tolist()) == sorted(planted.tolist())


# ----------------------------------------------------------------------------
# invariants and metamorphic relations
# ----------------------------------------------------------------------------


@pytest.fixture(scope="module")
def small_case():
    return make_inputs("iid", "f32", T=6, N=300, H=4, D=16, topk=20, seed=11)


def test_invariants(small_case):
    inp = small_case
    res = indexer_topk(inp.q, inp.w, inp.k, None, "f32", inp.topk, inp.causal_offset, keep_scores=True)
    for t in range(inp.T):
        n = visible_keys(t, inp.N, inp.causal_offset)
        assert n == inp.causal_offset + t + 1 == inp.visible(t)
        idx = res.idx[t]
        assert len(set(idx.tolist())) == inp.topk and idx.min() >= 0 and idx.max() < n
        rest = np.setdiff1d(np.arange(n), idx)
        assert res.full[t][rest].max() <= res.score[t, -1]
        assert np.all(np.diff(res.score[t]) <= 0)
        assert np.array_equal(res.score[t], res.full[t][idx])


def test_keys_beyond_causal_bound_do_not_matter(small_case):
    inp = small_case
    base = indexer_topk(inp.q, inp.w, inp.k, None, "f32", inp.topk, inp.causal_offset)
    k2 = np.concatenate([inp.k, 100 * np.ones((50, inp.D), np.float32)])
    more = indexer_topk(inp.q, inp.w, k2, None, "f32", inp.topk, inp.causal_offset)
    assert np.array_equal(base.idx, more.idx)
    dense = indexer_scores(inp.q, inp.w, k2, None, "f32", inp.causal_offset, rows=[0, 5])
    assert np.isneginf(dense[0, inp.causal_offset + 1:]).all() and np.isfinite(dense[0, : inp.causal_offset + 1]).all()
    assert np.isneginf(dense[1, inp.causal_offset + 6:]).all() and np.isfinite(dense[1, inp.causal_offset + 5])


def test_key_permutation_permutes_answer(small_case):
    inp = small_case
    co = inp.N - 1  # no masking, so any permutation is legal
    base = indexer_topk(inp.q, inp.w, inp.k, None, "f32", inp.topk, co)
    perm = np.random.default_rng(2).permutation(inp.N)
    res = indexer_topk(inp.q, inp.w, inp.k[perm], None, "f32", inp.topk, co)
    # rows whose selected scores are all distinct have a unique answer (exact-zero scores tie)
    distinct = [t for t in range(inp.T) if np.unique(base.score[t]).shape[0] == inp.topk]
    assert len(distinct) >= 3
    for t in distinct:
        assert np.array_equal(perm[res.idx[t]], base.idx[t])
    assert np.allclose(res.score, base.score, rtol=1e-12)


def test_positive_row_scaling_and_chunk_split(small_case):
    inp = small_case
    base = indexer_topk(inp.q, inp.w, inp.k, None, "f32", inp.topk, inp.causal_offset)
    scaled = indexer_topk(inp.q, inp.w * np.float32(4.0), inp.k, None, "f32", inp.topk, inp.causal_offset)
    assert np.array_equal(base.idx, scaled.idx) and np.allclose(scaled.score, 4 * base.score, rtol=1e-12)
    # rows 3.. as a separate call with the offset advanced by 3
    tail = indexer_topk(inp.q[3:], inp.w[3:], inp.k, None, "f32", inp.topk, inp.causal_offset + 3)
    assert np.array_equal(tail.idx, base.idx[3:]) and np.array_equal(tail.score, base.score[3:])


def test_key_scale_is_a_per_key_factor():
    inp = make_inputs("ar1", "e4m3", T=4, N=120, H=4, D=16, topk=9, seed=21)
    with_scale = indexer_scores(inp.q, inp.w, inp.k, inp.k_scale, "e4m3", inp.N - 1, rows=range(4))
    without = indexer_scores(inp.q, inp.w, inp.k, np.ones(inp.N, np.float32), "e4m3", inp.N - 1, rows=range(4))
    assert np.allclose(with_scale, without * inp.k_scale.astype(np.float64)[None, :], rtol=1e-14)


def test_select_topk_signed_zero_and_padding():
    idx, val = select_topk(np.array([0.0, -0.0, 1.0, -0.0, 0.0]), 4)
    assert idx.tolist() == [2, 0, 1, 3]
    idx, val = select_topk(np.array([1.0, 2.0]), 4)
    assert idx.tolist() == [1, 0, -1, -1] and np.isneginf(val[2:]).all()
    idx, _ = select_topk(np.zeros(0), 2)
    assert idx.tolist() == [-1, -1]


# ---------------------------------------------------------------------------------------------
# previous-chunk sampler (paper Sec. 3.2 "Sampling"): most frequent positions of a top-k matrix
# ---------------------------------------------------------------------------------------------

def test_frequent_positions_matches_counter_brute_force():
    from collections import Counter

    from oracle import frequent_positions

    rng = np.random.default_rng(11)
    for trial in range(40):
        N = int(rng.integers(5, 60))
        T = int(rng.integers(1, 12))
        k = int(rng.integers(1, min(N, 9) + 1))
        idx = np.stack([rng.permutation(N)[:k] for _ in range(T)]).astype(np.int64)
        idx[rng.random(idx.shape) < 0.1] = -1  # padding entries
        n_out = int(rng.integers(1, N + 1))
        c = Counter(int(v) for v in idx.reshape(-1) if v >= 0)
        ranked = sorted(range(N), key=lambda p: (-c.get(p, 0), p))[:n_out]
        pos, cnt = frequent_positions(idx, N, n_out)
        assert pos.tolist() == ranked
        assert cnt.tolist() == [c.get(p, 0) for p in ranked]


def test_frequent_positions_closed_form_and_invariants():
    from oracle import frequent_positions

    # position p appears in exactly (p % 7) rows -> ranking is by p % 7 descending, then p ascending
    N, T = 50, 6
    rows = [[p for p in range(N) if p % 7 > t] for t in range(T)]
    width = max(len(r) for r in rows)
    idx = np.full((T, width), -1, dtype=np.int64)
    for t, r in enumerate(rows):
        idx[t, :len(r)] = r
    pos, cnt = frequent_positions(idx, N, N)
    expect = sorted(range(N), key=lambda p: (-(p % 7), p))
    assert pos.tolist() == expect and cnt.tolist() == [p % 7 for p in expect]
    # invariants: distinct, counts non-increasing, a prefix of the full ranking, blind to row/slot order
    rng = np.random.default_rng(5)
    idx = rng.integers(0, 200, size=(30, 16))
    pos, cnt = frequent_positions(idx, 200, 48)
    assert len(set(pos.tolist())) == 48 and np.all(np.diff(cnt) <= 0)
    assert cnt.sum() <= idx.size and pos.tolist() == frequent_positions(idx, 200, 200)[0][:48].tolist()
    shuffled = rng.permuted(idx[rng.permutation(30)], axis=1)
    assert frequent_positions(shuffled, 200, 48)[0].tolist() == pos.tolist()
    with pytest.raises(ValueError):
        frequent_positions(idx, 100, 10)


# ---------------------------------------------------------------------------------------------
# LiteDSA union list + membership masks (paper Sec. 3.3)
# ---------------------------------------------------------------------------------------------

def test_union_and_masks_match_set_brute_force():
    from oracle import pack_mask_words, union_and_masks

    rng = np.random.default_rng(21)
    for trial in range(30):
        N = int(rng.integers(4, 80))
        T = int(rng.integers(1, 14))
        k = int(rng.integers(1, min(N, 10) + 1))
        group = int(rng.integers(1, 6))
        idx = np.stack([rng.permutation(N)[:k] for _ in range(T)]).astype(np.int64)
        idx[rng.random(idx.shape) < 0.15] = -1
        unions, masks = union_and_masks(idx, N, group)
        assert len(unions) == -(-T // group) and len(masks) == T
        for g, u in enumerate(unions):
            rows = range(g * group, min(T, (g + 1) * group))
            want = sorted(set(int(v) for t in rows for v in idx[t] if v >= 0))
            assert u.tolist() == want
            acc = np.zeros(len(want), dtype=bool)
            for t in rows:
                mine = set(int(v) for v in idx[t] if v >= 0)
                assert [want[s] for s in np.flatnonzero(masks[t])] == sorted(mine)
                acc |= masks[t]
                words = pack_mask_words(masks[t], (group * k + 31) // 32)
                for s in range(len(want)):
                    assert bool((int(words[s // 32]) >> (s % 32)) & 1) == bool(masks[t][s])
                assert all(int(w) == 0 for w in words[(len(want) + 31) // 32:])
            assert acc.all()  # every union entry belongs to at least one row


def test_union_and_masks_closed_form():
    from oracle import union_and_masks

    # row t selects the multiples of (t + 1) below 60; a group of all rows -> union = every position that is a
    # multiple of something in 1..T = everything from 0 to 59; one group per row -> the row's own list, full mask
    T, N = 5, 60
    width = N
    idx = np.full((T, width), -1, dtype=np.int64)
    for t in range(T):
        m = np.arange(0, N, t + 1)
        idx[t, :m.size] = m
    unions, masks = union_and_masks(idx, N, T)
    assert unions[0].tolist() == list(range(N))
    for t in range(T):
        assert np.flatnonzero(masks[t]).tolist() == list(range(0, N, t + 1))
    unions, masks = union_and_masks(idx, N, 1)
    for t in range(T):
        assert unions[t].tolist() == list(range(0, N, t + 1)) and masks[t].all()


# ---------------------------------------------------------------------------------------------
# k-NN (inner-product) variant: Eq. 2 with f(q, x) = q . x over the whole corpus
# ---------------------------------------------------------------------------------------------

def test_knn_oracle_matches_exact_rational_brute_force():
    from fractions import Fraction

    from oracle import decode_bf16, knn_topk
    from workloads import bf16_encode

    rng = np.random.default_rng(31)
    for trial in range(6):
        T, N, D, k = int(rng.integers(1, 4)), int(rng.integers(3, 20)), int(rng.integers(1, 9)), 3
        q = bf16_encode(rng.standard_normal((T, D)).astype(np.float32))
        x = bf16_encode(rng.standard_normal((N, D)).astype(np.float32))
        if trial == 0:
            x[1] = x[0]  # an exact tie: the lower index must win
        qf = [[Fraction(float(v)) for v in row] for row in decode_bf16(q)]
        xf = [[Fraction(float(v)) for v in row] for row in decode_bf16(x)]
        idx, val, rms, full = knn_topk(q, x, min(k, N))
        for t in range(T):
            scores = [sum(a * b for a, b in zip(qf[t], xv)) for xv in xf]
            order = sorted(range(N), key=lambda s: (-scores[s], s))[:min(k, N)]
            assert idx[t].tolist() == order
            assert all(abs(Fraction(float(val[t][j])) - scores[order[j]]) <= Fraction(1, 10 ** 12) for j in range(len(order)))


def test_knn_oracle_agrees_with_indexer_oracle_where_relu_is_identity():
    # H = 1, w = 1, non-negative coordinates: every dot product is >= 0, so Eq. 1 reduces to the inner product
    from oracle import indexer_topk, knn_topk
    from workloads import bf16_encode

    rng = np.random.default_rng(32)
    T, N, D, k = 5, 300, 16, 40
    q = bf16_encode(np.abs(rng.standard_normal((T, D))).astype(np.float32))
    x = bf16_encode(np.abs(rng.standard_normal((N, D))).astype(np.float32))
    idx, val, _, _ = knn_topk(q, x, k)
    ref = indexer_topk(q.reshape(T, 1, D), np.ones((T, 1), dtype=np.float32), x, None, "bf16", k, N)  # every key visible
    assert np.array_equal(idx, ref.idx) and np.allclose(val, ref.score, rtol=0, atol=1e-12)
    # scaling a query by a power of two scales its scores exactly and keeps the selected set
    from oracle import decode_bf16
    q2 = bf16_encode(decode_bf16(q).astype(np.float32) * np.float32(4.0))
    idx2, val2, _, _ = knn_topk(q2, x, k)
    assert np.array_equal(idx2, idx) and np.array_equal(val2, 4.0 * val)
