"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU oracle, element by element.

Tolerance (written here as the acceptance rule demands): scores within 1e-3 x the row's RMS score
(oracle.acceptance.REL_TOL); indices equal up to swaps of keys whose oracle scores lie within that
tolerance of the k-th score; and the indices must be bit-exactly the (score desc, index asc) top-k
of the library's own dumped scores.
"""
import numpy as np
import pytest
import torch

from oracle import indexer_scores, oracle_topk
from oracle.acceptance import REL_TOL
from paper_2607_11976_b200 import binding as lt
from workloads import bf16_encode, make_config, make_inputs
from workloads.gen import IndexerInputs

from gpu_util import assert_matches_oracle, assert_own_scores_rule, dump_scores, run_topk, run_unfused

pytestmark = pytest.mark.gpu


def _score_parity(inp, rows, path):
    got = dump_scores(inp, rows[0], rows[-1] + 1, path)
    want = indexer_scores(inp.q, inp.w, inp.k, inp.k_scale, inp.dtype, inp.causal_offset, rows=list(range(rows[0], rows[-1] + 1)))
    worst = 0.0
    for r in range(want.shape[0]):
        vis = np.isfinite(want[r])
        rms = np.sqrt(np.mean(want[r][vis] ** 2)) if vis.any() else 0.0
        assert np.all(np.isneginf(got[r][~vis])), "masked keys must be -inf"
        if vis.any():
            err = np.abs(got[r][vis] - want[r][vis]).max()
            assert err <= REL_TOL * rms, f"row {rows[0] + r}: |err| {err:.3e} > {REL_TOL * rms:.3e}"
            worst = max(worst, err / (REL_TOL * rms))
    return worst


# ---------------------------------------------------------------------------------------------
# config 1 (tiny fp32): generic path, every row
# ---------------------------------------------------------------------------------------------

def test_tiny_f32_scores_and_topk_all_rows():
    inp = make_config("tiny_f32")
    rows = list(range(inp.T))
    _score_parity(inp, rows, lt.LT_PATH_GENERIC)
    idx, score, status = run_topk(inp)
    assert status[0] == 0
    dumped = dump_scores(inp, 0, inp.T)
    assert_matches_oracle(inp, idx, score, rows, dumped)


@pytest.mark.parametrize("dtype", ["bf16", "e4m3"])
def test_generic_path_other_dtypes(dtype):
    inp = make_inputs("ar1" if dtype == "e4m3" else "iid", dtype, T=10, N=700, H=5, D=24, topk=33, seed=3)
    _score_parity(inp, list(range(inp.T)), lt.LT_PATH_GENERIC)
    idx, score, status = run_topk(inp)
    assert_matches_oracle(inp, idx, score, list(range(inp.T)), dump_scores(inp, 0, inp.T))


# ---------------------------------------------------------------------------------------------
# tensor-core scoring (tcgen05) against the oracle and against the SIMT path
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype,recipe", [("bf16", "drift"), ("e4m3", "ar1")])
def test_mma_scores_ragged_shapes(dtype, recipe):
    # T not a multiple of 8, N not a multiple of 128, rows not aligned to the 8-row block
    inp = make_inputs(recipe, dtype, T=27, N=1000, H=64, D=128, topk=16, seed=5)
    _score_parity(inp, list(range(inp.T)), lt.LT_PATH_FUSED)
    _score_parity(inp, list(range(3, 21)), lt.LT_PATH_FUSED)
    a = dump_scores(inp, 0, inp.T, lt.LT_PATH_FUSED)
    b = dump_scores(inp, 0, inp.T, lt.LT_PATH_GENERIC)
    fin = np.isfinite(b)
    assert np.array_equal(np.isfinite(a), fin)
    assert np.abs(a[fin] - b[fin]).max() <= 1e-4 * np.abs(b[fin]).max()


# ---------------------------------------------------------------------------------------------
# fused path: every row of small problems that span several tiles and a ragged tail
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype,recipe", [("bf16", "drift"), ("e4m3", "ar1")])
@pytest.mark.parametrize("T,N,topk", [(40, 5000, 64), (9, 1337, 100), (64, 20000, 512)])
def test_fused_topk_all_rows(dtype, recipe, T, N, topk):
    inp = make_inputs(recipe, dtype, T=T, N=N, H=64, D=128, topk=topk, seed=T + N)
    idx, score, status = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert status[0] & lt.LT_STATUS_TIMEOUT == 0
    dumped = dump_scores(inp, 0, inp.T, lt.LT_PATH_FUSED)
    assert_matches_oracle(inp, idx, score, list(range(inp.T)), dumped)


def test_fused_13_argument_entry_point():
    for name in ("dsa_bf16", "fp8_ar1"):
        inp = make_config(name, T=32, N=6000, topk=128)
        idx, score, status = run_topk(inp, entry="13")
        assert status[0] & lt.LT_STATUS_TIMEOUT == 0
        assert_matches_oracle(inp, idx, score, list(range(inp.T)), dump_scores(inp, 0, inp.T))
    lt.load().lt_shutdown()


# ---------------------------------------------------------------------------------------------
# edge cases
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", ["bf16", "e4m3"])
def test_short_rows_are_padded(dtype):
    # the chunk starts at position 0: row t sees t + 1 keys, fewer than topk for most rows
    inp = make_inputs("ar1" if dtype == "e4m3" else "iid", dtype, T=48, N=48, H=64, D=128, topk=20, seed=9, causal_offset=0)
    idx, score, status = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert_matches_oracle(inp, idx, score, list(range(inp.T)), dump_scores(inp, 0, inp.T, lt.LT_PATH_FUSED))
    assert idx[0].tolist() == [0] + [-1] * 19


def test_no_masking_single_row_and_topk_equals_n():
    inp = make_inputs("iid", "bf16", T=1, N=300, H=64, D=128, topk=300, seed=10, causal_offset=10**6)
    idx, score, _ = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert_matches_oracle(inp, idx, score, [0], dump_scores(inp, 0, 1, lt.LT_PATH_FUSED))
    assert sorted(idx[0].tolist()) == list(range(300))


def test_largest_topk_and_single_row_long_context():
    # topk at the library maximum (8192) on both the fused and the generic path
    inp = make_inputs("iid", "bf16", T=10, N=40000, H=64, D=128, topk=8192, seed=31)
    idx, score, status = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert status[0] & lt.LT_STATUS_TIMEOUT == 0
    assert_matches_oracle(inp, idx, score, list(range(inp.T)), dump_scores(inp, 0, inp.T, lt.LT_PATH_FUSED))
    g_idx, g_score, _ = run_topk(inp, lt.Tunables(path=lt.LT_PATH_GENERIC))
    assert_matches_oracle(inp, g_idx, g_score, list(range(inp.T)), dump_scores(inp, 0, inp.T, lt.LT_PATH_GENERIC))
    # one decode-like row against a long context (many key segments, a single query block)
    one = make_inputs("ar1", "e4m3", T=1, N=300000, H=64, D=128, topk=2048, seed=32)
    idx, score, _ = run_topk(one, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert_matches_oracle(one, idx, score, [0], dump_scores(one, 0, 1, lt.LT_PATH_FUSED))


def test_rows_that_see_nothing():
    inp = make_inputs("iid", "bf16", T=16, N=500, H=64, D=128, topk=8, seed=12, causal_offset=-5)
    idx, score, _ = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert np.all(idx[:4] == -1) and np.all(np.isneginf(score[:4]))
    assert_matches_oracle(inp, idx, score, list(range(inp.T)))


# ---------------------------------------------------------------------------------------------
# the exact fallback and invariance under tunables
# ---------------------------------------------------------------------------------------------

def _axis_inputs(v, T, topk, w_sign=1.0):
    """Head 0 of every query is e0 + 2^-8 e1 with weight w_sign, all other heads are zero, and
    k[s] = (v[s] >> 8) e0 + (v[s] & 255) e1 for integers |v| < 2^16, so every factor is exact in
    bf16 and I[t, s] = w_sign * max(v[s], 0) / 256 exactly: the score order is known in closed form."""
    v = np.asarray(v, dtype=np.int64)
    N = v.shape[0]
    q = np.zeros((T, 64, 128), np.float32)
    q[:, 0, 0] = 1.0
    q[:, 0, 1] = 2.0 ** -8
    k = np.zeros((N, 128), np.float32)
    k[:, 0] = np.sign(v) * (np.abs(v) >> 8)
    k[:, 1] = np.sign(v) * (np.abs(v) & 255)
    w = np.zeros((T, 64), np.float32)
    w[:, 0] = w_sign
    return IndexerInputs("axis", "bf16", bf16_encode(q), w, bf16_encode(k), None, topk, N - T)


def test_monotone_scores_overflow_into_exact_fallback():
    # scores increase with the key index: every key beats the running k-th best, so nothing is
    # filtered, the candidate buffers overflow and the rows must come back exact from the fallback
    N, T, topk = 8192, 24, 32
    inp = _axis_inputs(np.arange(1, N + 1), T, topk)
    # (the paper's 3k-key sample and rank-k rule: the default sample would cover this short context entirely)
    idx, score, status = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED, cap_mult=4, sample_mult=3, sample_rank=-1))
    assert status[0] & lt.LT_STATUS_FALLBACK and status[1] == T and status[4] == T
    for t in range(T):
        p = inp.causal_offset + t
        assert idx[t].tolist() == list(range(p, p - topk, -1))
        assert score[t].tolist() == [(s + 1) / 256.0 for s in range(p, p - topk, -1)]


def test_decreasing_scores_and_negative_weight_ties():
    N, T, topk = 4096, 16, 40
    inp = _axis_inputs(N - np.arange(N), T, topk)
    idx, score, _ = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert all(idx[t].tolist() == list(range(topk)) for t in range(T))
    assert score[0].tolist() == [(N - s) / 256.0 for s in range(topk)]
    # w < 0: every key with v <= 0 scores exactly +0 and beats all positive dots; lowest indices win
    b = np.where(np.arange(N) % 3 == 0, -256, 512)
    inp = _axis_inputs(b, T, topk, w_sign=-1.0)
    idx, score, _ = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert all(idx[t].tolist() == list(range(0, 3 * topk, 3)) for t in range(T))
    assert np.all(score.view(np.uint32) == 0)  # +0.0, never -0.0


def test_overfull_threshold_bin_is_rebinned_not_redone():
    # Scores crowd into one equal-width bin: a few outliers at both ends stretch the sampled range to [0, 254] (bins
    # one unit wide) while 14,000 keys score between 78.1 and 78.9 in steps of 1/256.  The threshold bin then holds
    # more candidates than the final select keeps in shared memory; it must re-bin inside that bin, not give up.
    N, T, topk = 14000, 12, 512
    rng = np.random.default_rng(5)
    v = 20000 + rng.integers(0, 200, size=N)
    # the outliers sit on sampled positions (the strided sample the library will take), so they set the bin range
    n_sample, stride, _ = lt.lt_indexer_sample_plan(N, topk, N - T)
    sampled = stride * rng.choice(n_sample, size=46, replace=False)
    v[sampled[:6]] = 65000
    v[sampled[6:]] = 1
    inp = _axis_inputs(v, T, topk)
    idx, score, status = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert status[1] == 0 and status[0] & lt.LT_STATUS_FALLBACK == 0, "the rows must not need the unfused fallback"
    assert status[2] > 8192, "the case must overfill the final select's buffer, or it tests nothing"
    for t in range(T):
        vis = inp.causal_offset + t + 1
        order = np.lexsort((np.arange(vis), -v[:vis]))[:topk]  # score descending, index ascending
        assert idx[t].tolist() == order.tolist()
        assert score[t].tolist() == (v[order] / 256.0).tolist()


def test_forced_overflow_matches_default_bits():
    inp = make_config("dsa_bf16", T=40, N=12000, topk=256)
    base_idx, base_score, st0 = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    idx, score, st = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED, cap_mult=1))
    assert st[1] > 0 and st[0] & lt.LT_STATUS_FALLBACK
    assert np.array_equal(idx, base_idx) and np.array_equal(score.view(np.uint32), base_score.view(np.uint32))


def test_misjudging_sample_is_caught_and_redone_exactly():
    # rank 1: the initial gate sits at the largest sampled score, far above the true k-th score, so most
    # rows end the scan with fewer than topk survivors; the final select must flag them for the exact fallback
    inp = make_config("fp8_ar1", T=40, N=20000, topk=256)
    base_idx, base_score, st0 = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    idx, score, st = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED, sample_rank=1))
    assert st0[1] == 0
    assert st[1] > 0 and st[0] & lt.LT_STATUS_FALLBACK
    assert np.array_equal(idx, base_idx) and np.array_equal(score.view(np.uint32), base_score.view(np.uint32))
    assert_matches_oracle(inp, idx, score, list(range(0, inp.T, 7)))


@pytest.mark.parametrize("name", ["dsa_bf16", "fp8_ar1"])
def test_tunables_do_not_change_any_output_bit(name):
    inp = make_config(name, T=72, N=30000, topk=512)
    base_idx, base_score, _ = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    for tun in (lt.Tunables(segment_tiles=3), lt.Tunables(segment_tiles=1000, grid=5), lt.Tunables(sample_mult=1),
                lt.Tunables(sample_mult=8, cap_mult=20), lt.Tunables(grid=296, segment_tiles=16),
                lt.Tunables(sample_rank=-1), lt.Tunables(sample_rank=100), lt.Tunables(sample_rank=10 ** 6)):
        tun.path = lt.LT_PATH_FUSED
        idx, score, st = run_topk(inp, tun)
        assert st[0] & lt.LT_STATUS_TIMEOUT == 0
        assert np.array_equal(idx, base_idx) and np.array_equal(score.view(np.uint32), base_score.view(np.uint32))
    u_idx, u_score, _ = run_unfused(inp, rows_per_pass=20)
    assert np.array_equal(u_idx, base_idx) and np.array_equal(u_score.view(np.uint32), base_score.view(np.uint32))


# ---------------------------------------------------------------------------------------------
# adversarial inputs (reduced context; the full-size sweep is in test_gpu_full_size.py)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["adv_planted", "adv_cluster", "adv_ties", "adv_ties_exact"])
@pytest.mark.parametrize("topk", [64, 512, 2048, 4096])
def test_adversarial_reduced(name, topk):
    inp = make_config(name, T=24, N=16384, topk=topk)
    idx, score, status = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert status[0] & lt.LT_STATUS_TIMEOUT == 0
    dumped = dump_scores(inp, 0, inp.T, lt.LT_PATH_FUSED)
    assert_matches_oracle(inp, idx, score, list(range(inp.T)), dumped)
    if name == "adv_ties_exact":
        # every product and sum is exact in fp32 and fp64: the GPU must agree with the oracle bit for bit
        ora = oracle_topk(inp)
        assert np.array_equal(idx.astype(np.int64), ora.idx)
        assert np.array_equal(score.astype(np.float64), ora.score)


def test_random_shapes_fused_path():
    """Seeded random (T, N, topk, causal offset) on both tensor-core dtypes: own-scores rule on every row, oracle on a few."""
    rng = np.random.default_rng(77)
    for i in range(10):
        name = ["dsa_bf16", "fp8_ar1", "hot_fp8", "adv_ties"][i % 4]
        T = int(rng.integers(1, 100))
        N = int(rng.integers(T + 64, 30000))
        topk = int(rng.integers(1, min(N - T, 2500) + 1))
        inp = make_config(name, T=T, N=N, topk=topk)
        idx, score, status = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
        assert status[0] & lt.LT_STATUS_TIMEOUT == 0, (name, T, N, topk)
        dumped = dump_scores(inp, 0, T, lt.LT_PATH_FUSED)
        rows = sorted(set(int(r) for r in rng.integers(0, T, size=3)))
        assert_matches_oracle(inp, idx, score, rows, dumped, 0)
        assert_own_scores_rule(inp, idx, score, dumped, range(T))


@pytest.mark.parametrize("name", ["dsa_bf16", "fp8_ar1"])
@pytest.mark.parametrize("T", [1, 2, 4, 5])
def test_chunks_of_a_few_rows(name, T):
    """Decode-like chunks.  Up to four rows take the one-unit launch of the fused scan (only the first accumulator half
    is issued and finished), five rows the regular one; the dump that arbitrates always runs the regular kernel, so the
    own-scores rule also shows that both launches produce the same score bits."""
    inp = make_config(name, T=T, N=50000, topk=777)
    idx, score, status = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert status[0] & lt.LT_STATUS_TIMEOUT == 0
    dumped = dump_scores(inp, 0, T, lt.LT_PATH_FUSED)
    assert_matches_oracle(inp, idx, score, list(range(T)), dumped, 0)
    # a forced overflow sends the rows through the exact fallback: same bits
    idx2, score2, status2 = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED, cap_mult=1, sample_rank=1))
    assert status2[1] > 0
    assert np.array_equal(idx2, idx) and np.array_equal(score2.view(np.uint32), score.view(np.uint32))


def test_soak_random_problems_with_random_tunables():
    """A wider seeded sweep than the test above: eight recipes, chunks of 1 - 400 rows, up to 600,000 keys, any causal
    offset, k up to 4096, random capacity / sample size / sample rank / work-item length / grid.  The arbiter is the
    library's own dense dump (own-scores rule on every row, bit for bit), so a problem costs a fraction of a second.
    LT_SOAK_PROBLEMS sets how many problems are drawn (default 24; 861 were run once, also against the bounds-checking
    build, without a failure) and LT_SOAK_SEED which sequence."""
    import os
    rng = np.random.default_rng(int(os.environ.get("LT_SOAK_SEED", "1")))
    names = ["dsa_bf16", "fp8_ar1", "hot_fp8", "adv_ties", "adv_planted", "adv_cluster", "adv_ties_exact", "fp8_1m"]
    for _ in range(int(os.environ.get("LT_SOAK_PROBLEMS", "24"))):
        name = names[int(rng.integers(0, len(names)))]
        big = rng.random() < 0.2
        T = int(rng.integers(1, 120 if big else 400))
        N = int(rng.integers(T + 64, 600000 if big else 60000))
        topk = int(rng.integers(1, min(N - T, 4096) + 1))
        co = int(rng.integers(0, N - T + 1)) if rng.random() < 0.5 else None
        r = rng.random()
        if r < 0.25:
            tun = lt.Tunables(path=lt.LT_PATH_FUSED, sample_mult=int(rng.integers(1, 8)), cap_mult=int(rng.integers(2, 16)))
        elif r < 0.4:
            tun = lt.Tunables(path=lt.LT_PATH_FUSED, sample_rank=int(rng.integers(1, 50)))
        elif r < 0.5:
            tun = lt.Tunables(path=lt.LT_PATH_FUSED, segment_tiles=int(rng.integers(1, 64)), grid=int(rng.integers(1, 149)))
        else:
            tun = lt.Tunables(path=lt.LT_PATH_FUSED)
        inp = make_config(name, T=T, N=N, topk=topk, causal_offset=co, seed=int(rng.integers(0, 1 << 30)))
        what = (name, T, N, topk, co, tun.cap_mult, tun.sample_mult, tun.sample_rank, tun.segment_tiles, tun.grid)
        idx, score, status = run_topk(inp, tun)
        assert status[0] & lt.LT_STATUS_TIMEOUT == 0, what
        dumped = dump_scores(inp, 0, T, lt.LT_PATH_FUSED)
        try:
            assert_own_scores_rule(inp, idx, score, dumped, range(T))
        except AssertionError as e:
            raise AssertionError(f"{what}: {e}") from None


@pytest.mark.parametrize("name", ["dsa_bf16", "fp8_ar1", "adv_ties_exact"])
def test_final_select_branches(name):
    """Output sizes on both sides of the final select's branch points (radix sort of 512 .. 4096 gathered candidates,
    select + bitonic sort beyond, tie rows): every row must be the top-k of the library's own scores, in order."""
    for topk in (300, 511, 512, 2047, 3000, 4095, 4096, 5000):
        inp = make_config(name, T=12, N=40000, topk=topk)
        idx, score, status = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
        assert status[0] & lt.LT_STATUS_TIMEOUT == 0, (name, topk)
        dumped = dump_scores(inp, 0, inp.T, lt.LT_PATH_FUSED)
        assert_own_scores_rule(inp, idx, score, dumped, range(inp.T))
