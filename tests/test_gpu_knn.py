"""k-NN (inner-product) variant on the GPU against its fp64 oracle: dense scores, exact top-k through the
fused path, the bit-exact own-scores rule, forced fallback, tunables."""
import numpy as np
import pytest
import torch

from oracle import knn_topk
from oracle.acceptance import REL_TOL, canonical_topk_of, check_row_indices
from paper_2607_11976_b200 import binding as lt
from workloads import make_knn

pytestmark = pytest.mark.gpu


def to_dev(inp):
    q = torch.from_numpy(inp.q.view("int16")).cuda().view(torch.bfloat16)
    x = torch.from_numpy(inp.x.view("int16")).cuda().view(torch.bfloat16)
    return q, x


def gpu_scores(inp, r0, r1):
    q, x = to_dev(inp)
    out = torch.full((r1 - r0, inp.N), float("nan"), dtype=torch.float32, device="cuda")
    lt.lt_knn_scores(q, x, r0, r1, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def gpu_topk(inp, tunables=None):
    q, x = to_dev(inp)
    out_idx = torch.full((inp.T, inp.topk), -7, dtype=torch.int32, device="cuda")
    out_score = torch.full((inp.T, inp.topk), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(lt.lt_knn_topk_workspace_bytes(inp.T, inp.N, inp.D, inp.topk, tunables), dtype=torch.uint8, device="cuda")
    lt.lt_knn_topk(q, x, inp.topk, out_idx, out_score, ws, tunables)
    status = lt.lt_read_status(ws)
    return out_idx.cpu().numpy(), out_score.cpu().numpy(), status


def check(inp, idx, score, rows, dumped=None):
    o_idx, o_val, rms, full = knn_topk(inp.q, inp.x, inp.topk, rows=rows)
    for r, t in enumerate(rows):
        tol = REL_TOL * rms[r]
        kth = o_val[r][inp.topk - 1]
        ok, msg = check_row_indices(idx[t].astype(np.int64), o_idx[r], full[r], kth, tol)
        assert ok, f"row {t}: {msg}"
        err = np.abs(score[t].astype(np.float64) - full[r][idx[t]]).max()
        assert err <= tol, f"row {t}: score error {err:.3e} > {tol:.3e}"
        if dumped is not None:
            assert np.abs(dumped[t].astype(np.float64) - full[r]).max() <= tol
            want_idx, want_val = canonical_topk_of(dumped[t], inp.N, inp.topk)
            assert np.array_equal(idx[t].astype(np.int64), want_idx), f"row {t}: not the exact top-k of the library's own scores"
            assert np.array_equal(score[t].view(np.uint32), want_val.view(np.uint32))


@pytest.mark.parametrize("T,N,D", [(5, 1000, 128), (64, 5000, 768), (70, 3001, 256), (1, 129, 64), (130, 777, 192)])
def test_dense_scores_match_oracle(T, N, D):
    inp = make_knn(T=T, N=N, D=D, topk=8)
    got = gpu_scores(inp, 0, T)
    _, _, rms, full = knn_topk(inp.q, inp.x, 8)
    assert not np.isnan(got).any()
    assert np.all(np.abs(got.astype(np.float64) - full) <= REL_TOL * rms[:, None])
    # a row sub-range addresses its output relative to row_begin
    if T > 3:
        part = gpu_scores(inp, 2, T - 1)
        assert np.array_equal(part.view(np.uint32), got[2:T - 1].view(np.uint32))


@pytest.mark.parametrize("T,N,D,topk", [(64, 40000, 768, 512), (9, 20000, 128, 64), (100, 30001, 256, 1024), (64, 9000, 768, 4096)])
def test_topk_matches_oracle_and_own_scores(T, N, D, topk):
    inp = make_knn(T=T, N=N, D=D, topk=topk)
    idx, score, st = gpu_topk(inp)
    assert st[0] & lt.LT_STATUS_TIMEOUT == 0
    dumped = gpu_scores(inp, 0, T)
    check(inp, idx, score, list(range(0, T, max(1, T // 9))), dumped)
    for t in range(T):  # own-scores rule for every row
        want_idx, want_val = canonical_topk_of(dumped[t], inp.N, inp.topk)
        assert np.array_equal(idx[t].astype(np.int64), want_idx)
        assert np.array_equal(score[t].view(np.uint32), want_val.view(np.uint32))


def test_fallback_and_tunables_keep_every_bit():
    inp = make_knn(T=20, N=30000, D=256, topk=256)
    base_idx, base_score, st0 = gpu_topk(inp)
    assert st0[1] == 0
    for tun in (lt.Tunables(cap_mult=1), lt.Tunables(sample_rank=1), lt.Tunables(sample_rank=-1), lt.Tunables(segment_tiles=3, grid=7),
                lt.Tunables(sample_mult=1), lt.Tunables(segment_tiles=1000)):
        idx, score, st = gpu_topk(inp, tun)
        assert st[0] & lt.LT_STATUS_TIMEOUT == 0
        assert np.array_equal(idx, base_idx) and np.array_equal(score.view(np.uint32), base_score.view(np.uint32))
    _, _, st = gpu_topk(inp, lt.Tunables(sample_rank=1))
    assert st[1] > 0 and st[0] & lt.LT_STATUS_FALLBACK


def test_bad_arguments():
    inp = make_knn(T=4, N=500, D=128, topk=8)
    q, x = to_dev(inp)
    out = torch.empty((4, 8), dtype=torch.int32, device="cuda")
    ws = torch.empty(lt.lt_knn_topk_workspace_bytes(4, 500, 128, 8), dtype=torch.uint8, device="cuda")
    with pytest.raises(lt.LtError) as e:
        lt.lt_knn_topk(q[:, :100].contiguous(), x[:, :100].contiguous(), 8, out, None, ws)  # D not a multiple of 64
    assert e.value.code == -2
    with pytest.raises(lt.LtError) as e:
        lt.lt_knn_topk(q, x, 8, out, None, ws[:512])
    assert e.value.code == -3
    assert lt.lt_knn_topk_workspace_bytes(4, 500, 100, 8) == 0


def test_full_size_benchmark_shape():
    """The shape bench.py times (64 queries x 1,048,576 vectors x 768, k = 1024, default tunables): every row
    against the oracle's index and score rules, and bit-exactly against the library's own dumped scores."""
    inp = make_knn()
    idx, score, st = gpu_topk(inp)
    assert st[0] == 0 and st[1] == 0, st
    srt = np.sort(idx, axis=1)
    assert idx.min() >= 0 and idx.max() < inp.N and np.all(srt[:, 1:] != srt[:, :-1])
    assert np.all(np.diff(score.astype(np.float64), axis=1) <= 0)
    dumped = np.concatenate([gpu_scores(inp, r, r + 16) for r in range(0, inp.T, 16)])
    check(inp, idx, score, list(range(inp.T)), dumped)


def test_random_shapes():
    rng = np.random.default_rng(2026)
    for _ in range(10):
        T = int(rng.integers(1, 150))
        D = int(rng.choice([64, 128, 320, 768]))
        N = int(rng.integers(200, 40000))
        topk = int(rng.integers(1, min(N, 3000) + 1))
        inp = make_knn(T=T, N=N, D=D, topk=topk)
        idx, score, st = gpu_topk(inp)
        assert st[0] & lt.LT_STATUS_TIMEOUT == 0, (T, N, D, topk)
        dumped = gpu_scores(inp, 0, T)
        rows = sorted(set(int(r) for r in rng.integers(0, T, size=3)))
        check(inp, idx, score, rows, dumped)
        for t in range(T):
            want_idx, want_val = canonical_topk_of(dumped[t], inp.N, inp.topk)
            assert np.array_equal(idx[t].astype(np.int64), want_idx), (T, N, D, topk, t)
