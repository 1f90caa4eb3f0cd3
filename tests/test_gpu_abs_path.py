"""The alternative fp8 scan (lt_tunables.path = LT_PATH_FUSED_ABS): Eq. 1 evaluated as
sum_h (w_h / 2) |x_h| + (1/2) (sum_h w_h q_h) . k, the linear term as e4m3-split columns on the tensor core.
Same acceptance rules as the default path: scores within 1e-3 x the row's RMS score of the oracle, index sets equal
up to swaps inside that tolerance, indices and score bits exactly the top-k of the path's OWN dense scores
(lt_indexer_scores with the same path); fused, dumped and fallback scores of the path agree bit for bit."""
import numpy as np
import pytest
import torch

from paper_2607_11976_b200 import binding as lt
from workloads import make_config

from gpu_util import assert_matches_oracle, dump_scores, run_topk
from test_gpu_paged import make_pool, run_paged

pytestmark = pytest.mark.gpu

ABS = lt.LT_PATH_FUSED_ABS


@pytest.mark.parametrize("name,T,N,topk", [("fp8_ar1", 72, 30000, 512), ("fp8_ar1", 9, 4097, 64), ("hot_fp8", 33, 20031, 300),
                                           ("fp8_ar1", 6, 128, 16), ("fp8_ar1", 130, 9000, 2048), ("fp8_ar1", 7, 700, 900)])
def test_abs_path_matches_oracle_and_its_own_scores(name, T, N, topk):
    inp = make_config(name, T=T, N=N, topk=min(topk, N))
    idx, score, status = run_topk(inp, lt.Tunables(path=ABS))
    assert status[0] & (lt.LT_STATUS_TIMEOUT | lt.LT_STATUS_BOUNDS) == 0
    dumped = dump_scores(inp, 0, inp.T, ABS)
    worst, _ = assert_matches_oracle(inp, idx, score, list(range(inp.T)), dumped)
    assert worst < 0.1, "the five-term split of the linear part should leave the error far inside the tolerance"


def test_abs_path_fallback_and_tunables_keep_every_bit():
    inp = make_config("fp8_ar1", T=50, N=20000, topk=400)
    base = run_topk(inp, lt.Tunables(path=ABS))
    for tun in (lt.Tunables(path=ABS, cap_mult=1, sample_rank=1), lt.Tunables(path=ABS, segment_tiles=16, grid=37),
                lt.Tunables(path=ABS, sample_rank=-1, sample_mult=3)):
        got = run_topk(inp, tun)
        assert np.array_equal(got[0], base[0]) and np.array_equal(got[1].view(np.uint32), base[1].view(np.uint32))
    forced = run_topk(inp, lt.Tunables(path=ABS, cap_mult=1, sample_rank=1))
    assert forced[2][1] > 0, "this tunable set should send rows through the exact fallback"


def test_abs_path_agrees_with_default_path_within_tolerance_and_on_paged_keys():
    inp = make_config("fp8_ar1", T=40, N=9000, topk=256)
    a = run_topk(inp, lt.Tunables(path=ABS))
    pool, scale, table = make_pool(inp, seed=11)
    p = run_paged(inp, pool, scale, table, lt.Tunables(path=ABS))
    assert np.array_equal(p[0], a[0]) and np.array_equal(p[1].view(np.uint32), a[1].view(np.uint32))
    d = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    # two exact evaluations of Eq. 1 with different rounding: nearly all indices coincide, scores agree closely
    same = (a[0] == d[0]).mean()
    assert same > 0.98
    assert np.abs(a[1] - d[1]).max() < 1e-3 * np.abs(d[1]).max()


def test_abs_path_is_fp8_only():
    inp = make_config("dsa_bf16", T=8, N=512, topk=16)
    q, w, k, ks = lt.to_device(inp)
    out_idx = torch.empty((inp.T, inp.topk), dtype=torch.int32, device="cuda")
    ws = lt.alloc_workspace(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk)
    with pytest.raises(lt.LtError) as e:
        lt.lt_indexer_topk_ex(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, out_idx, None, ws, lt.Tunables(path=ABS))
    assert e.value.code == -2
