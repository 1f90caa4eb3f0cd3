"""Paged key cache: the same keys scattered over a pool of 64-row pages must give the same output bits as the
dense layout (same arithmetic, only the addresses differ), including when rows take the exact fallback."""
import numpy as np
import pytest
import torch

from paper_2607_11976_b200 import binding as lt
from workloads import make_config

from gpu_util import assert_matches_oracle, run_topk

pytestmark = pytest.mark.gpu

PAGE = 64


def make_pool(inp, seed, spare_pages=5):
    """Scatters the keys (and scales) of a workload over a pool of pages in random order, with junk pages in between."""
    rng = np.random.default_rng(seed)
    n_pages = -(-inp.N // PAGE)
    pool_pages = n_pages + spare_pages
    table = rng.permutation(pool_pages)[:n_pages].astype(np.int32)
    k = inp.k
    pool = rng.integers(0, 120, size=(pool_pages * PAGE, inp.D)).astype(k.dtype)  # junk everywhere first (finite codes)
    scale = None if inp.k_scale is None else rng.random(pool_pages * PAGE).astype(np.float32)
    for j, phys in enumerate(table):
        lo, hi = j * PAGE, min(inp.N, (j + 1) * PAGE)
        pool[phys * PAGE: phys * PAGE + (hi - lo)] = k[lo:hi]
        if scale is not None:
            scale[phys * PAGE: phys * PAGE + (hi - lo)] = inp.k_scale[lo:hi]
    return pool, scale, table


def run_paged(inp, pool, scale, table, tunables=None):
    q, w, _, _ = lt.to_device(inp)
    if inp.dtype == "bf16":
        k_pool = torch.from_numpy(pool.view("int16")).cuda().view(torch.bfloat16)
    else:
        k_pool = torch.from_numpy(pool).cuda()
    ks_pool = None if scale is None else torch.from_numpy(scale).cuda()
    pt = torch.from_numpy(table).cuda()
    out_idx = torch.full((inp.T, inp.topk), -7, dtype=torch.int32, device="cuda")
    out_score = torch.full((inp.T, inp.topk), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(lt.lt_indexer_topk_paged_workspace_bytes(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk, tunables),
                     dtype=torch.uint8, device="cuda")
    lt.lt_indexer_topk_paged(inp.dtype, q, w, k_pool, ks_pool, pt, inp.N, inp.topk, inp.causal_offset, out_idx, out_score, ws, tunables)
    status = lt.lt_read_status(ws)
    return out_idx.cpu().numpy(), out_score.cpu().numpy(), status


@pytest.mark.parametrize("name,T,N,topk", [("fp8_ar1", 72, 30000, 512), ("dsa_bf16", 40, 12000, 256), ("fp8_ar1", 9, 4097, 64),
                                           ("dsa_bf16", 64, 16384, 256), ("hot_fp8", 33, 20031, 300)])
def test_paged_cache_gives_the_dense_bits(name, T, N, topk):
    inp = make_config(name, T=T, N=N, topk=topk)
    base_idx, base_score, st0 = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    pool, scale, table = make_pool(inp, seed=T + N)
    idx, score, st = run_paged(inp, pool, scale, table)
    assert st[0] & lt.LT_STATUS_TIMEOUT == 0
    assert np.array_equal(idx, base_idx) and np.array_equal(score.view(np.uint32), base_score.view(np.uint32))
    assert st[3] == st0[3]  # even the number of survivors: the gathered sample holds the same keys as the strided view
    assert_matches_oracle(inp, idx, score, list(range(0, T, max(1, T // 5))))


def test_paged_cache_through_the_fallback_and_bad_arguments():
    inp = make_config("fp8_ar1", T=40, N=20000, topk=256)
    base_idx, base_score, _ = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    pool, scale, table = make_pool(inp, seed=3)
    for tun in (lt.Tunables(cap_mult=1), lt.Tunables(sample_rank=1), lt.Tunables(segment_tiles=3, grid=5)):
        idx, score, st = run_paged(inp, pool, scale, table, tun)
        assert np.array_equal(idx, base_idx) and np.array_equal(score.view(np.uint32), base_score.view(np.uint32))
    _, _, st = run_paged(inp, pool, scale, table, lt.Tunables(cap_mult=1))
    assert st[1] > 0 and st[0] & lt.LT_STATUS_FALLBACK
    with pytest.raises(lt.LtError) as e:
        run_paged(inp, pool, scale, table[:10])  # page table too short for N
    assert e.value.code == -1
    tiny = make_config("tiny_f32")
    assert lt.lt_indexer_topk_paged_workspace_bytes("f32", tiny.T, tiny.N, tiny.H, tiny.D, tiny.topk) == 0
