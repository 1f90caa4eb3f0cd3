"""LiteDSA union list + membership masks (paper Sec. 3.3) on the GPU against the set-operation oracle.
Integer work: every output word must match."""
import numpy as np
import pytest
import torch

from oracle import pack_mask_words, union_and_masks
from paper_2607_11976_b200 import binding as lt
from workloads import make_config

from gpu_util import run_topk

pytestmark = pytest.mark.gpu


def gpu_union(idx_np, N, group):
    T, topk = idx_np.shape
    n_groups = -(-T // group)
    cap = group * topk
    idx = torch.from_numpy(np.ascontiguousarray(idx_np.astype(np.int32))).cuda()
    union_pos = torch.full((n_groups, cap), 12345, dtype=torch.int32, device="cuda")
    union_len = torch.full((n_groups,), -3, dtype=torch.int32, device="cuda")
    mask = torch.full((T, (cap + 31) // 32), -1, dtype=torch.int32, device="cuda")
    lt.lt_dsa_union_mask(idx, N, group, union_pos, union_len, mask)
    torch.cuda.synchronize()
    return union_pos.cpu().numpy(), union_len.cpu().numpy(), mask.cpu().numpy().view(np.uint32)


def check_against_oracle(idx_np, N, group):
    T, topk = idx_np.shape
    clean = np.where((idx_np >= 0) & (idx_np < N), idx_np, -1)
    unions, masks = union_and_masks(clean, N, group)
    union_pos, union_len, mask = gpu_union(idx_np, N, group)
    cap = group * topk
    for g, u in enumerate(unions):
        assert union_len[g] == u.size, (g, union_len[g], u.size)
        assert np.array_equal(union_pos[g, :u.size].astype(np.int64), u)
        assert np.all(union_pos[g, u.size:] == -1)
    for t in range(T):
        assert np.array_equal(mask[t], pack_mask_words(masks[t], (cap + 31) // 32)), t
    return unions


@pytest.mark.parametrize("T,topk,N,group", [(1, 1, 1, 1), (5, 3, 40, 2), (64, 256, 4096, 8), (70, 100, 30001, 16),
                                            (33, 31, 5000, 7), (128, 2048, 1 << 20, 64), (16, 512, 3_500_000, 8)])
def test_union_and_masks_bit_exact(T, topk, N, group):
    rng = np.random.default_rng(T * 7 + topk)
    # rows of a group share most of their picks (the situation the union list is built for)
    pool = rng.permutation(N)[:min(N, 3 * topk)]
    idx = np.stack([rng.permutation(pool)[:min(topk, pool.size)] for _ in range(T)]).astype(np.int64)
    if idx.shape[1] < topk:
        idx = np.concatenate([idx, np.full((T, topk - idx.shape[1]), -1, dtype=np.int64)], axis=1)
    fresh = rng.random(idx.shape) < 0.1
    idx[fresh] = rng.integers(0, N, size=int(fresh.sum()))  # may repeat a position inside a row: must be harmless
    idx[rng.random(idx.shape) < 0.03] = -1
    unions = check_against_oracle(idx, N, group)
    assert all(u.size <= group * topk for u in unions)


def test_union_of_real_topk_rows_and_bad_arguments():
    inp = make_config("hot_fp8", T=64, N=24000, topk=256)
    idx, _, _ = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    unions = check_against_oracle(idx.astype(np.int64), inp.N, 16)
    # the shared high-scoring keys make a group's union far smaller than group * topk
    assert max(u.size for u in unions) < 4 * inp.topk
    # out-of-range entries are skipped
    weird = idx.astype(np.int64).copy()
    weird[0, :5] = [inp.N, inp.N + 7, 2 ** 31 - 1, -9, -1]
    check_against_oracle(weird, inp.N, 16)
    t = torch.zeros((4, 8), dtype=torch.int32, device="cuda")
    with pytest.raises(lt.LtError) as e:
        lt.lt_dsa_union_mask(t, 100, 0, t, t, t)
    assert e.value.code == -1
