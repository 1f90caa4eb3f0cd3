"""Previous-chunk sampler (paper Sec. 3.2 "Sampling") on the GPU: lt_topk_frequent against its oracle
(integer work: bit-exact) and lt_indexer_topk_sampled against lt_indexer_topk_ex (any sample must
leave every output bit unchanged; the previous chunk's frequent positions must tighten the gate)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import frequent_positions
from paper_2607_11976_b200 import binding as lt
from workloads import make_config

from gpu_util import assert_matches_oracle, run_topk

pytestmark = pytest.mark.gpu


def gpu_frequent(idx_np, N, n_out, want_counts=True):
    idx = torch.from_numpy(np.ascontiguousarray(idx_np.astype(np.int32))).cuda()
    out_pos = torch.full((n_out,), -5, dtype=torch.int32, device="cuda")
    out_cnt = torch.full((n_out,), -5, dtype=torch.int32, device="cuda") if want_counts else None
    ws = torch.empty(lt.lt_topk_frequent_workspace_bytes(N), dtype=torch.uint8, device="cuda")
    lt.lt_topk_frequent(idx, N, out_pos, out_cnt, ws)
    torch.cuda.synchronize()
    return out_pos.cpu().numpy(), (out_cnt.cpu().numpy() if want_counts else None)


@pytest.mark.parametrize("T,topk,N,n_out", [(1, 1, 1, 1), (3, 5, 17, 17), (64, 256, 4096, 768), (72, 512, 30001, 1536),
                                            (200, 2048, 1 << 20, 6144), (33, 7, 1000, 999), (500, 64, 100000, 8192)])
def test_frequent_positions_bit_exact(T, topk, N, n_out):
    rng = np.random.default_rng(T * 131 + topk)
    # skewed popularity so that counts have many distinct values and many ties
    weights = 1.0 / (1.0 + np.arange(N) % 977)
    weights /= weights.sum()
    idx = np.stack([rng.choice(N, size=min(topk, N), replace=False, p=weights) for _ in range(T)]).astype(np.int64)
    if idx.shape[1] < topk:
        idx = np.concatenate([idx, np.full((T, topk - idx.shape[1]), -1, dtype=np.int64)], axis=1)
    idx[rng.random(idx.shape) < 0.02] = -1
    pos, cnt = gpu_frequent(idx, N, n_out)
    want_pos, want_cnt = frequent_positions(idx, N, n_out)
    assert np.array_equal(pos.astype(np.int64), want_pos)
    assert np.array_equal(cnt.astype(np.int64), want_cnt)
    pos2, _ = gpu_frequent(idx, N, n_out, want_counts=False)
    assert np.array_equal(pos2, pos)


def test_frequent_positions_ignores_out_of_range_entries_and_rejects_bad_arguments():
    N = 500
    idx = np.array([[3, 3 + N, -1, 499], [499, 7, 2 ** 31 - 1, 3]], dtype=np.int64)
    clean = np.where((idx >= 0) & (idx < N), idx, -1)
    pos, cnt = gpu_frequent(idx, N, 4)
    want_pos, want_cnt = frequent_positions(clean, N, 4)
    assert np.array_equal(pos.astype(np.int64), want_pos) and np.array_equal(cnt.astype(np.int64), want_cnt)
    t = torch.zeros((2, 4), dtype=torch.int32, device="cuda")
    ws = torch.empty(lt.lt_topk_frequent_workspace_bytes(N), dtype=torch.uint8, device="cuda")
    out = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(lt.LtError) as e:
        lt.lt_topk_frequent(t, 4, out, None, ws)  # n_out > N
    assert e.value.code == -1
    with pytest.raises(lt.LtError) as e:
        lt.lt_topk_frequent(t, N, out, None, ws[:256])  # workspace too small
    assert e.value.code == -3


def chunk_of(inp, r0, r1):
    """Rows [r0, r1) of a workload as a prefill chunk of their own: the context ends at the chunk's last position."""
    n_ctx = inp.causal_offset + r1
    return dataclasses.replace(inp, q=inp.q[r0:r1], w=inp.w[r0:r1], k=inp.k[:n_ctx],
                               k_scale=None if inp.k_scale is None else inp.k_scale[:n_ctx],
                               causal_offset=inp.causal_offset + r0)


def run_sampled(inp, sample_np, tunables=None):
    q, w, k, ks = lt.to_device(inp)
    sample = torch.from_numpy(np.ascontiguousarray(sample_np.astype(np.int32))).cuda()
    out_idx = torch.full((inp.T, inp.topk), -7, dtype=torch.int32, device="cuda")
    out_score = torch.full((inp.T, inp.topk), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(lt.lt_indexer_topk_sampled_workspace_bytes(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk,
                                                                sample.numel(), tunables), dtype=torch.uint8, device="cuda")
    lt.lt_indexer_topk_sampled(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, sample, out_idx, out_score, ws, tunables)
    status = lt.lt_read_status(ws)
    return out_idx.cpu().numpy(), out_score.cpu().numpy(), status


def previous_chunk_sample(prev, n_sample):
    prev_idx, _, _ = run_topk(prev, lt.Tunables(path=lt.LT_PATH_FUSED))
    sample, counts = gpu_frequent(prev_idx, prev.N, n_sample)
    want_pos, want_cnt = frequent_positions(prev_idx, prev.N, n_sample)
    assert np.array_equal(sample.astype(np.int64), want_pos) and np.array_equal(counts.astype(np.int64), want_cnt)
    return sample


def test_previous_chunk_sample_tightens_the_gate_and_keeps_every_bit():
    # two consecutive chunks of a context whose high-scoring keys are shared by all rows (the structure the
    # paper's sampler relies on): chunk 1's most frequent top-k positions are the sample of chunk 2
    T, topk = 64, 256
    both = make_config("hot_fp8", T=2 * T, N=24000, topk=topk)
    prev, cur = chunk_of(both, 0, T), chunk_of(both, T, 2 * T)
    sample = previous_chunk_sample(prev, 3 * topk)
    assert sample.max() <= cur.causal_offset  # every sampled position is visible to every row of the next chunk
    assert len(set(sample.tolist()) & set(both.meta["hot_pos"].tolist())) >= topk

    # reference point: the paper's rule (3k keys, k-th largest sampled score) on a position-strided sample
    base_idx, base_score, st_default = run_topk(cur, lt.Tunables(path=lt.LT_PATH_FUSED, sample_mult=3, sample_rank=-1))
    idx, score, st = run_sampled(cur, sample, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert st[0] == 0 and st[1] == 0, st
    assert np.array_equal(idx, base_idx) and np.array_equal(score.view(np.uint32), base_score.view(np.uint32))
    assert_matches_oracle(cur, idx, score, list(range(0, T, 9)))
    # survivors per row: close to topk with the previous chunk's sample, several times topk with the strided one
    assert st[3] / T < 1.6 * topk, st
    assert st[3] < 0.5 * st_default[3], (st, st_default)


@pytest.mark.parametrize("name", ["fp8_ar1", "dsa_bf16"])
def test_previous_chunk_sample_without_shared_structure_is_still_exact(name):
    # iid keys: the previous chunk says little about this one, the gate starts loose (or the small candidate
    # buffer of this reduced case overflows and rows take the fallback); the outputs must not move
    T, topk = 64, 256
    both = make_config(name, T=2 * T, N=24000, topk=topk)
    prev, cur = chunk_of(both, 0, T), chunk_of(both, T, 2 * T)
    sample = previous_chunk_sample(prev, 3 * topk)
    base_idx, base_score, _ = run_topk(cur, lt.Tunables(path=lt.LT_PATH_FUSED))
    idx, score, st = run_sampled(cur, sample, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert st[0] & lt.LT_STATUS_TIMEOUT == 0
    assert np.array_equal(idx, base_idx) and np.array_equal(score.view(np.uint32), base_score.view(np.uint32))
    assert_matches_oracle(cur, idx, score, list(range(0, T, 9)))


def test_any_sample_gives_the_same_bits():
    inp = make_config("fp8_ar1", T=40, N=20000, topk=256)
    fused = lt.Tunables(path=lt.LT_PATH_FUSED)
    base_idx, base_score, _ = run_topk(inp, fused)
    rng = np.random.default_rng(3)
    best = base_idx[0][:256].astype(np.int64)
    samples = {
        "one position": np.array([5]),
        "duplicates of a top key": np.full(768, best[0]),
        "out of range and negative": np.concatenate([rng.integers(0, inp.N, 700), [-4, inp.N, 2 ** 31 - 1, -2 ** 31]]),
        "positions past the causal offset": np.arange(inp.N - 768, inp.N),
        "row 0's own top-k three times": np.tile(best, 3),
        "maximum size": rng.integers(0, inp.causal_offset, 32768),
    }
    for what, sample in samples.items():
        idx, score, st = run_sampled(inp, np.asarray(sample), fused)
        assert st[0] & lt.LT_STATUS_TIMEOUT == 0, what
        assert np.array_equal(idx, base_idx), what
        assert np.array_equal(score.view(np.uint32), base_score.view(np.uint32)), what
    # a sample that makes the gate too tight must show up as fallback rows, not as wrong output
    _, _, st = run_sampled(inp, np.tile(best, 3), fused)
    assert st[1] > 0 and st[0] & lt.LT_STATUS_FALLBACK
    # generic path (fp32 inputs): the sample is ignored
    tiny = make_config("tiny_f32")
    t_idx, t_score, _ = run_topk(tiny)
    s_idx, s_score, _ = run_sampled(tiny, np.arange(100))
    assert np.array_equal(s_idx, t_idx) and np.array_equal(s_score.view(np.uint32), t_score.view(np.uint32))
