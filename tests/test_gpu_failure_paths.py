"""Failure handling exercised without faulting the GPU: a bounded wait that is made to run out returns an
error status and leaves the context usable; the 13-argument entry point's per-device arena grows and shrinks
without changing a bit; a row-strided key view gives the dense layout's bits."""
import numpy as np
import pytest
import torch

from paper_2607_11976_b200 import binding as lt
from workloads import make_config

from gpu_util import assert_matches_oracle, run_topk

pytestmark = pytest.mark.gpu


def test_bounded_wait_gives_up_and_reports():
    """One warp waits 200 us on a barrier nobody arrives at: the wait returns false and raises the abort flag."""
    res = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    lt.lt_debug_wait_timeout(200, res)
    stop.record()
    torch.cuda.synchronize()
    assert res.cpu().tolist() == [0, 1]
    assert 0.1 <= start.elapsed_time(stop) < 50.0  # it did wait about the limit, and not the 2 s default


@pytest.mark.parametrize("name", ["fp8_ar1", "dsa_bf16"])
def test_skipped_key_tile_times_out_and_the_next_call_is_clean(name):
    """The producer of one CTA is told not to load a key tile, the wait limit is 1 ms: the call returns with
    LT_STATUS_TIMEOUT instead of hanging, and an ordinary call right after it matches the oracle."""
    inp = make_config(name, T=8, N=256, topk=32)
    tun = lt.Tunables(path=lt.LT_PATH_FUSED, wait_limit_us=1000, debug_flags=lt.LT_DEBUG_SKIP_ONE_KTILE)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    _, _, status = run_topk(inp, tun)
    stop.record()
    torch.cuda.synchronize()
    assert status[0] & lt.LT_STATUS_TIMEOUT, "the skipped tile should have made a wait run out"
    assert start.elapsed_time(stop) < 1000.0
    idx, score, status = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    assert status[0] & lt.LT_STATUS_TIMEOUT == 0
    assert_matches_oracle(inp, idx, score, list(range(inp.T)))


def test_wait_limit_is_not_a_result_tunable():
    inp = make_config("fp8_ar1", T=24, N=5000, topk=128)
    a = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    b = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED, wait_limit_us=500000))
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))


def test_arena_of_the_13_argument_entry_grows_and_is_reused():
    """small -> larger -> small problems through lt_indexer_topk: each equals lt_indexer_topk_ex bit for bit."""
    for T, N, topk in [(16, 3000, 64), (80, 40000, 512), (16, 3000, 64), (33, 9000, 100)]:
        inp = make_config("fp8_ar1", T=T, N=N, topk=topk)
        want = run_topk(inp, None, entry="ex")
        got = run_topk(inp, None, entry="13")
        assert np.array_equal(got[0], want[0]) and np.array_equal(got[1].view(np.uint32), want[1].view(np.uint32))
        assert got[2][0] & lt.LT_STATUS_TIMEOUT == 0


@pytest.mark.parametrize("name,T,N,topk,pitch", [("fp8_ar1", 40, 9000, 256, 192), ("dsa_bf16", 24, 5000, 128, 136),
                                                 ("fp8_ar1", 9, 4097, 64, 128)])
def test_row_strided_keys_give_the_dense_bits(name, T, N, topk, pitch):
    """Keys as the first D columns of a wider cache (row pitch > D, junk in between)."""
    inp = make_config(name, T=T, N=N, topk=topk)
    want_idx, want_score, _ = run_topk(inp, lt.Tunables(path=lt.LT_PATH_FUSED))
    q, w, k, ks = lt.to_device(inp)
    wide = torch.randint(0, 100, (inp.N, pitch), dtype=torch.uint8 if inp.dtype == "e4m3" else torch.int16, device="cuda")
    if inp.dtype != "e4m3":
        wide = wide.view(torch.bfloat16)
    wide[:, : inp.D] = k
    out_idx = torch.full((inp.T, inp.topk), -7, dtype=torch.int32, device="cuda")
    out_score = torch.full((inp.T, inp.topk), float("nan"), dtype=torch.float32, device="cuda")
    ws = lt.alloc_workspace(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk)
    lt.lt_indexer_topk_strided(inp.dtype, q, w, wide[:, : inp.D], ks, inp.topk, inp.causal_offset, out_idx, out_score, ws)
    st = lt.lt_read_status(ws)
    assert st[0] & lt.LT_STATUS_TIMEOUT == 0
    assert np.array_equal(out_idx.cpu().numpy(), want_idx)
    assert np.array_equal(out_score.cpu().numpy().view(np.uint32), want_score.view(np.uint32))
    # the exact fallback reads the keys through the same pitch: force every row through it
    tun = lt.Tunables(path=lt.LT_PATH_FUSED, cap_mult=1, sample_rank=1)
    ws2 = lt.alloc_workspace(inp.dtype, inp.T, inp.N, inp.H, inp.D, inp.topk, tun)
    out_idx.fill_(-7)
    lt.lt_indexer_topk_strided(inp.dtype, q, w, wide[:, : inp.D], ks, inp.topk, inp.causal_offset, out_idx, out_score, ws2, tun)
    st = lt.lt_read_status(ws2)
    assert st[1] > 0, "this tunable set should send rows through the fallback"
    assert np.array_equal(out_idx.cpu().numpy(), want_idx)
    assert np.array_equal(out_score.cpu().numpy().view(np.uint32), want_score.view(np.uint32))
