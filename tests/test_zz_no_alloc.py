"""The allocation-free entry point (scratch inside the library) against the regular one.

Serving processes that give all spare HBM to their KV cache, and latency-critical callers that cannot
take the device-wide synchronisation of cudaMalloc / cudaFree, call lt_indexer_topk_static instead of
lt_indexer_topk_ex.  It must return the same bits.  Two calls in a row share the library's fixed
scratch array, so the second call also shows that nothing stale from the first one leaks through.
This file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2607_11976_b200 import binding as lt
from workloads import make_config, make_inputs

from gpu_util import run_topk

pytestmark = pytest.mark.gpu


def _run_static(inp):
    q, w, k, ks = lt.to_device(inp)
    out_idx = torch.full((inp.T, inp.topk), -7, dtype=torch.int32, device="cuda")
    out_score = torch.full((inp.T, inp.topk), float("nan"), dtype=torch.float32, device="cuda")
    lt.lt_indexer_topk_static(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, out_idx, out_score)
    torch.cuda.synchronize()
    return out_idx.cpu().numpy(), out_score.cpu().numpy()


def test_static_entry_matches_regular_entry_twice_in_a_row():
    # two different problems back to back: tensor-core dtype first, then the generic fp32 path,
    # then the first one again (its scratch rows were overwritten in between)
    first = make_config("fp8_ar1", T=40, N=9000, topk=300)
    second = make_config("tiny_f32")
    for inp in (first, second, first):
        want_idx, want_score, _ = run_topk(inp)
        got_idx, got_score = _run_static(inp)
        # same tolerance as the other parity tests between two paths of the library: identical bits
        assert np.array_equal(got_idx, want_idx)
        assert np.array_equal(got_score.view(np.uint32), want_score.view(np.uint32))


def test_static_entry_runs_several_passes_over_its_fixed_array():
    """A row of 600,000 scores takes 2.4 MB of the 16 MiB array: 6 rows per pass, four passes, the later
    ones starting at rows that are no multiple of the scan's 8-row blocks.  Same bits as the regular entry,
    a clean status block, and no device memory taken or returned by the call."""
    inp = make_config("dsa_bf16", T=20, N=600000, topk=64)
    want_idx, want_score, _ = run_topk(inp)
    q, w, k, ks = lt.to_device(inp)
    out_idx = torch.full((inp.T, inp.topk), -7, dtype=torch.int32, device="cuda")
    out_score = torch.full((inp.T, inp.topk), float("nan"), dtype=torch.float32, device="cuda")
    lt.lt_indexer_topk_static(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, out_idx, out_score)  # loads the kernels
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    lt.lt_indexer_topk_static(inp.dtype, q, w, k, ks, inp.topk, inp.causal_offset, out_idx, out_score)
    status = lt.lt_read_status_static()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the allocation-free entry point changed the device's free memory"
    assert status[0] & (lt.LT_STATUS_TIMEOUT | lt.LT_STATUS_BOUNDS) == 0
    assert np.array_equal(out_idx.cpu().numpy(), want_idx)
    assert np.array_equal(out_score.cpu().numpy().view(np.uint32), want_score.view(np.uint32))


def test_static_entry_rejects_what_does_not_fit():
    lib = lt.load()
    fake = ctypes.c_void_p(0x1000)
    null = ctypes.c_void_p(None)
    n_too_big = (16 << 20) // 4  # one row of N floats no longer fits behind the 256-byte status block
    rc = lib.lt_indexer_topk_static(1, fake, fake, fake, null, 8, n_too_big, 64, 128, 4, n_too_big - 8, fake, null, null)
    assert rc == -5 and b"fixed scratch" in lib.lt_strerror(rc)
    n_max = lib.lt_indexer_topk_static_max_keys()
    assert n_max == ((16 << 20) - 256) // 4 == 4194240
    # one key more than the largest accepted N is refused before anything is enqueued
    assert lib.lt_indexer_topk_static(1, fake, fake, fake, null, 8, n_max + 1, 64, 128, 4, n_max - 7, fake, null, null) == -5
    assert lib.lt_indexer_topk_static(1, null, fake, fake, null, 8, 64, 64, 128, 4, 56, fake, null, null) == -1
