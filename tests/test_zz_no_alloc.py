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


def test_static_entry_rejects_what_does_not_fit():
    lib = lt.load()
    fake = ctypes.c_void_p(0x1000)
    null = ctypes.c_void_p(None)
    n_too_big = (16 << 20) // 4  # one row of N floats no longer fits behind the 256-byte status block
    rc = lib.lt_indexer_topk_static(1, fake, fake, fake, null, 8, n_too_big, 64, 128, 4, n_too_big - 8, fake, null, null)
    assert rc == -5 and b"fixed scratch" in lib.lt_strerror(rc)
    assert lib.lt_indexer_topk_static(1, null, fake, fake, null, 8, 64, 64, 128, 4, 56, fake, null, null) == -1
