"""The bounds-checking build (-DLT_DEBUG_BOUNDS) stands in for a memory checker: every global store / gather
with a known bound is checked, a failing access is skipped and LT_STATUS_BOUNDS is recorded.  Ordinary cases
must leave the bit clear and return the release build's bits; a page table that points outside the pool must be
caught before the access happens."""
import numpy as np
import pytest
import torch

from paper_2607_11976_b200 import binding as lt
from paper_2607_11976_b200 import build as lt_build
from workloads import make_config, make_knn

from gpu_util import run_topk
from test_gpu_paged import make_pool, run_paged

pytestmark = pytest.mark.gpu


@pytest.fixture()
def debug_library():
    path = lt_build.build(debug_bounds=True)
    lt.use_library(path)
    yield path
    lt.use_library(None)


CASES = [("fp8_ar1", 72, 30000, 512), ("dsa_bf16", 40, 12000, 256), ("tiny_f32", 16, 1500, 64), ("adv_ties_exact", 24, 6000, 300)]


@pytest.mark.parametrize("name,T,N,topk", CASES)
def test_ordinary_cases_leave_the_bounds_bit_clear(name, T, N, topk, debug_library):
    inp = make_config(name, T=T, N=N, topk=topk)
    lt.use_library(None)
    want = run_topk(inp)
    lt.use_library(debug_library)
    for tun in (None, lt.Tunables(cap_mult=1, sample_rank=1)):  # the second one forces rows through the exact fallback
        got = run_topk(inp, tun)
        assert got[2][0] & lt.LT_STATUS_BOUNDS == 0, "a bounds check failed on a valid problem"
        assert got[2][0] & lt.LT_STATUS_TIMEOUT == 0
        assert np.array_equal(got[0], want[0]) and np.array_equal(got[1].view(np.uint32), want[1].view(np.uint32))


def test_paged_cache_is_clean_and_a_bad_page_table_is_caught(debug_library):
    inp = make_config("fp8_ar1", T=40, N=9000, topk=256)
    pool, scale, table = make_pool(inp, seed=5)
    lt.use_library(None)
    want = run_paged(inp, pool, scale, table)
    lt.use_library(debug_library)
    got = run_paged(inp, pool, scale, table)
    assert got[2][0] & lt.LT_STATUS_BOUNDS == 0
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1].view(np.uint32), want[1].view(np.uint32))
    # host-made fault: one visible logical page points far outside the pool.  The checks replace the page by
    # page 0 before any address is formed from it, flag the call, and the call completes.
    bad = table.copy()
    bad[3] = pool.shape[0] // 64 + 1000
    got = run_paged(inp, pool, scale, bad)
    assert got[2][0] & lt.LT_STATUS_BOUNDS, "the page-table entry outside the pool was not caught"
    assert got[2][0] & lt.LT_STATUS_TIMEOUT == 0


def test_knn_is_clean(debug_library):
    from test_gpu_knn import gpu_topk  # the driver of the k-NN parity tests
    inp = make_knn(T=64, N=20000, D=256, topk=128)
    lt.use_library(None)
    want = gpu_topk(inp)
    lt.use_library(debug_library)
    got = gpu_topk(inp)
    assert got[2][0] & lt.LT_STATUS_BOUNDS == 0
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1].view(np.uint32), want[1].view(np.uint32))
