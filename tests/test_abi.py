"""The C-ABI library builds, loads, and exports every symbol the public header declares.
No GPU is needed: only host-side argument checks are exercised."""
import ctypes
import os
import re

import pytest

from paper_2607_11976_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "lt_indexer.h")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lt_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_exported(lib):
    names = declared_functions()
    assert {"lt_indexer_topk", "lt_indexer_topk_ex", "lt_indexer_scores", "lt_unfused_topk",
            "lt_indexer_topk_workspace_bytes", "lt_read_status", "lt_strerror", "lt_version", "lt_shutdown"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in lt_indexer.h but not exported"


def test_version_and_strerror(lib):
    assert lib.lt_version() == 100
    assert lib.lt_strerror(0) == b"ok"
    assert b"invalid" in lib.lt_strerror(-1)
    assert b"unknown" in lib.lt_strerror(-77)


def test_host_side_argument_checks(lib):
    null = ctypes.c_void_p(None)
    fake = ctypes.c_void_p(0x1000)  # aligned, never dereferenced: the checks fail first
    odd = ctypes.c_void_p(0x1004)
    # null pointers
    assert lib.lt_indexer_topk(null, fake, fake, null, 8, 64, 64, 128, 4, 56, fake, null, null) == -1
    # topk > N and non-positive sizes
    assert lib.lt_indexer_topk(fake, fake, fake, null, 8, 64, 64, 128, 65, 56, fake, null, null) == -1
    assert lib.lt_indexer_topk(fake, fake, fake, null, 0, 64, 64, 128, 4, 56, fake, null, null) == -1
    # misaligned q
    assert lib.lt_indexer_topk(odd, fake, fake, null, 8, 64, 64, 128, 4, 56, fake, null, null) == -1
    # unknown dtype, fp8 without scales
    assert lib.lt_indexer_topk_ex(9, fake, fake, fake, null, 8, 64, 64, 128, 4, 56, fake, null, fake, 1 << 30, None, null) == -2
    assert lib.lt_indexer_topk_ex(2, fake, fake, fake, null, 8, 64, 64, 128, 4, 56, fake, null, fake, 1 << 30, None, null) == -1
    # workspace too small / missing
    assert lib.lt_indexer_topk_ex(1, fake, fake, fake, null, 8, 64, 64, 128, 4, 56, fake, null, fake, 16, None, null) == -3
    assert lib.lt_indexer_topk_ex(1, fake, fake, fake, null, 8, 64, 64, 128, 4, 56, fake, null, null, 0, None, null) == -3
    # sampled form: missing sample, sample too large
    assert lib.lt_indexer_topk_sampled(1, fake, fake, fake, null, 8, 64, 64, 128, 4, 56, null, 8, fake, null, fake, 1 << 30, None, null) == -1
    assert lib.lt_indexer_topk_sampled(1, fake, fake, fake, null, 8, 64, 64, 128, 4, 56, fake, 32769, fake, null, fake, 1 << 30, None, null) == -1
    assert lib.lt_indexer_topk_sampled_workspace_bytes(1, 8, 64, 64, 128, 4, 0, None) == 0
    assert lib.lt_indexer_topk_sampled_workspace_bytes(1, 8, 64, 64, 128, 4, 12, None) > lib.lt_indexer_topk_workspace_bytes(1, 8, 64, 64, 128, 4, None) - 4096
    # frequency selector: sizes, workspace
    assert lib.lt_topk_frequent(fake, 8, 4, 64, 65, fake, null, fake, 1 << 20, null) == -1
    assert lib.lt_topk_frequent(fake, 8, 4, 64, 8, fake, null, fake, 16, null) == -3
    assert lib.lt_topk_frequent_workspace_bytes(0) == 0 and lib.lt_topk_frequent_workspace_bytes(1000) >= 4000
    # LiteDSA union builder: group size, slot limit
    assert lib.lt_dsa_union_mask(fake, 8, 4, 64, 0, fake, fake, fake, null) == -1
    assert lib.lt_dsa_union_mask(fake, 8, 8192, 1 << 20, 4096, fake, fake, fake, null) == -1
    # the fused path cannot be forced onto a shape it does not support
    tun = binding.Tunables(path=binding.LT_PATH_FUSED)
    assert lib.lt_indexer_topk_ex(0, fake, fake, fake, null, 8, 64, 8, 64, 4, 56, fake, null, fake, 1 << 30,
                                  ctypes.byref(tun), null) == -2
    assert lib.lt_indexer_scores(1, fake, fake, fake, null, 8, 64, 64, 128, 56, 3, 2, fake, 0, null) == -1
    assert lib.lt_unfused_topk(1, fake, fake, fake, null, 8, 64, 64, 128, 4, 56, fake, null, null, 0, 0, null) == -3


def test_workspace_arithmetic(lib):
    # candidate buffer: 8192 rows x 12k (24,576) entries x 8 B = 1.5 GiB, the figure the paper's Sec. 4.2
    # quotes for k = 2048; the total adds histograms, the sample scores and the fallback scratch
    T, N, H, D, k = 8192, 1 << 20, 64, 128, 2048
    total = binding.lt_indexer_topk_workspace_bytes("e4m3", T, N, H, D, k)
    cand = T * 12 * k * 8
    assert cand == 1536 << 20
    assert cand < total < cand + (1 << 30)
    half = binding.lt_indexer_topk_workspace_bytes("e4m3", T, N, H, D, k, binding.Tunables(cap_mult=6))
    assert total - half == cand // 2
    # invalid problems report 0
    assert binding.lt_indexer_topk_workspace_bytes("bf16", 8, 64, 64, 128, 65) == 0
    assert binding.lt_indexer_topk_workspace_bytes("bf16", 8, 64, 64, 128, 9000) == 0
    # generic path: a bounded dense-score scratch
    g = binding.lt_indexer_topk_workspace_bytes("f32", 64, 4096, 8, 64, 256)
    assert 64 * 4096 * 4 <= g <= 64 * 4096 * 4 + 4096


def test_sample_plan_rank_keeps_misjudgement_below_1e6(lib):
    """The initial gate is too tight for a row only if at least `rank` of the sampled keys fall inside
    the row's true top-k.  With the sample a fixed fraction of the positions the chunk shares and the
    top-k positions unrelated to the stride, that count is hypergeometric; its tail must stay below
    the 1e-6 the header promises.  The paper's rule (rank = topk) can never misjudge."""
    from scipy.stats import hypergeom

    for N, topk, causal_offset in [(1048576, 2048, 1048576 - 4096), (131072, 2048, 131072 - 8192), (65536, 2048, 61440),
                                   (65536, 64, 61440), (65536, 4096, 61440), (4096, 256, 4032), (16384, 256, 16320),
                                   (1 << 22, 8192, (1 << 22) - 128), (20000, 256, 19960)]:
        n_sample, stride, rank = binding.lt_indexer_sample_plan(N, topk, causal_offset)
        prefix = min(causal_offset + 1, N)
        enough = -(-(-(-64 * prefix // topk)) // 128) * 128  # 64 expected top-k keys in the sample, whole key tiles
        floor_n = min(8192, prefix // 32)  # at least 8192 samples, but never more than 1/32 of the prefix
        assert n_sample == min(max(3 * topk, floor_n), enough, prefix) and stride == prefix // n_sample and 1 <= rank <= topk
        if rank < topk:
            # worst case for the tail: all topk of the row's best keys lie in the sampled prefix
            tail = hypergeom.sf(rank - 1, prefix, topk, n_sample)
            assert tail < 1e-6, (N, topk, rank, tail)
        # the paper's rule keeps the paper's sample size
        n2, s2, r2 = binding.lt_indexer_sample_plan(N, topk, causal_offset, binding.Tunables(sample_rank=-1))
        assert (n2, s2, r2) == (min(3 * topk, prefix), prefix // min(3 * topk, prefix), topk)
        assert binding.lt_indexer_sample_plan(N, topk, causal_offset, binding.Tunables(sample_mult=3))[0] == min(3 * topk, prefix)
        assert binding.lt_indexer_sample_plan(N, topk, causal_offset, binding.Tunables(sample_rank=7))[2] == min(7, topk)
    # a sample that is the whole prefix is exhaustive: the deterministic rank is used
    assert binding.lt_indexer_sample_plan(4096, 2048, 4095, binding.Tunables(sample_mult=3)) == (4096, 1, 2048)
    buf = (ctypes.c_int * 3)()
    assert lib.lt_indexer_sample_plan(100, 200, 50, None, buf) == -1
