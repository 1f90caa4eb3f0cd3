"""The entry points are plain stream work (no allocation, no synchronisation, no host read-back), so a
whole call can be captured into a CUDA graph and replayed: what a serving loop does to shed the launch
overhead of the small kernels around the scan.  A replay must return the bits of an eager call, also
after the inputs behind the captured pointers have changed.
"""
import numpy as np
import pytest
import torch

from paper_2607_11976_b200 import binding as lt
from workloads import make_config, make_knn

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("name", ["dsa_bf16", "fp8_ar1"])
def test_indexer_topk_replays_from_a_cuda_graph(name):
    a = make_config(name, T=72, N=20000, topk=384)
    q, w, k, ks = lt.to_device(a)
    idx = torch.empty((a.T, a.topk), dtype=torch.int32, device="cuda")
    score = torch.empty((a.T, a.topk), dtype=torch.float32, device="cuda")
    ws = lt.alloc_workspace(a.dtype, a.T, a.N, a.H, a.D, a.topk)

    def call():
        lt.lt_indexer_topk_ex(a.dtype, q, w, k, ks, a.topk, a.causal_offset, idx, score, ws)

    call()  # eager once: loads the kernels and sets their attributes outside the capture
    torch.cuda.synchronize()
    want_idx, want_score = idx.clone(), score.clone()

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    idx.fill_(-1)
    score.fill_(float("nan"))
    launches = lt.lt_launch_count()
    graph.replay()
    torch.cuda.synchronize()
    assert lt.lt_launch_count() == launches  # a replay goes through no library call
    assert lt.lt_read_status(ws)[0] == 0
    assert torch.equal(idx, want_idx) and np.array_equal(_bits(score), _bits(want_score))

    # new inputs behind the same pointers: reversed key order (and scales), rows shifted by one
    k.copy_(k.flip(0).contiguous())
    if ks is not None:
        ks.copy_(ks.flip(0).contiguous())
    q.copy_(q.roll(1, 0).contiguous())
    w.copy_(w.roll(1, 0).contiguous())
    graph.replay()
    torch.cuda.synchronize()
    got_idx, got_score = idx.clone(), score.clone()
    call()
    torch.cuda.synchronize()
    assert not torch.equal(idx, want_idx)
    assert torch.equal(got_idx, idx) and np.array_equal(_bits(got_score), _bits(score))


def test_knn_topk_replays_from_a_cuda_graph():
    kn = make_knn(T=24, N=30000, D=256, topk=200)
    q = torch.from_numpy(kn.q.view("int16")).to("cuda").view(torch.bfloat16)
    x = torch.from_numpy(kn.x.view("int16")).to("cuda").view(torch.bfloat16)
    idx = torch.empty((kn.T, kn.topk), dtype=torch.int32, device="cuda")
    score = torch.empty((kn.T, kn.topk), dtype=torch.float32, device="cuda")
    ws = torch.empty(lt.lt_knn_topk_workspace_bytes(kn.T, kn.N, kn.D, kn.topk), dtype=torch.uint8, device="cuda")

    def call():
        lt.lt_knn_topk(q, x, kn.topk, idx, score, ws)

    call()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    q.copy_(q.roll(3, 0).contiguous())
    graph.replay()
    torch.cuda.synchronize()
    got_idx, got_score = idx.clone(), score.clone()
    call()
    torch.cuda.synchronize()
    assert lt.lt_read_status(ws)[0] == 0
    assert torch.equal(got_idx, idx) and np.array_equal(_bits(got_score), _bits(score))
