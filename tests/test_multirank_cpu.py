"""The path has no exchange step, so N > 1 means N independent replicas; the only cross-rank logic
is the timing rule (max over ranks) and the whole-job aggregate.  Exercised with two gloo ranks on CPU."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank  # rank 1 is the slow one
    slowest = bench.max_over_ranks(local_ms, world, "cpu")
    value = bench.aggregate_throughput(pairs_per_rank=1000, steps=4, total_ms_max=slowest, world=world)
    dist.barrier()
    out.put((rank, slowest, value))
    dist.destroy_process_group()


def test_two_rank_timing_and_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in results:
        assert slowest == 15.0  # every rank sees the maximum
        assert value == 2 * 1000 * 4 / 15e-3  # whole-job aggregate over both replicas


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(7.5, 1, "cpu") == 7.5
    assert bench.aggregate_throughput(10, 2, 4.0, 1) == 10 * 2 / 4e-3
