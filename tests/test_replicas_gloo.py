"""N > 1 logic of the benchmark on CPU: two gloo ranks, no GPU.

The path has no exchange step, so N GPUs run N independent replicas; what the ranks share is the timing protocol
(barrier, slowest rank's time) and the whole-job aggregate.  This test runs that protocol with world_size 2.
"""
import os
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))      # rank 1 is the slow one
        val = bench.aggregate_value(2.0e12, steps=4, world=world, ms=ms)
        out.put((rank, ms, val))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_slowest_rank_sets_the_time_and_value_is_whole_job():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, val in res:
        assert ms == 15.0                                    # max over ranks on every rank
        assert abs(val - 2.0e12 * 4 * 2 / 15e-3 / 1e12) < 1e-9   # two replicas' work over the slowest time


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.aggregate_value(1e12, 2, 1, 1000.0) == pytest.approx(2.0)


def test_captured_traffic_is_tied_to_kernel_sources_and_workload(tmp_path, monkeypatch):
    """The bench line prints DRAM traffic only for the kernel sources, workload and call kind the capture was taken on."""
    sys.path.insert(0, ROOT)
    import bench
    assert bench.captured_traffic("spmm_fwd", "another workload") is None
    assert bench.captured_traffic("topology_update", bench.WORKLOAD) is None
    t = bench.captured_traffic("sddmm_dw", bench.WORKLOAD)
    if t is not None:                      # sources unchanged since the capture
        per = bench.NCU_TRAFFIC["launches_per_kind"]
        assert t == (bench.NCU_TRAFFIC["read"]["sddmm_dw"] + bench.NCU_TRAFFIC["write"]["sddmm_dw"]) / per
    # any other digest of the sources: no figure
    monkeypatch.setitem(bench.NCU_TRAFFIC, "sha256_16", "0" * 16)
    assert bench.captured_traffic("sddmm_dw", bench.WORKLOAD) is None
