"""The multi-GPU mode of the benchmark is "replicas only": ranks run independent copies of the
path and exchange one number, the step time, whose maximum gives the whole-job throughput.
That host logic runs here on two CPU ranks over gloo."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow replica
    ms = bench.max_over_ranks(local_ms, world, "cpu")
    value = bench.whole_job_value(1000, world, ms)
    out[rank] = (ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_tokens():
    world = 2
    port = 29500 + os.getpid() % 1000
    # a spawned manager: forking a process that already runs torch's threads is unsafe
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, value = res[0]
    assert ms == 15.0
    assert abs(value - 2 * 1000 / 15e-3) < 1e-6


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(7.5, 1, "cpu") == 7.5
    assert bench.whole_job_value(10, 1, 5.0) == 2000.0
