"""The N > 1 path of bench.py is 'replicas only': no data-path collective, each rank runs the same
work, the job's rate is all ranks' bytes over the slowest rank's time.  The only distributed logic
is that reduction; it is exercised here with two gloo ranks on the CPU."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from conftest import ROOT


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms_local = 2.0 if rank == 0 else 5.0          # rank 1 is the slow one
    slowest = bench.max_over_ranks(ms_local)
    rate = bench.whole_job_gbs(1e9, ms_local, world)
    dist.barrier()
    out.put((rank, slowest, rate))
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time_and_the_whole_job_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, rate in got:
        assert slowest == 5.0                                   # max over ranks, on every rank
        assert rate == pytest.approx(2 * 1e9 / 5e-3 / 1e9)      # 2 replicas' bytes / slowest time


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_gbs(2e9, 1.0, 1) == pytest.approx(2000.0)
