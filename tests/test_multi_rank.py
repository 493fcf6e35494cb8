"""The N > 1 path of bench.py: independent replicas, a barrier on both sides of the timed region,
device time as the maximum over ranks, whole-job throughput = all ranks' updates / that time.
Runs as two gloo ranks on CPU."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank r "measured" (10 + 5 r) ms on the device and (20 + r) ms end to end
    dev_ms, e2e_ms = bench.max_over_ranks([10.0 + 5.0 * rank, 20.0 + rank], world, device="cpu")
    value = bench.whole_job_rate(world, batch=1000, steps=4, ms=dev_ms)
    out[rank] = (dev_ms, e2e_ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_rank_and_the_whole_job():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    for r in range(world):
        dev_ms, e2e_ms, value = res[r]
        assert dev_ms == pytest.approx(15.0) and e2e_ms == pytest.approx(21.0)
        assert value == pytest.approx(2 * 1000 * 4 / 0.015)


def test_single_rank_is_a_no_op():
    import bench
    assert bench.max_over_ranks([3.0, 4.0], 1) == [3.0, 4.0]
    assert bench.whole_job_rate(1, 10, 5, 2.0) == pytest.approx(10 * 5 / 0.002)
