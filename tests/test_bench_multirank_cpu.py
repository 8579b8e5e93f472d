"""The N > 1 path of bench.py on CPU: two gloo ranks, no GPU.

The hot path has no exchange step, so ranks are independent replicas; what the ranks share is the
timing protocol: barrier, MAX over ranks of the per-rank time, and the whole-job value."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    dist.barrier()
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, torch.device("cpu"), world)
    value = bench.whole_job_value(100.0 / ms, world)
    out[rank] = (ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_the_whole_job_value():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0] == out[1]
    ms, value = out[0]
    assert ms == pytest.approx(15.0)
    assert value == pytest.approx(2 * 100.0 / 15.0)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu"), 1) == 3.5
    assert bench.whole_job_value(7.0, 1) == 7.0
