"""The multi-rank arithmetic of bench.py on CPU: two gloo ranks, each an independent replica; the job's time is the
slowest rank's and the throughput is the aggregate.  (The transform has no exchange step, so this is all there is.)"""
import os
import socket

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)           # rank 1 is the slower replica
    out[rank] = (ms, bench.job_throughput(1.0e6, world, ms, 3))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_slowest_time_and_aggregate_throughput():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0
    # 2 ranks x 1e6 samples per step, 3 steps in 15 ms -> 5 ms per step -> 400 Msamples/s
    assert abs(res[0][1] - 400.0) < 1e-9


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks(7.5) == 7.5
    assert abs(bench.job_throughput(32 * 441000.0, 1, 73.5, 100) - 19200.0) < 1.0
