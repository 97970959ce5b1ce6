"""World-size-2 check of the data-parallel bookkeeping on CPU (gloo): replicas share nothing on
the decode path, the job time is the slowest rank's and the job work is the sum."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_22481_b200 import dp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert dp.world() == (rank, world)
        times, units = dp.job_throughput([10.0 + rank, 5.0 - rank], 100.0 * (rank + 1))
        mine = dp.shard_requests(33, world, rank)
        gathered = [None] * world
        dist.all_gather_object(gathered, list(mine))
        out.put((rank, times, units, gathered))
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_slowest_time_and_total_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, times, units, gathered in results:
        assert times == [11.0, 5.0]                  # max over ranks of each timed region
        assert units == 300.0                        # 100 + 200
        assert sorted(gathered[0] + gathered[1]) == list(range(33))
        assert not set(gathered[0]) & set(gathered[1])


def test_single_process_is_its_own_world():
    assert dp.world() == (0, 1)
    assert dp.job_throughput([3.0], 7.0) == ([3.0], 7.0)
    assert [len(dp.shard_requests(10, 4, r)) for r in range(4)] == [3, 3, 2, 2]
    with pytest.raises(ValueError):
        dp.shard_requests(10, 2, 2)
