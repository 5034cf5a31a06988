"""The N>1 benchmark path on CPU: two gloo ranks, each timing its own replica; the combined number
uses the slowest rank's time and counts both replicas' bytes."""
import os
import socket

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_15602_b200 import dist_util


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [10.0 + rank, 5.0 - rank]                 # e.g. device-timed ms, end-to-end ms of this rank
        got = dist_util.max_over_ranks(mine)
        dist.barrier()
        out.put((rank, got))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1] == [11.0, 5.0]
    # two replicas of 1 GB per step, slowest rank 11 ms -> 2 GB / 11 ms
    assert abs(dist_util.replica_throughput(10 ** 9, res[0][0], world) - 2e9 / 11e-3 / 1e9) < 1e-9


def test_single_process_is_identity():
    assert dist_util.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert dist_util.replica_throughput(2 * 10 ** 9, 1.0, 1) == 2000.0
