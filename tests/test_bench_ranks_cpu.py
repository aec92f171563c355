"""The benchmark's multi-rank bookkeeping on CPU: two gloo ranks, replicas only.

The path does not shard (one GPU per replica, no collective on the data path); the only
cross-rank step is the max over ranks of the timed region, after which rank 0 reports
the sum of the replicas' bytes over that time."""
import os
import socket
import sys

import pytest

torch = pytest.importorskip("torch")

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + rank, 20.0 - rank]                 # rank 1 is slower on the first, rank 0 on the second
    red = bench.reduce_max(mine, dist, "cpu")
    dist.barrier()
    q.put((rank, red, bench.whole_job_gbs(world, 1_000_000_000, red[0])))
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_bytes():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(2)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, red, gbs in got:
        assert red == [11.0, 20.0]
        assert gbs == pytest.approx(2 * 1e9 / (11.0e-3) / 1e9)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max([3.0, 4.0], None, "cpu") == [3.0, 4.0]
    assert bench.whole_job_gbs(1, 2_833_383_424, 0.5) == pytest.approx(5666.766848)
