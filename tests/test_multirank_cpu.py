"""The N > 1 path of the benchmark is "replicas only": every rank runs the same layer on its own
GPU and the only exchange is the max of the measured times.  That reduction and the aggregate are
exercised here with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 2.0 + rank                       # rank 1 is the slow one
    slow = bench.slowest_rank(mine)
    dist.barrier()
    out.put((rank, slow, bench.aggregate_value(256, world, slow)))
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_sum_of_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [3.0, 3.0]
    assert all(abs(r[2] - 2 * 256 / 3.0) < 1e-12 for r in res)


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.slowest_rank(1.25) == 1.25
    assert bench.aggregate_value(10, 1, 2.0) == 5.0
