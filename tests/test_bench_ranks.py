"""The N > 1 path of bench.py (independent replicas, slowest rank decides) on two gloo ranks."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [1.0 + rank, 10.0 - rank]            # rank 1 is slower on the first timer, rank 0 on the second
    got = bench.max_over_ranks(mine, "cpu")
    value, unit = bench.whole_job_value("hbm", 8e9, 0.0, world, got[0])
    out.put((rank, got, value, unit))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_replicas_take_the_slowest_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value, unit in res:
        assert got == [2.0, 10.0]
        # 2 ranks x 8 GB each over the slowest rank's 2 s
        assert unit == "GB/s" and abs(value - 8.0) < 1e-9


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.5, 1.25]) == [3.5, 1.25]
    v, u = bench.whole_job_value("tensor", 0.0, 2e12, 1, 1.0)
    assert u == "TFLOP/s" and v == 2.0
