"""The N > 1 path of bench.py is "replicas only": no data-path collective, only the timing is reduced (max over ranks)
and the throughput summed.  Two gloo ranks on CPU exercise exactly that aggregation."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = [10.0, 12.5][rank]  # rank 1 is slower
    slow = bench.max_over_ranks(dist, ms)
    val = bench.aggregate_throughput(world, 1000, slow * 1e-3)
    dist.barrier()
    out.put((rank, slow, val))
    dist.destroy_process_group()


def test_two_gloo_ranks_report_max_time_and_summed_throughput():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slow, val in res:
        assert slow == 12.5
        assert abs(val - 2 * 1000 / 0.0125) < 1e-6


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(None, 3.25) == 3.25
    assert bench.aggregate_throughput(1, 20000, 0.5) == 40000
