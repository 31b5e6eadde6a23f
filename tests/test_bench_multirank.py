"""Host-side logic of the multi-GPU benchmark path (replicas only: no data-path collective), run as
two gloo ranks on the CPU: the reported time is the slowest rank's and the value is the whole-job
aggregate."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 2.0 if rank == 0 else 5.0          # rank 1 is the slow replica
    dist.barrier()
    ms = bench.max_over_ranks(local_ms, world, device="cpu")
    q.put((rank, ms, bench.aggregate_throughput(1e9, ms, world)))
    dist.destroy_process_group()


def test_two_ranks_report_slowest_time_and_aggregate_value():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in out:
        assert ms == 5.0
        assert abs(value - 2 * 1e9 / 5e-3 / 1e9) < 1e-9   # two replicas' bytes over the slowest rank's time


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.aggregate_throughput(2e9, 1.0, 1) == 2000.0
