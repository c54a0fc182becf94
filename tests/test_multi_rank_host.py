"""The N > 1 path of the benchmark on CPU: the layer has no exchange step, so ranks are independent replicas and the
only cross-rank logic is the timing reduction (maximum over ranks) and the aggregate throughput.  Two gloo ranks."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + rank, 5.0 - rank]                       # rank 1 is slower on the first timing, rank 0 on the second
    got = bench.max_over_ranks(mine, dist, "cpu")
    out.put((rank, got, bench.aggregate_throughput(8192, world, got[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_replica_and_add_up_their_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value in res:
        assert got == [11.0, 5.0]                           # maximum over ranks, element by element
        assert value == 2 * 8192 / 11.0e-3                  # both replicas' rows over the slowest replica's time


def test_single_process_is_the_identity():
    import bench
    assert bench.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert bench.aggregate_throughput(100, 1, 2.0) == 100 / 2.0e-3
