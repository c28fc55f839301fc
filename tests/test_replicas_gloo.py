"""N > 1 runs are independent replicas; the only cross-rank logic is the aggregation of the timing
(max over ranks) and of the processed units (sum over ranks).  Checked with two gloo ranks on CPU."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, units = bench.aggregate(10.0 + 5.0 * rank, 1000 * (rank + 1), world, dist, None)
    q.put((rank, ms, units))
    dist.barrier()
    dist.destroy_process_group()


def test_aggregate_takes_max_time_and_sum_of_units():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29517, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, ms, units in got:
        assert ms == 15.0 and units == 3000.0


def test_aggregate_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(3.5, 77, 1) == (3.5, 77)
