"""The N > 1 path of the benchmark on CPU: two gloo ranks own disjoint layers (the path
shards over independent units, no data-path collective), the job's time is the maximum over
ranks and the reported throughput is the whole job's."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        layers = bench.rank_layers(rank, 3)
        mine = [10.0 + rank, 2.0 - rank, 5.0]          # per-rank step / prefill / decode times
        agreed = bench.max_over_ranks(mine, dist, "cpu")
        gathered = [None] * world
        dist.all_gather_object(gathered, layers)
        if rank == 0:
            out.put((gathered, agreed, bench.aggregate_throughput(10 ** 9, world, agreed[2])))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_layers_and_agree_on_the_slowest_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, agreed, gbs = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert gathered == [[0, 1, 2], [3, 4, 5]]
    assert agreed == [11.0, 2.0, 5.0]
    assert abs(gbs - 2 * 1.0 / 5e-3) < 1e-9      # 2 ranks x 1 GB in 5 ms
