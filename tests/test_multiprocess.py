"""The N > 1 path of bench.py on CPU: two gloo ranks agree on the max-over-ranks time and
each rank draws its own batch (weak scaling over independent matrices, no collective on the
data path)."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2607_04422_b200 import workloads
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"), world)
    value = bench.aggregate_value(world, 28, 4, ms)
    name, m, n, seed = workloads.stack_3b_shapes(4)[0]
    g = workloads.gradient_like(m // 8, n // 8, seed=bench.rank_seed(seed, rank))
    q.put((rank, ms, value, float(g[0, 0])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_max_time_and_distinct_batches():
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
    assert res[0][1] == res[1][1] == 15.0                  # max over ranks
    assert res[0][2] == res[1][2] == 2 * 28 * 4 / 0.015    # whole-job matrices/s
    assert res[0][3] != res[1][3]                          # different seeds per rank
