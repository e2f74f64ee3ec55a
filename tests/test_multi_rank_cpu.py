"""The N > 1 path of bench.py on CPU: two gloo ranks, each owning its own batch of streams (weak
scaling, no collective on the data path); only the timing is reduced (max over ranks)."""
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
    from paper_1804_10727_b200 import workloads
    w = workloads.get("mnist2d", n_streams=8)
    x = bench.rank_input(w, rank, world)
    t = torch.tensor([10.0 + rank, 20.0 - rank], dtype=torch.float64)
    t = bench.max_over_ranks(t, world)
    q.put((rank, x.shape, int(x.astype(np.int64).sum()), t.tolist(), bench.whole_job_value(w, world, steps=3, ms=6.0)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_streams_and_reduce_time_by_max():
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
    (r0, shape0, sum0, t0, v0), (r1, shape1, sum1, t1, v1) = res
    assert shape0 == shape1 == (8, 28, 28, 1)                 # every rank keeps the full per-GPU batch
    assert sum0 != sum1                                        # ... of different streams
    assert t0 == t1 == [11.0, 20.0]                            # max over ranks
    # whole-job throughput: all ranks' pixels over the slowest rank's time
    assert v0 == v1 == 2 * 8 * 28 * 28 * 3 / 6e-3
