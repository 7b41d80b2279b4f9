"""The N > 1 arm of bench.py on CPU: two gloo ranks, each with its own batch (no data-path
collective), the job charged the slowest rank's time."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2408_06995_b200 import inputs as I
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    L = bench.rank_layer(I, rank, world)
    slowest = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    value = bench.whole_job_value(L.flops, 7, world, slowest)
    dist.barrier()
    out.put((rank, float(L.x[0, 0, 0, 0]), float(np.abs(L.x).sum()), L.x.shape, slowest, value, L.flops))
    dist.destroy_process_group()


def test_two_ranks_have_their_own_batches_and_share_the_slowest_time():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=300) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, a0, s0, shape0, slow0, v0, f0), (r1, a1, s1, shape1, slow1, v1, f1) = res
    assert shape0 == shape1 == (64, 128, 32, 32)
    assert a0 != a1 and s0 != s1                      # different draws on each rank
    assert slow0 == slow1 == 15.0                     # everyone is charged the slowest rank
    assert v0 == v1 == world * f0 * 7 / 15e-3 / 1e12  # whole-job throughput
