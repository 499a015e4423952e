"""The N > 1 path of bench.py on CPU: two gloo ranks.  The hot path has no
exchange step, so what ranks share is only the batch sharding (each rank its own
utterances) and the reduction of the timing (max) and of the work (sum)."""

import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2609_33645_b200 import workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.reduced(wl.CONFIGS["c2"], V=512, D=16, N=4, T_div=10, U_div=5, name="mr")
    batch = wl.make_batch(cfg, seed=bench.rank_seed(cfg, rank))
    ms, frames, flops = bench.reduce_over_ranks(10.0 + 5.0 * rank, float(batch.M), 8.0 * batch.M * cfg.D * cfg.V)
    out[rank] = (ms, frames, flops, batch.M, int(batch.targets.sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_batches_and_reduce_max_time_sum_work():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    r0, r1 = out[0], out[1]
    assert r0[:3] == r1[:3]                       # every rank holds the same whole-job figures
    assert r0[0] == 15.0                          # max over ranks
    assert r0[1] == r0[3] + r1[3]                 # frames are summed
    assert np.isclose(r0[2], 8.0 * (r0[3] + r1[3]) * 16 * 512)
    assert (r0[3], r0[4]) != (r1[3], r1[4])       # different utterances per rank


def test_single_process_reduction_is_identity():
    import bench
    assert bench.reduce_over_ranks(3.0, 5.0, 7.0) == (3.0, 5.0, 7.0)
