"""The multi-rank host logic of the benchmark (replicas only: no data-path collective),
run as two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # each replica measured a different time; the job's time is the slowest one
    ms = bench.max_over_ranks(1.0 + rank * 0.5, world, device="cpu")
    out[rank] = (ms, bench.whole_job_gbs(73117696, 8, ms, world))
    # replicas draw different inputs: seeds differ per rank
    from dataclasses import replace
    from paper_2501_08192_b200 import inputs as I
    shape = replace(I.small_shape(), seed=I.small_shape().seed + 1000 * rank)
    t = I.make_layers(shape, 1)[0]
    sums = [torch.tensor([float(t["residual_in"].astype("int64").sum())]) for _ in range(world)]
    dist.all_gather(sums, sums[rank])
    out[rank + world] = [float(x) for x in sums]
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate_by_slowest_rank():
    world, port = 2, 29531
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        ms, gbs = out[rank]
        assert ms == 1.5                                   # max over ranks, same on every rank
        assert abs(gbs - 2 * 73117696 * 8 / 1.5e-3 / 1e9) < 1e-6
    a, b = out[world]
    assert a != b and out[world] == out[world + 1]         # different seeds, consistent view
