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


def test_bench_spawns_its_own_ranks_when_started_without_a_launcher():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment starts two ranks itself
    (here with --dry-run: CPU, gloo, nothing timed) and rank 0 reports n_gpus = 2."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run"],
                       capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                     # rank 0 alone prints
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["dry_run"] is True
    assert out["ms_per_step"] == 1.25          # the slowest rank's time

    import bench
    cmd = bench.spawn_command(4, 29999, ["--gpus", "4", "--steps", "7"])
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-4:] == ["--gpus", "4", "--steps", "7"]


def test_bench_byte_accounting_matches_the_library():
    """bench.py's per-kernel byte table sums to the library's algorithmic bytes for every config
    (the reference arm uses the table alone and never loads the CUDA library)."""
    import bench
    from paper_2501_08192_b200 import binding as P
    from paper_2501_08192_b200 import build as B
    from paper_2501_08192_b200 import inputs as I
    B.build()
    for s in I.CONFIGS:
        for sum_ctx in (s.batch * s.ctx, s.batch * 17):
            assert bench.algorithmic_bytes(s, sum_ctx) == P.preserve_algorithmic_bytes(P.make_config(s), s.batch, sum_ctx)
    src = open(os.path.join(ROOT, "bench.py")).read()
    ref = src[src.index("def run_reference"):src.index("def main")]
    assert "binding" not in ref and "libpreserve" not in ref


# ------------------------------------------------ host protocol of the real communication window
class _FakeComm:
    """Stands in for binding.Comm on the CPU: handles are 64 recognisable bytes."""

    def __init__(self, rank, n_ranks):
        self.rank, self.n_ranks, self.imported = rank, n_ranks, {}

    def export_handle(self):
        return bytes([self.rank + 1]) * 64

    def import_handle(self, r, h):
        assert r != self.rank and r not in self.imported
        self.imported[r] = h


def _comm_worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from datetime import timedelta
    dist.init_process_group("gloo", rank=rank, world_size=world, timeout=timedelta(seconds=20))
    from paper_2501_08192_b200 import comm as CM
    c = _FakeComm(rank, world)
    CM.connect(c)
    out[("imported", rank)] = {r: h[0] for r, h in c.imported.items()}
    guard = CM.StepGuard(CM.control_group(10.0), timeout_s=2.0)
    # two steps with everybody present; then the last rank leaves BETWEEN steps (nothing in flight)
    events = []
    for _ in range(2):
        events.append(guard.begin_step())
    if rank == world - 1:
        out[("events", rank)] = events + ["left"]
        os._exit(0)                     # gone without a goodbye
    try:
        guard.begin_step()
        events.append("no error")
    except CM.PeerLost as e:
        events.append("peer lost")
        out[("message", rank)] = str(e)
    out[("events", rank)] = events
    os._exit(0)                          # (a normal shutdown would wait for the rank that left)


def test_exchange_block_handles_travel_and_a_leaving_rank_is_noticed_on_the_host():
    world, port = 3, 29547
    mgr = mp.Manager()
    out = mgr.dict()
    ctx = mp.get_context("spawn")
    procs = [ctx.Process(target=_comm_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    for rank in range(world):
        # every rank mapped every other rank's block, with that rank's handle
        assert out[("imported", rank)] == {r: r + 1 for r in range(world) if r != rank}
    assert out[("events", world - 1)] == [1, 2, "left"]
    # the survivors got a clean error at the next step, not a hang
    assert out[("events", 0)] == [1, 2, "peer lost"]
    assert "step 2" in out[("message", 0)]
    assert out[("events", 1)][:2] == [1, 2] and out[("events", 1)][2] in ("peer lost", "no error")
