"""Host side of the real communication window (one process per GPU).

Two jobs, both plumbing over torch.distributed - the reduction itself runs in the window kernel:

* connect(): every rank exports the 64-byte handle of its exchange block, the handles are
  all-gathered, and every rank maps every other rank's block (preserve_comm_import).
* StepGuard: before a step is queued every rank confirms ON THE HOST that all ranks are still
  there.  A rank that left between steps (crashed, exited, never joined) is noticed here, as a
  PeerLost error with the missing rank named, before any kernel would wait for it on the GPU (where
  the wait is bounded as well, but costs its time limit).  Uses a gloo group: host-side control
  messages do not belong on the device collectives' streams.
"""
from __future__ import annotations

from datetime import timedelta
from typing import Optional


class PeerLost(RuntimeError):
    """A rank did not confirm the next step in time."""


def connect(comm, group=None) -> None:
    """All-gather the ranks' exchange-block handles and map the peers' blocks into this process.
    `comm` needs rank, n_ranks, export_handle() -> bytes and import_handle(rank, bytes)."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    if world != comm.n_ranks:
        raise ValueError(f"comm was created for {comm.n_ranks} ranks, the group has {world}")
    mine = comm.export_handle()
    if len(mine) != 64:
        raise ValueError("an exchange-block handle is 64 bytes")
    handles = [None] * world
    dist.all_gather_object(handles, (comm.rank, mine), group=group)
    seen = set()
    for r, h in handles:
        if r in seen or not 0 <= r < world:
            raise ValueError(f"rank {r} announced twice or out of range")
        seen.add(r)
        if r != comm.rank:
            comm.import_handle(r, h)
    dist.barrier(group=group)       # nobody starts a step before everybody has mapped everybody


class StepGuard:
    """Host-side liveness check in front of every step."""

    def __init__(self, control_group, timeout_s: float = 5.0):
        self.group = control_group
        self.timeout = timedelta(seconds=timeout_s)
        self.steps = 0

    def begin_step(self) -> int:
        """Returns the step number once every rank has confirmed it; raises PeerLost otherwise."""
        import torch.distributed as dist
        try:
            dist.monitored_barrier(group=self.group, timeout=self.timeout, wait_all_ranks=False)
        except RuntimeError as e:       # gloo reports which rank failed to respond
            raise PeerLost(f"step {self.steps}: {e}") from e
        self.steps += 1
        return self.steps


def control_group(timeout_s: float = 30.0):
    """A gloo group over all ranks for StepGuard (the default group may be NCCL)."""
    import torch.distributed as dist
    return dist.new_group(backend="gloo", timeout=timedelta(seconds=timeout_s))
