"""Analytical performance model of a decode layer with and without prefetching (host only).

Follows the model of the paper's design-space exploration (Section 5, "Performance & cost
model" and its parameter table): compute time is linear in the accelerator's peak throughput;
memory time is linear in the off-chip bandwidth for bytes that miss the L2 and in the L2 bus
bandwidth for bytes that hit; a collective costs a constant initial latency plus the data size
over the link bandwidth, on a ring.  An operator takes the larger of its compute and memory
times.  Without prefetching every operand byte comes from off-chip memory.  With prefetching,
while a communication operator runs, the operands that Algorithm 1 selected for it (at most C
bytes, and no more than the off-chip memory can deliver during the window) are moved into L2 and
the following operators read those bytes at the L2 bandwidth.

Two additions for a GPU, both off (zero) in the paper's parameter set: a fixed cost per kernel
(launch hand-over and tail, which the paper's graph-engine model does not have) and the share of
that cost that early launch hides.  This module does no device work and imports nothing from the
CUDA binding; the bench prints its predictions beside the measurements.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Sequence


@dataclass(frozen=True)
class Hardware:
    flops: float                  # peak throughput of one device, operations per second
    hbm_bw: float                 # off-chip memory bandwidth, bytes per second
    l2_bw: float                  # L2 bus bandwidth, bytes per second
    l2_bytes: float               # L2 capacity = Algorithm 1's C unless a smaller budget is given
    link_bw: float                # bytes per second per link
    link_latency: float           # seconds, constant part of a transfer
    n_devices: int                # ring size of the collective
    kernel_overhead: float = 0.0  # seconds added to every operator (GPU extension; 0 in the paper's model)
    early_launch_hides: float = 0.0  # seconds of that overhead hidden per operator when operators are launched early


# The paper's parameter table (Section 5): 800 TeraOps/s, HBM 1.84 TB/s, L2 bus 12 TB/s,
# interconnect 200 Gbit/s with 25 us latency; 32 devices unless stated otherwise.
PAPER_TABLE = Hardware(flops=800e12, hbm_bw=1.84e12, l2_bw=12e12, l2_bytes=104 * 2**20, link_bw=200e9 / 8,
                       link_latency=25e-6, n_devices=32)


@dataclass(frozen=True)
class Op:
    name: str
    kind: str                     # "comm" | "matmul" | "attention" | "other"
    flops: float = 0.0
    prefetchable: float = 0.0     # read-only operand bytes (weights, or cached K and V): Algorithm 1's memSize
    other_bytes: float = 0.0      # activations read and written (never prefetched)
    comm_bytes: float = 0.0       # payload of a collective
    overhead: float = 0.0         # seconds of fixed cost of this operator on top of Hardware.kernel_overhead


def allreduce_time(hw: Hardware, nbytes: float) -> float:
    """Ring all-reduce: 2 (P - 1) steps, each moving nbytes / P over one link after the link latency."""
    p = hw.n_devices
    if p <= 1:
        return 0.0
    return 2 * (p - 1) * (hw.link_latency + nbytes / p / hw.link_bw)


def op_time(hw: Hardware, op: Op, l2_hit_bytes: float = 0.0) -> float:
    if op.kind == "comm":
        return allreduce_time(hw, op.comm_bytes) + hw.kernel_overhead + op.overhead
    hit = min(l2_hit_bytes, op.prefetchable)
    mem = (op.prefetchable - hit + op.other_bytes) / hw.hbm_bw + hit / hw.l2_bw
    return max(op.flops / hw.flops, mem) + hw.kernel_overhead + op.overhead


def layer_ops(hidden: int, n_q_heads: int, n_kv_heads: int, head_dim: int, ffn: int, batch: int, sum_ctx: int,
              bytes_per_weight: float = 2.0, bytes_per_kv: float = 2.0, bytes_per_act: float = 2.0,
              window_bytes: float = None) -> List[Op]:
    """One shard's decode layer as the model sees it, in execution order (per-shard sizes)."""
    d, B, H = head_dim, batch, hidden
    nqd, nkvd = n_q_heads * d, n_kv_heads * d
    act = lambda n: n * bytes_per_act
    comm = act(B * H) if window_bytes is None else window_bytes
    return [
        Op("window_a", "comm", comm_bytes=comm, other_bytes=act(3 * B * H)),
        Op("qkv_proj", "matmul", flops=2.0 * B * H * (nqd + 2 * nkvd), prefetchable=H * (nqd + 2 * nkvd) * bytes_per_weight,
           other_bytes=act(B * H + B * (nqd + 2 * nkvd))),
        Op("attention", "attention", flops=4.0 * n_q_heads * d * (sum_ctx + B),
           prefetchable=2.0 * sum_ctx * nkvd * bytes_per_kv, other_bytes=act(2 * B * nqd)),
        Op("o_proj", "matmul", flops=2.0 * B * nqd * H, prefetchable=nqd * H * bytes_per_weight, other_bytes=act(B * nqd + B * H)),
        Op("window_b", "comm", comm_bytes=comm, other_bytes=act(3 * B * H)),
        Op("gate_up_proj", "matmul", flops=4.0 * B * H * ffn, prefetchable=2.0 * H * ffn * bytes_per_weight,
           other_bytes=act(B * H + B * ffn)),
        Op("down_proj", "matmul", flops=2.0 * B * ffn * H, prefetchable=ffn * H * bytes_per_weight, other_bytes=act(B * ffn + B * H)),
    ]


def insert_prefetches(ops: Sequence[Op], budget: float, truncate: bool = False) -> Dict[int, Dict[int, float]]:
    """Algorithm 1 over the operator chain: {index of comm op: {index of op: bytes prefetched}}."""
    plan: Dict[int, Dict[int, float]] = {}
    for i, op in enumerate(ops):
        if op.kind != "comm":
            continue
        plan[i] = {}
        cache_sum = 0.0
        for j in range(i + 1, len(ops)):
            nxt = ops[j]
            if nxt.kind == "comm":
                break
            if nxt.kind in ("matmul", "attention"):
                if cache_sum + nxt.prefetchable < budget:
                    cache_sum += nxt.prefetchable
                    plan[i][j] = nxt.prefetchable
                else:
                    if truncate and budget > cache_sum:
                        plan[i][j] = min(nxt.prefetchable, budget - cache_sum)
                    break
    return plan


def predict(hw: Hardware, ops: Sequence[Op], budget: float = None, truncate: bool = False,
            window_time: float = None) -> Dict[str, float]:
    """Seconds per layer without prefetching, with early launch only, and with prefetching at `budget`
    (default: the L2 capacity).  `window_time` overrides the modelled duration of a communication
    operator (e.g. a measured one)."""
    budget = hw.l2_bytes if budget is None else budget
    win = lambda op: (window_time + hw.kernel_overhead) if window_time is not None else op_time(hw, op)
    off = sum(win(op) if op.kind == "comm" else op_time(hw, op) for op in ops)
    early = off - hw.early_launch_hides * sum(1 for op in ops if op.kind != "comm")
    plan = insert_prefetches(ops, budget, truncate)
    on = 0.0
    hits: Dict[int, float] = {}
    for i, op in enumerate(ops):
        if op.kind == "comm":
            t = win(op)
            on += t
            room = max(t - hw.kernel_overhead, 0.0) * hw.hbm_bw     # what the memory can deliver meanwhile
            for j, nbytes in plan[i].items():
                take = min(nbytes, room)
                hits[j] = take
                room -= take
        else:
            on += op_time(hw, op, hits.get(i, 0.0))
    on -= hw.early_launch_hides * sum(1 for op in ops if op.kind != "comm")
    return {"off": off, "early_launch_only": early, "on": on, "speedup_on_vs_off": off / on,
            "speedup_on_vs_early": early / on,
            "prefetched_bytes": float(sum(hits.values())), "planned_bytes": float(sum(sum(v.values()) for v in plan.values()))}


def calibrate_overheads(hw: Hardware, ops: Sequence[Op], measured_seconds: Sequence[float]) -> List[Op]:
    """Per-operator fixed cost from measured durations of the operators run alone (cold L2):
    overhead = measured - (the model's compute / memory term), never negative.  The calibrated
    operators reproduce the measured times without prefetching; what the model then predicts is
    the effect of moving bytes into L2."""
    out = []
    for op, t in zip(ops, measured_seconds):
        if op.kind == "comm":
            out.append(replace(op, overhead=0.0))
            continue
        base = op_time(replace(hw, kernel_overhead=0.0), replace(op, overhead=0.0))
        out.append(replace(op, overhead=max(t - base - hw.kernel_overhead, 0.0)))
    return out


def l2_size_sweep(hw: Hardware, ops: Sequence[Op], sizes_mib: Sequence[float]) -> List[Dict[str, float]]:
    """Latency versus L2 capacity (the paper's L2-size study), C = the capacity."""
    out = []
    for mib in sizes_mib:
        r = predict(replace(hw, l2_bytes=mib * 2**20), ops)
        out.append({"l2_mib": mib, "latency": r["on"], "speedup": r["speedup_on_vs_off"]})
    return out


def b200_measured(hbm_gbs: float = 6900.0, l2_gbs: float = 18500.0, bf16_tflops: float = 1418.0,
                  l2_bytes: int = 132644864, kernel_overhead_us: float = 2.6, early_hides_us: float = 1.6) -> Hardware:
    """This machine's B200 from measurements: bulk-copy read streams from HBM and from L2 (the stream
    microbenchmark), sustained bf16 throughput, and the fixed per-kernel cost read off the kernel
    timelines (tail plus hand-over to the next kernel; early launch hides part of it).  No link: the
    single-GPU window is a local stand-in whose measured duration is passed to predict()."""
    return Hardware(flops=bf16_tflops * 1e12, hbm_bw=hbm_gbs * 1e9, l2_bw=l2_gbs * 1e9, l2_bytes=l2_bytes,
                    link_bw=770e9, link_latency=2e-6, n_devices=1, kernel_overhead=kernel_overhead_us * 1e-6,
                    early_launch_hides=early_hides_us * 1e-6)
