#!/usr/bin/env python
"""Benchmark of the decode-layer hot path (one tensor-parallel shard's decode step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config I]

Metric: decode-layer us/step and effective HBM GB/s (weights + KV + activation
bytes over time), prefetch on vs off.  A "step" is one pass of the whole hot path
over a rotation of R distinct layer instances of the workload (distinct weight
arenas and KV-caches, R x (weights + KV) >= 4 x L2), so every layer-step starts
with a cold L2; per-layer figures are the step's divided by R.
`value` is the effective GB/s with the library's default prefetch setting and
inputs resident in HBM; `e2e` is the same metric through the host-buffer entry
point with host<->device copies inside the timed region.  With --gpus N each rank
runs an independent shard replica (no data-path collective; weak scaling).
The reference arm times the CPU oracle on the host cores.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode-layer us/step and effective HBM GB/s (% of roofline), prefetch on vs off"
SWEEP_FRACS = (0.0, 1 / 16, 1 / 8, 1 / 4, 3 / 8, 1 / 2, 5 / 8, 3 / 4, 7 / 8, 1.0)

# DRAM traffic per launch of the dominant kernel from an ncu capture (bytes), keyed by
# (kernel, workload); see profiles/.  None where no capture exists.
NCU_TRAFFIC = {
    # profiles/ncu_full_gemv_attn_window_config1_small.md (dram__bytes_read.sum + dram__bytes_write.sum)
    # gate/up: its own 29.45 MB + the 14.68 MB of down-projection weights that its CTAs prefetch into L2 at the end
    ("gate_up_proj", 1): 44220000, ("down_proj", 1): 14790000, ("qkv_proj", 1): 6470000, ("o_proj", 1): 4260000,
    ("attn_splitkv", 1): 16830000, ("attn_merge", 1): 380000, ("window_a", 1): 630000, ("window_b", 1): 760000,
    # profiles/ncu_full_gemm_tcgen05_config3_small.md, profiles/ncu_full_attn_splitkv_config5.md
    ("gate_up_proj", 2): 121910000, ("down_proj", 2): 59230000, ("qkv_proj", 2): 21560000, ("o_proj", 2): 16890000,
    ("attn_splitkv", 4): 542870000,
}
NCU_TRAFFIC_NOTE = {
    ("gate_up_proj", 1): "captured in the layer chain: includes 14.68 MB of the next kernel's weights, prefetched into L2 by "
                         "this kernel's CTAs once their own stream is over (served from L2 to the down projection: 256 B of "
                         "DRAM reads there); its own bytes are 29.54 MB, and the kernel timed alone does not prefetch",
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy bandwidth)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        super().__init__(daemon=True)
        self.gpu = gpu_index
        self.samples = []
        self.stop_flag = threading.Event()

    def run(self):
        while not self.stop_flag.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5)
                if out.returncode == 0 and out.stdout.strip():
                    self.samples.append([s.strip() for s in out.stdout.strip().split(",")])
            except Exception:
                pass
            self.stop_flag.wait(0.2)

    def summary(self):
        self.stop_flag.set()
        self.join(timeout=6)
        sm = [int(s[0]) for s in self.samples if s[0].isdigit()]
        mx = [int(s[1]) for s in self.samples if len(s) > 1 and s[1].isdigit()]
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        reasons = sorted({n for s in self.samples for n, v in zip(names, s[2:6]) if v.lower().startswith("active")})
        return {"sm_mhz": int(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def kernel_bytes(s, sum_ctx: int):
    """Algorithmic bytes per launch of each main-stream kernel (order: binding.KERNEL_NAMES)."""
    B, H, d, P_ = s.batch, s.hidden, s.head_dim, s.tp_degree
    BH, Bq, Bkv, BF = B * H * 2, B * s.n_q_heads * d * 2, B * s.n_kv_heads * d * 2, B * s.ffn * 2
    wqkv = 2 * H * (s.n_q_heads + 2 * s.n_kv_heads) * d
    wo, wgu, wdn = 2 * s.n_q_heads * d * H, 2 * H * 2 * s.ffn, 2 * s.ffn * H
    kv = 2 * sum_ctx * s.n_kv_heads * d * 2
    win = (P_ + 1) * BH + H * 2 + 2 * BH
    return [win, wqkv + BH + Bq + 2 * Bkv, kv + Bq, Bq, wo + Bq + BH, win, wgu + BH + BF, wdn + BF + BH]


def max_over_ranks(ms: float, world: int, device: str = "cuda") -> float:
    """Slowest rank's time: the whole job is only as fast as its slowest replica."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    tns = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(tns, op=dist.ReduceOp.MAX)
    return float(tns.item())


def whole_job_gbs(alg_bytes_per_layer: int, layers_per_step: int, ms_per_step: float, world: int) -> float:
    """Aggregate effective bandwidth of `world` independent replicas that all take ms_per_step."""
    return alg_bytes_per_layer * layers_per_step * world / (ms_per_step * 1e-3) / 1e9


def rotation_size(shape, l2_bytes: int) -> int:
    per_layer = shape.weight_bytes() + 2 * shape.batch * shape.ctx * shape.n_kv_heads * shape.head_dim * 2
    return max(2, math.ceil(4 * l2_bytes / per_layer))


# --------------------------------------------------------------------------- ours
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2501_08192_b200 import binding as P
    from paper_2501_08192_b200 import build as B
    from paper_2501_08192_b200 import inputs as I

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    B.build()
    from dataclasses import replace
    shape = replace(I.CONFIGS[args.config], seed=I.CONFIGS[args.config].seed + 1000 * rank)
    l2 = torch.cuda.get_device_properties(local_rank).L2_cache_size
    R = args.rotation or rotation_size(shape, l2)

    def to_dev(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    rng = np.random.Generator(np.random.PCG64(shape.seed))
    layers, ios, keep, hios = [], [], [], []
    cfg = P.make_config(shape)
    for _ in range(R):
        t = I.make_layer(shape, rng, nan_fill_tail=False)
        w = {n: to_dev(t[n]) for n in ("w_q", "w_k", "w_v", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")}
        L = P.Layer(cfg, w)
        del w
        parts = [to_dev(t["partials_in"][p]) for p in range(shape.tp_degree)]
        peers = [to_dev(t["attn_peer_partials"][p]) for p in range(shape.tp_degree - 1)]
        resid = to_dev(t["residual_in"])
        kc, vc = to_dev(t["k_cache"]), to_dev(t["v_cache"])
        ctx_host = np.ascontiguousarray(t["ctx_len"], np.int32)
        ctx_dev = torch.from_numpy(ctx_host).cuda()
        r_out = torch.empty((shape.batch, shape.hidden), dtype=torch.bfloat16, device="cuda")
        m_out = torch.empty_like(r_out)
        ios.append(L.make_io(shape.batch, ctx_dev, ctx_host, parts, peers, resid, kc, vc, r_out, m_out))
        layers.append(L)
        # pinned host copies for the end-to-end arm
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
        hp = [pin(t["partials_in"][p]) for p in range(shape.tp_degree)]
        hq = [pin(t["attn_peer_partials"][p]) for p in range(shape.tp_degree - 1)]
        hr = pin(t["residual_in"])
        ho1 = torch.zeros((shape.batch, shape.hidden), dtype=torch.int16).pin_memory()
        ho2 = torch.zeros((shape.batch, shape.hidden), dtype=torch.int16).pin_memory()
        hios.append(P.make_host_io(cfg, shape.batch, ctx_host, hp, hq, hr, kc, vc, ho1, ho2))
        keep.append((t["ctx_len"], ho1, ho2))
        del t
    sum_ctx = int(sum(int(x) for x in keep[0][0]))
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    info = layers[0].get_info()
    default_budget = int(info.prefetch_budget) if args.budget_bytes < 0 else args.budget_bytes

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def set_budget(b):
        for L in layers:
            L.set_prefetch_bytes(b)

    def time_steps(step_fn, steps, warmup):
        """Mean ms per step over exactly `steps` steps (events on the launching stream), max over ranks,
        plus the per-step times of this rank."""
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                step_fn()
        barrier()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        with torch.cuda.stream(stream):
            evs[0].record(stream)
            for i in range(steps):
                step_fn()
                evs[i + 1].record(stream)
        barrier()
        total = evs[0].elapsed_time(evs[steps]) / steps
        per = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]
        return max_over_ranks(total, world), per

    def chain_step():
        P.preserve_decode_chain(layers, ios, link=False, stream=stream)

    def host_step():
        for L, h in zip(layers, hios):
            L.decode_step_host(h, stream)

    alg = int(P.preserve_algorithmic_bytes(cfg, shape.batch, sum_ctx))
    assert alg > 0

    def set_delay(ns):
        for L in layers:
            L.set_window_delay_ns(ns)

    # ---- headline: default prefetch setting, with clocks sampled during the timed region
    sampler = ClockSampler(local_rank)
    sampler.start()
    set_budget(default_budget)
    ms_on, per_on = time_steps(chain_step, args.steps, args.warmup)
    # ---- prefetch off (vanilla execution), early launch only (budget of one byte: nothing planned for
    # L2), and the sweep over the L2 budget (fewer steps each)
    set_budget(0)
    ms_off, per_off = time_steps(chain_step, args.steps, args.warmup)
    set_budget(1)
    ms_early, _ = time_steps(chain_step, max(10, args.steps // 2), 3)
    sweep = []
    if not args.no_sweep:
        for f in SWEEP_FRACS:
            set_budget(int(f * l2))
            ms, _ = time_steps(chain_step, max(10, args.steps // 4), 3)
            sweep.append({"frac_of_l2": round(f, 4), "us_per_layer": round(ms * 1e3 / R, 3)})
    # ---- modelled communication latency added to every window (the single-GPU stand-in has none)
    modelled = []
    if not args.no_sweep:
        for delay_us in (10, 20):
            set_delay(delay_us * 1000)
            row = {"window_delay_us": delay_us}
            for name, b in (("off", 0), ("early_launch_only", 1), ("on", default_budget)):
                set_budget(b)
                ms, _ = time_steps(chain_step, max(10, args.steps // 4), 3)
                row[name + "_us_per_layer"] = round(ms * 1e3 / R, 3)
            modelled.append(row)
        set_delay(0)
    # ---- end to end through the host-buffer entry point
    set_budget(default_budget)
    ms_e2e, _ = time_steps(host_step, args.steps, args.warmup)
    h2d = (2 * shape.tp_degree) * shape.batch * shape.hidden * 2 + shape.batch * 4
    d2h = 2 * shape.batch * shape.hidden * 2
    # ---- per-kernel times: each main-stream kernel alone, launched back to back over the R layer
    # instances (cold L2 by rotation) from a captured graph, CUDA events on the launching stream
    # around many replays.  Launches of one kernel are independent of each other, so this is the
    # kernel's own duration including its launch hand-over, not a dependency chain.
    kms = np.full(len(P.KERNEL_NAMES), 1e-9)
    with torch.cuda.stream(stream):
        chain_step()
        torch.cuda.synchronize()
    for k in range(len(P.KERNEL_NAMES) if not args.no_kernels else 0):
        def one():
            for L, io in zip(layers, ios):
                L.run_kernel(io, k, stream)
        with torch.cuda.stream(stream):
            one()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for _ in range(4):
                    one()
        ms, _ = time_steps(lambda: g.replay(), 10, 3)
        kms[k] = ms / (4 * R)
        del g
    status = max(L.last_status() for L in layers)
    # ---- the read roofline of this GPU, measured live: a pure 128-bit read stream over 1 GiB (HBM)
    # and over 32 MiB read repeatedly (L2)
    big = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
    read_bw = {"hbm_read_gbs": round(P.preserve_measure_read_bandwidth(big, 5, stream), 1),
               "l2_read_gbs": round(P.preserve_measure_read_bandwidth(big[: 32 << 20], 50, stream), 1)}
    del big
    clocks = sampler.summary()      # sampled from before the first timed region to after the last

    peak, peak_src = load_peaks()
    kb = kernel_bytes(shape, sum_ctx)
    dom = int(np.argmax(kms))
    achieved = kb[dom] / (kms[dom] * 1e-3) / 1e9
    gbs = lambda ms: alg * R / (ms * 1e-3) / 1e9
    us = lambda ms: ms * 1e3 / R
    best = min(sweep, key=lambda e: e["us_per_layer"]) if sweep else None
    info = layers[0].get_info()
    n_pf = sum(1 for w in range(2) if sum(info.planned_bytes[w]) > 0)
    launches_per_layer = len(P.KERNEL_NAMES) + n_pf
    out = {
        "metric": METRIC, "value": round(whole_job_gbs(alg, R, ms_on, world), 2), "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_on, 5),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 (fp32 accumulate)",
        "data": "synthetic (seeded N(0,0.02) weights, N(0,1) activations and KV, shapes of the named config)",
        "config": {"workload": f"configs[{args.config}] {shape.name}: hidden {shape.hidden}, "
                               f"{shape.n_q_heads}q/{shape.n_kv_heads}kv heads, ffn {shape.ffn}, batch {shape.batch}, "
                               f"ctx {shape.ctx}, P={shape.tp_degree}",
                   "layers_per_step": R,
                   "cold_l2": f"rotation of {R} distinct layer instances per step "
                              f"({R * (shape.weight_bytes() + 2 * sum_ctx * shape.n_kv_heads * 256) / 1e6:.0f} MB "
                              f"> 4 x L2 of {l2 / 1e6:.0f} MB); inputs larger than L2, no flush",
                   "algorithmic_bytes_per_layer": alg,
                   "prefetch_budget_bytes": default_budget, "plan_mode": "truncate",
                   "parallelism": f"{world} independent shard replica(s)"},
        "us_per_layer": round(us(ms_on), 3),
        "frac_of_nominal_8TBs": round(gbs(ms_on) / 8000.0, 4),
        "frac_of_measured_copy_bw": round(gbs(ms_on) / peak, 4),
        "prefetch": {"on_us_per_layer": round(us(ms_on), 3), "off_us_per_layer": round(us(ms_off), 3),
                     "early_launch_only_us_per_layer": round(us(ms_early), 3),
                     "on_gbs": round(gbs(ms_on), 1), "off_gbs": round(gbs(ms_off), 1),
                     "speedup_on_vs_off": round(ms_off / ms_on, 4),
                     "p10_p50_p90_on_us": [round(float(np.percentile(per_on, q)) * 1e3 / R, 3) for q in (10, 50, 90)],
                     "p10_p50_p90_off_us": [round(float(np.percentile(per_off, q)) * 1e3 / R, 3) for q in (10, 50, 90)],
                     "meaning": "off = vanilla execution (budget 0: no early launch, no side stream); "
                                "early_launch_only = consumer kernels stage operands in shared memory during "
                                "the window; on = that plus the L2 prefetch kernel at the default budget",
                     "sweep": sweep, "best": best, "modelled_window": modelled,
                     "paper_context": "up to 1.6x end to end on 8x Ascend 910B, int8 (another machine; not a target)"},
        "e2e": {"value": round(gbs(ms_e2e) * world, 2), "unit": "GB/s", "us_per_layer": round(us(ms_e2e), 3),
                "h2d_bytes_per_step": h2d * R, "d2h_bytes_per_step": d2h * R},
        "gpu_launches": launches_per_layer * R * args.steps,
        "kernels_us": {n: round(float(v) * 1e3, 3) for n, v in zip(P.KERNEL_NAMES, kms)},
        "kernels_gbs": {n: round(kb[i] / (float(kms[i]) * 1e-3) / 1e9, 1) for i, n in enumerate(P.KERNEL_NAMES)},
        "roofline": {"bound": "hbm", "kernel": P.KERNEL_NAMES[dom], "achieved": round(achieved, 1),
                     "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4),
                     "traffic": NCU_TRAFFIC.get((P.KERNEL_NAMES[dom], args.config)),
                     "traffic_note": NCU_TRAFFIC_NOTE.get((P.KERNEL_NAMES[dom], args.config)), "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": kb[dom],
                     "how": "kernel launched alone, back to back over the rotation, from a captured graph"},
        "read_bandwidth": read_bw, "frac_of_measured_read_bw": round(gbs(ms_on) / read_bw["hbm_read_gbs"], 4),
        "clocks": clocks, "device_status": status,
    }
    if rank == 0:
        if args.cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline(args.config, alg, budget_s=12.0)
        print(json.dumps(out), flush=True)
        det = os.path.join(ROOT, "gpurun_out")
        if os.path.isdir(det):
            with open(os.path.join(det, f"bench_config{args.config}_n{world}.json"), "w") as f:
                json.dump(out, f, indent=1)
    for L in layers:
        L.close()
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------- reference
def oracle_step_timer(config_idx: int):
    """Returns (fn, shape, algorithmic bytes): fn() runs the CPU oracle on one layer-step of the workload."""
    from oracle import oracle as O
    from paper_2501_08192_b200 import binding as P
    from paper_2501_08192_b200 import inputs as I
    O.build()
    shape = I.CONFIGS[config_idx]
    t = I.make_layers(shape, 1, nan_fill_tail=False)[0]
    sum_ctx = int(t["ctx_len"].sum())
    try:
        alg = int(P.preserve_algorithmic_bytes(P.make_config(shape), shape.batch, sum_ctx))
    except Exception:
        alg = shape.weight_bytes() + 2 * sum_ctx * shape.n_kv_heads * 256
    return (lambda: O.layer_step(shape, t)), shape, alg, O.num_threads()


def cpu_baseline(config_idx: int, alg: int, budget_s: float):
    fn, shape, _, threads = oracle_step_timer(config_idx)
    fn()
    t0 = time.perf_counter()
    n = 0
    while True:
        fn()
        n += 1
        if time.perf_counter() - t0 > budget_s or n >= 50:
            break
    dt = (time.perf_counter() - t0) / n
    return {"value": round(alg / dt / 1e9, 4), "unit": "GB/s", "us_per_layer": round(dt * 1e6, 1), "cores": threads,
            "kind": "oracle", "sample": f"{n} full layer-steps of configs[{config_idx}] ({shape.name}), "
                                        f"one layer instance, after one untimed run"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    fn, shape, alg, threads = oracle_step_timer(args.config)
    for _ in range(min(args.warmup, 2)):
        fn()
    steps = min(args.steps, 20)
    t0 = time.perf_counter()
    for _ in range(steps):
        fn()
    ms = (time.perf_counter() - t0) * 1e3 / steps
    val = round(alg / (ms * 1e-3) / 1e9, 4)
    sample = f"each step = one full layer-step of configs[{args.config}] ({shape.name}) on one layer instance"
    out = {"impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus,
           "steps": steps, "warmup": min(args.warmup, 2), "ms_per_step": round(ms, 3), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "fp32 values, fp64 accumulation",
           "data": "synthetic (same seeded inputs as the CUDA arm)",
           "config": {"workload": f"configs[{args.config}] {shape.name}", "layers_per_step": 1,
                      "algorithmic_bytes_per_layer": alg},
           "us_per_layer": round(ms * 1e3, 1),
           "cpu_baseline": {"value": val, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
           "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--config", type=int, default=1, help="index into the five benchmark configurations")
    ap.add_argument("--rotation", type=int, default=0, help="layer instances per step (0 = sized from L2)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-kernels", action="store_true", help="skip the isolated per-kernel timing")
    ap.add_argument("--budget-bytes", type=int, default=-1, help="prefetch budget per window (default: the library's)")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
