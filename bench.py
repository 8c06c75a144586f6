#!/usr/bin/env python
"""Benchmark of the decode-layer hot path (one tensor-parallel shard's decode step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config I]
    python bench.py --mode timeline --config I      per-kernel timeline of one layer-step
    python bench.py --mode decode-loop              32-layer chain, contexts advancing every token
    python bench.py --mode streams                  L2 / HBM streaming-read microbenchmark table

Metric: decode-layer us/step and effective HBM GB/s (weights + KV + activation bytes over
time), prefetch on vs off.  A "step" is one pass of the whole hot path over a rotation of R
distinct layer instances of the workload (distinct weight arenas and KV-caches, R x (weights +
KV) >= 4 x L2), so every layer-step starts with a cold L2; per-layer figures are the step's
divided by R.  Without --config all five benchmark configurations run in one invocation: the
top-level `value` / `config` / `roofline` are those of the largest single-GPU one (configs[3]:
70B-shaped TP=4 shard, batch 64, ragged contexts), `per_config` carries all five.
`value` is the effective GB/s with the library's default prefetch setting and inputs resident in
HBM; `e2e` is the same metric through the host-buffer entry point with host<->device copies
inside the timed region.  With --gpus N each rank runs an independent shard replica (no
data-path collective; weak scaling); started without a launcher, bench.py spawns the N ranks
itself.  The reference arm times the CPU oracle on the host cores.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import socket
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
HEADLINE_CONFIG = 3          # the largest single-GPU configuration
MIN_LAYER_STEPS = 200        # timed layer-steps per setting, whatever --steps says

# DRAM traffic per launch of a kernel from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum),
# keyed by (kernel, config index): (bytes, the profiles/ file the figure was read from).
NCU_TRAFFIC = {
    ("gate_up_proj", 1): (44220000, "profiles/ncu_full_gemv_attn_window_config1_small.md (includes 14.68 MB of the "
                                    "down projection's weights that this kernel's CTAs prefetch into L2)"),
    ("gate_up_proj", 2): (121910000, "profiles/ncu_full_gemm_tcgen05_config3_small.md"),
    ("attn_splitkv", 4): (542870000, "profiles/ncu_full_attn_splitkv_config5.md"),
    ("gate_up_proj", 3): (240296448, "profiles/ncu_full_gemm_tcgen05_gate_up_config4.md (read 236.03 MB + write 4.27 MB, "
                                     "full-size launch, 2-layer rotation)"),
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy bandwidth)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed regions run."""

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
    """Algorithmic bytes per launch of each main-stream kernel (order: window A, QKV, split-KV
    attention, merge, O, window B, gate/up, down).  Their sum is the layer-step's algorithmic bytes."""
    B, H, d, P_ = s.batch, s.hidden, s.head_dim, s.tp_degree
    BH, Bq, Bkv, BF = B * H * 2, B * s.n_q_heads * d * 2, B * s.n_kv_heads * d * 2, B * s.ffn * 2
    wqkv = 2 * H * (s.n_q_heads + 2 * s.n_kv_heads) * d
    wo, wgu, wdn = 2 * s.n_q_heads * d * H, 2 * H * 2 * s.ffn, 2 * s.ffn * H
    kv = 2 * sum_ctx * s.n_kv_heads * d * 2
    win = (P_ + 1) * BH + H * 2 + 2 * BH
    return [win, wqkv + BH + Bq + 2 * Bkv, kv + Bq, Bq, wo + Bq + BH, win, wgu + BH + BF, wdn + BF + BH]


def algorithmic_bytes(s, sum_ctx: int) -> int:
    return int(sum(kernel_bytes(s, sum_ctx)))


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


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def spawn_command(n_ranks: int, port: int, argv):
    """The launcher command that starts `n_ranks` ranks of this script on one node."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def spawn_ranks(args, argv) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks here, one per GPU."""
    return subprocess.call(spawn_command(args.gpus, free_port(), argv))


# --------------------------------------------------------------------------- ours
class Workload:
    """R layer instances of one configuration on the device, plus pinned host copies of the step
    inputs for the end-to-end arm.  Instance 0 holds the configuration's seeded draw; the other
    instances are distinct device buffers with the same bit patterns (the kernels' timing does not
    depend on the values; what the rotation needs is distinct addresses)."""

    def __init__(self, P, I, torch, idx: int, rank: int, l2: int, rotation: int = 0, keep_host: bool = False,
                 flags: int = 0):
        from dataclasses import replace
        base = I.CONFIGS[idx]
        self.shape = shape = replace(base, seed=base.seed + 1000 * rank)
        self.R = R = rotation or rotation_size(shape, l2)
        self.cfg = cfg = P.make_config(shape, flags=flags)
        rng = np.random.Generator(np.random.PCG64(shape.seed))
        t = I.make_layer(shape, rng, nan_fill_tail=False)

        def to_dev(bits):
            return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

        def pin(a):
            return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()

        w = {n: to_dev(t[n]) for n in ("w_q", "w_k", "w_v", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")}
        parts0 = [to_dev(t["partials_in"][p]) for p in range(shape.tp_degree)]
        peers0 = [to_dev(t["attn_peer_partials"][p]) for p in range(shape.tp_degree - 1)]
        self.ctx_host = np.ascontiguousarray(t["ctx_len"], np.int32)
        if flags & P.FLAG_INT8_KV:
            # int8 cache: one device buffer per tensor in the library's layout (codes, then scales)
            kv = I.make_int8_cache(shape, self.ctx_host)
            off, scap, total = P.preserve_kv8_layout(cfg)

            def kv8_buf(codes, scales):
                buf = torch.zeros(total, dtype=torch.uint8, device="cuda")
                buf[:codes.size] = torch.from_numpy(codes.view(np.uint8).reshape(-1)).cuda()
                padded = np.zeros(scales.shape[:2] + (scap,), np.float32)
                padded[:, :, :scales.shape[2]] = np.nan_to_num(scales)
                buf[off:off + padded.size * 4] = torch.from_numpy(padded.view(np.uint8).reshape(-1)).cuda()
                return buf
            kc0, vc0 = kv8_buf(kv["k_codes"], kv["k_scales"]), kv8_buf(kv["v_codes"], kv["v_scales"])
            del kv
        else:
            kc0, vc0 = to_dev(t["k_cache"]), to_dev(t["v_cache"])
        resid0 = to_dev(t["residual_in"])
        self.sum_ctx = int(self.ctx_host.sum())
        hp = [pin(t["partials_in"][p]) for p in range(shape.tp_degree)]
        hq = [pin(t["attn_peer_partials"][p]) for p in range(shape.tp_degree - 1)]
        hr = pin(t["residual_in"])
        self.layers, self.ios, self.hios, self.keep = [], [], [], []
        for i in range(R):
            L = P.Layer(cfg, w)
            c = (lambda x: x) if i == 0 else (lambda x: x.clone())
            parts, peers = [c(x) for x in parts0], [c(x) for x in peers0]
            resid, kc, vc = c(resid0), c(kc0), c(vc0)
            ctx_dev = torch.from_numpy(self.ctx_host).cuda()
            r_out = torch.empty((shape.batch, shape.hidden), dtype=torch.bfloat16, device="cuda")
            m_out = torch.empty_like(r_out)
            self.ios.append(L.make_io(shape.batch, ctx_dev, self.ctx_host, parts, peers, resid, kc, vc, r_out, m_out))
            self.layers.append(L)
            ho1 = torch.zeros((shape.batch, shape.hidden), dtype=torch.int16).pin_memory()
            ho2 = torch.zeros((shape.batch, shape.hidden), dtype=torch.int16).pin_memory()
            self.hios.append(P.make_host_io(cfg, shape.batch, self.ctx_host, hp, hq, hr, kc, vc, ho1, ho2))
            self.keep.append((ho1, ho2))
        del w
        self.host_tensors = t if keep_host else None
        self.alg = algorithmic_bytes(shape, self.sum_ctx)
        torch.cuda.synchronize()

    def set_budget(self, b):
        for L in self.layers:
            L.set_prefetch_bytes(b)

    def set_delay(self, ns):
        for L in self.layers:
            L.set_window_delay_ns(ns)

    def close(self):
        for L in self.layers:
            L.close()
        self.layers, self.ios, self.hios, self.keep = [], [], [], []


def bench_config(P, I, torch, dist, args, idx, rank, local_rank, world, stream, headline: bool):
    l2 = torch.cuda.get_device_properties(local_rank).L2_cache_size
    vflags = (P.FLAG_INT8_KV if args.int8_kv else 0) | (P.FLAG_INT8_WEIGHTS if args.int8_weights else 0)
    wl = Workload(P, I, torch, idx, rank, l2, args.rotation, keep_host=headline and rank == 0, flags=vflags)
    shape, R, alg = wl.shape, wl.R, wl.alg
    layers, ios, hios = wl.layers, wl.ios, wl.hios
    if vflags:      # (a profiling aid: the whole run at the int8 precisions; the byte count is the library's)
        alg = int(P.preserve_algorithmic_bytes(wl.cfg, shape.batch, wl.sum_ctx))
    assert alg == int(P.preserve_algorithmic_bytes(wl.cfg, shape.batch, wl.sum_ctx)) > 0
    info = layers[0].get_info()
    default_budget = int(info.prefetch_budget) if args.budget_bytes < 0 else args.budget_bytes

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def time_steps(step_fn, steps, warmup):
        """Mean ms per step over exactly `steps` steps (events on the launching stream), max over
        ranks, plus this rank's per-step times."""
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

    n_min = max(3, math.ceil(args.min_layer_steps / R))     # chain steps that make up >= 200 layer-steps
    n_short = max(3, math.ceil(args.min_layer_steps / 2 / R))
    us = lambda ms: ms * 1e3 / R
    gbs = lambda ms: alg * R / (ms * 1e-3) / 1e9
    pct = lambda per: [round(float(np.percentile(per, q)) * 1e3 / R, 3) for q in (10, 50, 90)]
    peak, peak_src = load_peaks()

    # ---- default prefetch setting ("on"): exactly --steps steps after --warmup warm-up steps
    wl.set_budget(default_budget)
    ms_on, per_on = time_steps(chain_step, args.steps, args.warmup)
    if args.steps < n_min:
        _, per_on = time_steps(chain_step, n_min, 3)
    # ---- prefetch off (vanilla execution) and early launch only (a budget of one byte plans nothing for L2)
    wl.set_budget(0)
    ms_off, per_off = time_steps(chain_step, n_min, 3)
    wl.set_budget(1)
    ms_early, per_early = time_steps(chain_step, n_min, 3)
    wl.set_budget(l2 // 16)
    ms_l2, per_l2 = time_steps(chain_step, n_min, 3)
    sweep, modelled = [], []
    if not args.no_sweep:
        for f in SWEEP_FRACS:
            wl.set_budget(int(f * l2))
            ms, _ = time_steps(chain_step, n_short, 3)
            sweep.append({"frac_of_l2": round(f, 4), "us_per_layer": round(us(ms), 3)})
        # modelled communication latency added to every window (the single-GPU stand-in has none)
        for delay_us in (10, 20, 40):
            wl.set_delay(delay_us * 1000)
            row = {"window_delay_us": delay_us}
            for name, b in (("off", 0), ("early_launch_only", 1), ("on_sixteenth_l2", l2 // 16), ("on_quarter_l2", l2 // 4),
                            ("on_half_l2", l2 // 2)):
                wl.set_budget(b)
                ms, _ = time_steps(chain_step, n_short, 3)
                row[name + "_us_per_layer"] = round(us(ms), 3)
            modelled.append(row)
        wl.set_delay(0)
    # ---- end to end through the host-buffer entry point
    wl.set_budget(default_budget)
    ms_e2e, _ = time_steps(host_step, n_min, 3)
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
        ms, _ = time_steps(lambda: g.replay(), max(5, math.ceil(args.min_layer_steps / (4 * R))), 3)
        kms[k] = ms / (4 * R)
        del g
    status = max(L.last_status() for L in layers)
    info = layers[0].get_info()
    n_pf = sum(1 for w in range(2) if sum(info.planned_bytes[w]) > 0)

    kb = kernel_bytes(shape, wl.sum_ctx)
    dom = int(np.argmax(kms))
    achieved = kb[dom] / (kms[dom] * 1e-3) / 1e9
    best = min(sweep, key=lambda e: e["us_per_layer"]) if sweep else None
    traffic = NCU_TRAFFIC.get((P.KERNEL_NAMES[dom], idx))
    res = {
        "config_index": idx, "name": shape.name,
        "workload": f"configs[{idx}] {shape.name}: hidden {shape.hidden}, {shape.n_q_heads}q/{shape.n_kv_heads}kv heads, "
                    f"ffn {shape.ffn}, batch {shape.batch}, ctx "
                    f"{'U[%d,%d]' % (shape.ctx_min, shape.ctx) if shape.ctx_min is not None else shape.ctx}, "
                    f"P={shape.tp_degree}",
        "layers_per_step": R, "algorithmic_bytes_per_layer": alg,
        "cold_l2": f"rotation of {R} distinct layer instances per step "
                   f"({R * (shape.weight_bytes() + 2 * wl.sum_ctx * shape.n_kv_heads * 256) / 1e6:.0f} MB "
                   f"> 4 x L2 of {l2 / 1e6:.0f} MB); inputs larger than L2, no flush",
        "prefetch_budget_bytes": default_budget, "plan_mode": "truncate",
        "timed_layer_steps_per_setting": n_min * R,
        "ms_per_step": round(ms_on, 5), "steps": args.steps,
        "us_per_layer": round(us(ms_on), 3), "gbs": round(gbs(ms_on), 1),
        "frac_of_measured_copy_bw": round(gbs(ms_on) / peak, 4), "frac_of_nominal_8TBs": round(gbs(ms_on) / 8000.0, 4),
        "prefetch": {
            "on_us_per_layer": round(us(ms_on), 3), "off_us_per_layer": round(us(ms_off), 3),
            "early_launch_only_us_per_layer": round(us(ms_early), 3),
            "on_gbs": round(gbs(ms_on), 1), "off_gbs": round(gbs(ms_off), 1), "early_gbs": round(gbs(ms_early), 1),
            "l2_sixteenth_us_per_layer": round(us(ms_l2), 3), "l2_sixteenth_gbs": round(gbs(ms_l2), 1),
            "speedup_on_vs_off": round(ms_off / ms_on, 4), "speedup_on_vs_early": round(ms_early / ms_on, 4),
            "speedup_early_vs_off": round(ms_off / ms_early, 4),
            "speedup_l2_sixteenth_vs_early": round(ms_early / ms_l2, 4),
            "p10_p50_p90_l2_sixteenth_us": pct(per_l2),
            "p10_p50_p90_on_us": pct(per_on), "p10_p50_p90_off_us": pct(per_off), "p10_p50_p90_early_us": pct(per_early),
            "sweep": sweep, "best": best, "modelled_window": modelled},
        "e2e": {"value": round(gbs(ms_e2e) * world, 2), "unit": "GB/s", "us_per_layer": round(us(ms_e2e), 3),
                "h2d_bytes_per_step": h2d * R, "d2h_bytes_per_step": d2h * R},
        "gpu_launches": (len(P.KERNEL_NAMES) + n_pf) * R * args.steps,
        "kernels_us": {n: round(float(v) * 1e3, 3) for n, v in zip(P.KERNEL_NAMES, kms)},
        "kernels_gbs": {n: round(kb[i] / (float(kms[i]) * 1e-3) / 1e9, 1) for i, n in enumerate(P.KERNEL_NAMES)},
        "kernels_frac_of_measured": {n: round(kb[i] / (float(kms[i]) * 1e-3) / 1e9 / peak, 3)
                                     for i, n in enumerate(P.KERNEL_NAMES)},
        "roofline": {"bound": "hbm", "kernel": P.KERNEL_NAMES[dom], "achieved": round(achieved, 1), "peak": peak,
                     "unit": "GB/s", "frac": round(achieved / peak, 4),
                     "traffic": traffic[0] if traffic else None,
                     "traffic_source": traffic[1] if traffic else None, "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": kb[dom],
                     "how": "kernel launched alone, back to back over the rotation, from a captured graph"},
        "device_status": status,
    }
    # ---- the analytical model (Section 5's linear compute / memory / communication terms, with this
    # GPU's measured bandwidths and per-kernel fixed cost) beside the measurements
    try:
        from paper_2501_08192_b200 import perf_model as M
        # per-kernel fixed costs calibrated from the kernels timed alone (attention = split-KV + merge);
        # early launch hides the hand-over between kernels, measured as (off - early) / kernels
        hw = M.b200_measured(l2_bytes=l2, kernel_overhead_us=0.0,
                             early_hides_us=max((ms_off - ms_early) * 1e3 / R / 6, 0.0))
        ops = M.layer_ops(shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn, shape.batch,
                          wl.sum_ctx)
        meas = [kms[0], kms[1], kms[2] + kms[3], kms[4], kms[5], kms[6], kms[7]]
        # (the kernels were timed alone WITH early launch, so the hidden hand-over is added back: the
        # model's "early" then reproduces the sum of the kernels, its "off" adds the hand-overs)
        ops = M.calibrate_overheads(hw, ops, [float(v) * 1e-3 + hw.early_launch_hides for v in meas])
        win = max(float(kms[0] + kms[5]) / 2 * 1e-3, 0.5e-6)                # measured stand-in window, seconds
        us_ = lambda x: round(x * 1e6, 2)
        m0 = M.predict(hw, ops, budget=l2 // 16, truncate=True, window_time=win)
        model = {"parameters": {"hbm_gbs": hw.hbm_bw / 1e9, "l2_gbs": hw.l2_bw / 1e9,
                                "fixed_cost_us_per_kernel": {o.name: us_(o.overhead) for o in ops if o.kind != "comm"},
                                "early_launch_hides_us_per_kernel": round(hw.early_launch_hides * 1e6, 2),
                                "window_us": us_(win)},
                 "note": "calibrated on the kernels timed alone and on (off - early); the budget and window rows are "
                         "predictions of what moving bytes into L2 during a window is worth at the measured bandwidths",
                 "off_us": us_(m0["off"]), "early_launch_only_us": us_(m0["early_launch_only"]),
                 "l2_sixteenth_us": us_(m0["on"]),
                 "sweep": [{"frac_of_l2": round(f, 4),
                            "us_per_layer": us_(M.predict(hw, ops, budget=max(int(f * l2), 1), truncate=True,
                                                          window_time=win)["on"])} for f in SWEEP_FRACS[1:]],
                 "modelled_window": [{"window_delay_us": d_,
                                      "early_launch_only_us": us_(M.predict(hw, ops, budget=1, truncate=True,
                                                                            window_time=win + d_ * 1e-6)["on"]),
                                      "on_quarter_l2_us": us_(M.predict(hw, ops, budget=l2 // 4, truncate=True,
                                                                        window_time=win + d_ * 1e-6)["on"])}
                                     for d_ in (10, 20, 40)]}
        res["model"] = model
    except Exception as e:      # noqa: BLE001
        res["model"] = {"error": str(e)}
    # ---- the same configuration at the precisions of the paper's runs (Section 4: int8 weights and
    # KV-cache): int8 KV-cache, int8 weights, and both.  Each row: vanilla and early-launch-only times,
    # and (int8 cache) the attention kernel alone.
    if not args.no_sweep:
        wl.close()
        variants = [("int8_kv", P.FLAG_INT8_KV), ("int8_weights", P.FLAG_INT8_WEIGHTS),
                    ("int8_weights_and_kv", P.FLAG_INT8_WEIGHTS | P.FLAG_INT8_KV)]
        for vname, vflags in variants:
            wl8 = Workload(P, I, torch, idx, rank, l2, args.rotation, flags=vflags)
            alg8 = int(P.preserve_algorithmic_bytes(wl8.cfg, shape.batch, wl8.sum_ctx))

            def chain8():
                P.preserve_decode_chain(wl8.layers, wl8.ios, link=False, stream=stream)

            def attn8():
                for L, io in zip(wl8.layers, wl8.ios):
                    L.run_kernel(io, 2, stream)
            row = {"algorithmic_bytes_per_layer": alg8}
            for name, b in (("off", 0), ("early_launch_only", 1)):
                wl8.set_budget(b)
                ms8, _ = time_steps(chain8, n_min, 3)
                row[name + "_us_per_layer"] = round(ms8 * 1e3 / wl8.R, 3)
                row[name + "_gbs"] = round(alg8 * wl8.R / (ms8 * 1e-3) / 1e9, 1)
            row["speedup_vs_bf16"] = round(us(ms_early) / row["early_launch_only_us_per_layer"], 4)
            row["speedup_early_vs_off"] = round(row["off_us_per_layer"] / row["early_launch_only_us_per_layer"], 4)
            if vflags & P.FLAG_INT8_KV:
                with torch.cuda.stream(stream):
                    attn8()
                    torch.cuda.synchronize()
                    g8 = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g8, stream=stream):
                        for _ in range(4):
                            attn8()
                ms_a, _ = time_steps(lambda: g8.replay(), max(5, math.ceil(args.min_layer_steps / (4 * wl8.R))), 3)
                ms_a /= 4 * wl8.R
                del g8
                kv_read = 2 * wl8.sum_ctx * shape.n_kv_heads * (shape.head_dim + 4)
                qo = 2 * shape.batch * shape.n_q_heads * shape.head_dim * 4
                row["attn_splitkv_us"] = round(ms_a * 1e3, 3)
                row["attn_splitkv_gbs"] = round((kv_read + qo) / (ms_a * 1e-3) / 1e9, 1)
                row["attn_splitkv_frac_of_measured"] = round(row["attn_splitkv_gbs"] / peak, 3)
            row["device_status"] = max(L.last_status() for L in wl8.layers)
            res[vname] = row
            wl8.close()
            del wl8
            torch.cuda.empty_cache()
    if headline and rank == 0 and args.cpu_baseline and world == 1:
        res["cpu_baseline"] = cpu_baseline(shape, wl.host_tensors, alg, budget_s=12.0, idx=idx)
    wl.close()
    del wl
    torch.cuda.empty_cache()
    return res


def measure_streams(P, torch, stream, quick: bool = True):
    """Single-launch streaming reads: L2-resident sizes and 1 GiB (HBM), by plain loads and by bulk
    copies into shared memory, at one and two CTAs per SM, and what one SM alone takes in."""
    sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    big = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
    big.zero_()
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    rows = []
    sizes = [(32 << 20, "l2")] if quick else [(s << 20, "l2") for s in (8, 16, 32, 64, 96)]
    sizes.append((1 << 30, "hbm"))
    for nbytes, kind in sizes:
        target = 8 << 30 if kind == "l2" else 4 << 30          # bytes moved per measurement
        passes = max(2, target // nbytes)
        for path, pname in ((0, "ld.global.nc"), (1, "cp.async.bulk")):
            for per_sm in (1, 2):
                g = P.preserve_measure_stream(big, nbytes, passes, path, sms * per_sm, 6, 16384, status, stream)
                rows.append({"buffer_mib": nbytes >> 20, "source": kind, "path": pname, "ctas_per_sm": per_sm,
                             "gbs": round(g, 1), "gbs_per_sm": round(g / sms, 2)})
    # one SM alone: a 256 KiB slice read over and over (L2), and 256 MiB read once (HBM)
    for slice_bytes, passes, kind in ((256 << 10, 1024, "l2"), (256 << 20, 1, "hbm")):
        for path, pname in ((0, "ld.global.nc"), (1, "cp.async.bulk")):
            for stages in ((6, 12) if path == 1 else (0,)):
                g = P.preserve_measure_stream(big, slice_bytes, passes, path, 1, stages or 6, 16384, status, stream)
                rows.append({"buffer_mib": round(slice_bytes / (1 << 20), 2), "source": kind + " (one CTA on one SM)",
                             "path": pname + (f" x{stages} stages" if path == 1 else ""), "ctas_per_sm": None,
                             "gbs": round(g, 1), "gbs_per_sm": round(g, 2)})
    if not quick:
        # what limits one CTA: bytes per copy and issuing threads per CTA (L2-resident 32 MiB and HBM)
        for nbytes, kind in ((32 << 20, "l2"), (1 << 30, "hbm")):
            passes = max(2, ((8 << 30) if kind == "l2" else (4 << 30)) // nbytes)
            for chunk, stages, producers in ((4096, 12, 1), (8192, 12, 1), (32768, 6, 1), (65536, 3, 1),
                                             (16384, 6, 2), (16384, 3, 4), (8192, 3, 8), (2048, 8, 8)):
                for per_sm in (1, 2):
                    if per_sm * stages * chunk * producers > 200 * 1024:
                        continue
                    g = P.preserve_measure_stream(big, nbytes, passes, 1, sms * per_sm, stages, chunk, status, stream,
                                                  producers)
                    rows.append({"buffer_mib": nbytes >> 20, "source": kind,
                                 "path": f"cp.async.bulk {chunk} B x{stages} stages x{producers} threads",
                                 "ctas_per_sm": per_sm, "gbs": round(g, 1), "gbs_per_sm": round(g / sms, 2)})
            # issuing threads that are lanes of ONE warp
            for chunk, stages, producers in ((16384, 3, 4), (8192, 3, 8)):
                g = P.preserve_measure_stream(big, nbytes, passes, 2, sms, stages, chunk, status, stream, producers)
                rows.append({"buffer_mib": nbytes >> 20, "source": kind,
                             "path": f"cp.async.bulk {chunk} B x{stages} stages x{producers} lanes of one warp",
                             "ctas_per_sm": 1, "gbs": round(g, 1), "gbs_per_sm": round(g / sms, 2)})
        # the tcgen05 GEMM's kind of load: 2-D tiled TMA boxes of 64 columns x 128 / 256 rows
        for nbytes, kind in ((32 << 20, "l2"), (1 << 30, "hbm")):
            passes = 40 if kind == "l2" else 2
            for box_rows, stages, producers in ((256, 4, 1), (256, 2, 3), (128, 6, 1), (128, 4, 3)):
                for per_sm in (1, 2):
                    if per_sm * stages * box_rows * 128 * producers > 200 * 1024:
                        continue
                    g = P.preserve_measure_stream_tma(big, nbytes, passes, sms * per_sm, stages, box_rows, producers,
                                                      status, stream)
                    rows.append({"buffer_mib": nbytes >> 20, "source": kind,
                                 "path": f"TMA 2-D box 64 x {box_rows} ({box_rows * 128} B) x{stages} stages x{producers} threads",
                                 "ctas_per_sm": per_sm, "gbs": round(g, 1), "gbs_per_sm": round(g / sms, 2)})
    assert int(status[0].item()) == 0
    del big
    return rows


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2501_08192_b200 import build as B

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.dry_run:
        # launch plumbing only (CPU, gloo): no kernel runs, nothing is timed
        if world > 1:
            dist.init_process_group("gloo")
        ms = max_over_ranks(1.0 + 0.25 * rank, world, device="cpu")
        if rank == 0:
            print(json.dumps({"metric": METRIC, "dry_run": True, "n_gpus": world, "ms_per_step": ms,
                              "value": None, "scaling": "weak"}), flush=True)
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    B.build()
    from paper_2501_08192_b200 import binding as P
    from paper_2501_08192_b200 import inputs as I
    stream = torch.cuda.Stream()

    if args.mode == "timeline":
        run_timeline(P, I, torch, args, stream)
        return
    if args.mode == "decode-loop":
        run_decode_loop(P, I, torch, args, stream)
        return
    if args.mode == "real-window":
        # the multi-GPU measurement alone (with one rank: a one-member group, which still runs every
        # code path of it - exchange blocks, fused window, library all-reduce - on one GPU)
        if world == 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", str(free_port()))
            dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", local_rank))
        out = bench_real_window(P, I, torch, dist, args, rank, local_rank, world, stream)
        if rank == 0:
            print(json.dumps({"mode": "real-window", "n_gpus": world, "real_window": out}), flush=True)
        dist.destroy_process_group()
        return
    if args.mode == "streams":
        rows = measure_streams(P, torch, stream, quick=False)
        print(json.dumps({"streams": rows}), flush=True)
        return

    configs = [args.config] if args.config >= 0 else list(range(len(I.CONFIGS)))
    head = args.config if args.config >= 0 else HEADLINE_CONFIG
    sampler = ClockSampler(local_rank)
    sampler.start()
    # the headline configuration first (its timed region is the one --steps / --warmup describe)
    order = [head] + [c for c in configs if c != head]
    per = {}
    for idx in order:
        per[idx] = bench_config(P, I, torch, dist, args, idx, rank, local_rank, world, stream, headline=idx == head)
    streams = measure_streams(P, torch, stream, quick=True) if not args.no_kernels else []
    clocks = sampler.summary()      # sampled from before the first timed region to after the last

    h = per[head]
    read_bw = {}
    for r in streams:
        if r["ctas_per_sm"] == 2 and r["path"] == "ld.global.nc":
            read_bw["hbm_read_gbs" if r["source"] == "hbm" else "l2_read_gbs"] = r["gbs"]
        if r["ctas_per_sm"] == 2 and r["path"] == "cp.async.bulk":
            read_bw["hbm_bulk_gbs" if r["source"] == "hbm" else "l2_bulk_gbs"] = r["gbs"]
    out = {
        "metric": METRIC, "value": round(whole_job_gbs(h["algorithmic_bytes_per_layer"], h["layers_per_step"],
                                                       h["ms_per_step"], world), 2),
        "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": h["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 (fp32 accumulate)" + (", int8 KV-cache" if args.int8_kv else "") + (", int8 weights" if args.int8_weights else ""),
        "data": "synthetic (seeded N(0,0.02) weights, N(0,1) activations and KV, shapes of the named config; the "
                "layer instances of a rotation are distinct device buffers holding the same seeded draw)",
        "config": {"workload": h["workload"], "layers_per_step": h["layers_per_step"], "cold_l2": h["cold_l2"],
                   "algorithmic_bytes_per_layer": h["algorithmic_bytes_per_layer"],
                   "prefetch_budget_bytes": h["prefetch_budget_bytes"], "plan_mode": h["plan_mode"],
                   "parallelism": f"{world} independent shard replica(s)"},
        "us_per_layer": h["us_per_layer"], "frac_of_nominal_8TBs": h["frac_of_nominal_8TBs"],
        "frac_of_measured_copy_bw": h["frac_of_measured_copy_bw"],
        "prefetch": dict(h["prefetch"], meaning="off = vanilla execution (budget 0: no early launch, no side stream); "
                         "early_launch_only = the consumer kernels are launched early and stage their leading operand "
                         "bytes in shared memory during the window (budget of one byte: nothing planned for L2); on = "
                         "the library's default, which is early launch only (the fastest measured setting with the "
                         "bare stand-in windows); l2_sixteenth = early launch plus the side-stream L2 prefetch kernel "
                         "with a budget of L2/16 per window.  speedup_on_vs_off is the gain of early launch with "
                         "shared-memory staging; speedup_l2_sixteenth_vs_early is what the L2 prefetch kernel adds "
                         "(below 1: it costs); modelled_window shows where it starts to pay",
                         paper_context="up to 1.6x end to end on 8x Ascend 910B, int8 (another machine; not a target)"),
        "e2e": h["e2e"], "gpu_launches": h["gpu_launches"],
        "kernels_us": h["kernels_us"], "kernels_gbs": h["kernels_gbs"], "roofline": h["roofline"],
        "read_bandwidth": read_bw, "streams": streams, "clocks": clocks, "device_status": h["device_status"],
        "per_config": [per[i] for i in sorted(per)],
    }
    if "cpu_baseline" in h:
        out["cpu_baseline"] = h.pop("cpu_baseline")
    if world > 1 and not args.no_real_window:
        try:
            out["real_window"] = bench_real_window(P, I, torch, dist, args, rank, local_rank, world, stream)
        except Exception as e:      # noqa: BLE001  (the replicas' result above must survive)
            out["real_window"] = {"error": f"{type(e).__name__}: {e}"}
    if rank == 0:
        print(json.dumps(out), flush=True)
        det = os.path.join(ROOT, "gpurun_out")
        if os.path.isdir(det):
            with open(os.path.join(det, f"bench_n{world}.json"), "w") as f:
                json.dump(out, f, indent=1)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------ other modes
def bench_real_window(P, I, torch, dist, args, rank, local_rank, world, stream):
    """N > 1: the communication window for real.  The ranks are the `world` shards of a
    configs[1]-shaped layer (tp_degree = world) chained over a rotation of R layers; per layer-step
    time with (a) the fused one-shot all-reduce window (peer reads in the window kernel), (b) the
    library-collective baseline (NCCL all-reduce + a one-buffer window, kernels queued one by one)
    and (c) the local stand-in, each with prefetch off / early launch only / on.  Every phase is
    agreed on over a gloo control group first, so a rank that fails makes all ranks skip, not hang."""
    from dataclasses import replace
    from datetime import timedelta
    from paper_2501_08192_b200 import comm as CM
    ctrl = dist.new_group(backend="gloo", timeout=timedelta(seconds=120))

    def all_ok(ok: bool) -> bool:
        t = torch.tensor([1 if ok else 0], dtype=torch.int32)
        dist.all_reduce(t, op=dist.ReduceOp.MIN, group=ctrl)
        return bool(t.item())

    res, err = {}, None
    l2 = torch.cuda.get_device_properties(local_rank).L2_cache_size
    base = replace(I.CONFIGS[1], tp_degree=world, seed=I.CONFIGS[1].seed + 1000 * rank)
    wl = wl1 = comm = None
    try:
        R = rotation_size(base, l2)
        # (Workload indexes I.CONFIGS: build from a patched copy of configs[1])
        saved = I.CONFIGS
        I.CONFIGS = tuple(replace(c, tp_degree=world) if i == 1 else c for i, c in enumerate(saved))
        try:
            wl = Workload(P, I, torch, 1, rank, l2, R)
            I.CONFIGS = tuple(replace(c, tp_degree=1) if i == 1 else c for i, c in enumerate(saved))
            wl1 = Workload(P, I, torch, 1, rank, l2, R)
        finally:
            I.CONFIGS = saved
        shape = wl.shape
        comm = P.Comm(rank, world, shape.batch, shape.hidden)
        handles = [None] * world
        dist.all_gather_object(handles, (rank, comm.export_handle()), group=ctrl)
        for r, h in handles:
            if r != rank:
                comm.import_handle(r, h)
        comm.write(0, wl.ios[0]._keep[4][0])          # the first window A reads the exchange buffers
        torch.cuda.synchronize()
    except Exception as e:      # noqa: BLE001
        err = f"setup: {type(e).__name__}: {e}"
    if not all_ok(err is None):
        return {"skipped": err or "another rank failed during setup"}

    def timed(step_fn, steps):
        with torch.cuda.stream(stream):
            for _ in range(3):
                step_fn()
        torch.cuda.synchronize()
        dist.barrier(group=ctrl)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(steps):
                step_fn()
            e1.record(stream)
        torch.cuda.synchronize()
        dist.barrier(group=ctrl)
        t = torch.tensor([e0.elapsed_time(e1) / steps], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=ctrl)
        return float(t.item())

    steps = max(3, math.ceil(MIN_LAYER_STEPS / wl.R))
    default_budget = int(wl.layers[0].get_info().prefetch_budget)
    settings = (("off", 0), ("early_launch_only", 1), ("on_l2_sixteenth", l2 // 16), ("on_l2_quarter", l2 // 4))

    def fused_step():
        P.preserve_decode_chain(wl.layers, wl.ios, link=False, stream=stream)

    def standin_step():
        P.preserve_decode_chain(wl.layers, wl.ios, link=False, stream=stream)

    nccl_bufs = []

    def nccl_step():
        # the prefetch operator goes right before the collective it runs beside (Algorithm 1)
        for L, io, (mlp_sum, attn_sum) in zip(wl1.layers, wl1.ios, nccl_bufs):
            L.prefetch_window(io, 0, stream)
            dist.all_reduce(mlp_sum)
            for k in range(5):
                L.run_kernel(io, k, stream)
            L.prefetch_window(io, 1, stream)
            dist.all_reduce(attn_sum)
            for k in range(5, 8):
                L.run_kernel(io, k, stream)

    try:
        # (c) the local stand-in first (no communication at all)
        row = {}
        for name, b in settings:
            wl.set_budget(b)
            row[name + "_us_per_layer"] = round(timed(standin_step, steps) * 1e3 / wl.R, 3)
        res["local_stand_in"] = row
        # (a) fused peer-read window
        for L in wl.layers:
            L.set_comm(comm)
        row = {}
        for name, b in settings:
            wl.set_budget(b)
            row[name + "_us_per_layer"] = round(timed(fused_step, steps) * 1e3 / wl.R, 3)
        # measured length of the real window (wait return to end of the window kernels, traced)
        for L in wl.layers:
            L.set_trace(True)
        wl.set_budget(1)
        with torch.cuda.stream(stream):
            fused_step()
        torch.cuda.synchronize()
        tr = [L.read_trace() for L in wl.layers[1:]]
        row["window_a_us"] = round(float(np.mean([t_[0][3] - t_[0][2] for t_ in tr])) / 1e3, 2)
        row["window_b_us"] = round(float(np.mean([t_[5][3] - t_[5][2] for t_ in tr])) / 1e3, 2)
        for L in wl.layers:
            L.set_trace(False)
        row["device_status_code"] = max(L.last_status_code() for L in wl.layers)
        res["fused_peer_read_window"] = row
        for L in wl.layers:
            L.set_comm(None)
        # (b) NCCL all-reduce + one-buffer window: layer j's window A reads the all-reduced MLP partial
        # sums of the layer before it in the rotation (reduced in place in that layer's output buffer),
        # its window B the all-reduced attention partial sums (reduced in place in its own buffer)
        n1 = len(wl1.layers)
        attn_bufs = [torch.zeros_like(io._keep[10]) for io in wl1.ios]
        new_ios = []
        for j, (L, io) in enumerate(zip(wl1.layers, wl1.ios)):
            mlp_sum = wl1.ios[(j - 1) % n1]._keep[10]       # mlp_partial_out of the previous layer
            new_ios.append(L.make_io(wl1.shape.batch, io._keep[3], io._keep[2], [mlp_sum], [], io._keep[6],
                                     io._keep[7], io._keep[8], io._keep[9], io._keep[10], attn_bufs[j]))
            L.set_external_attention_sum(attn_bufs[j])
            nccl_bufs.append((mlp_sum, attn_bufs[j]))
        wl1.ios = new_ios
        row = {}
        for name, b in settings:
            wl1.set_budget(b)
            # one CUDA graph per setting (collectives included), so that the host's launch cost of the
            # kernel-by-kernel flow is not what gets measured
            with torch.cuda.stream(stream):
                nccl_step()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                nccl_step()
            row[name + "_us_per_layer"] = round(timed(lambda: g.replay(), steps) * 1e3 / wl1.R, 3)
            del g
        res["nccl_allreduce_window"] = row
    except Exception as e:      # noqa: BLE001
        err = f"{type(e).__name__}: {e}"
        res["error"] = err
    res["workload"] = (f"{world} shards of a configs[1]-shaped layer (tp_degree {world}), rotation of {wl.R} layers, "
                       f"{steps * wl.R} layer-steps per setting, time = slowest rank")
    for w_ in (wl, wl1):
        if w_ is not None:
            w_.close()
    if comm is not None:
        comm.close()
    return res


def run_timeline(P, I, torch, args, stream):
    """Per-kernel timeline of one layer-step from the in-kernel global-timer trace, averaged over
    many cold steps: for each main-stream kernel, when its first CTA started, when the wait on its
    predecessor returned, when its operand stream ended, when it ended."""
    idx = args.config if args.config >= 0 else HEADLINE_CONFIG
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    vflags = (P.FLAG_INT8_KV if args.int8_kv else 0) | (P.FLAG_INT8_WEIGHTS if args.int8_weights else 0)
    wl = Workload(P, I, torch, idx, 0, l2, args.rotation, flags=vflags)
    if args.budget_bytes >= 0:
        wl.set_budget(args.budget_bytes)
    for L in wl.layers:
        L.set_trace(True)
    rows = []
    reps = max(10, args.steps)
    for rep in range(reps + 3):
        with torch.cuda.stream(stream):
            P.preserve_decode_chain(wl.layers, wl.ios, link=False, stream=stream)
        torch.cuda.synchronize()
        for li, L in enumerate(wl.layers):
            tr = L.read_trace()
            if rep >= 3 and li > 0:          # (layer 0 of a call has no kernel in front of it)
                rows.append(tr)
    a = np.array(rows, dtype=np.float64)      # [samples, kernel, slot]
    names = P.KERNEL_NAMES
    table = []
    for k, n in enumerate(names):
        s0, w0, w1, e1, s1, st, e0 = (a[:, k, j] for j in range(7))
        prev_end = a[:, k - 1, 3] if k > 0 else None
        nxt = a[:, k + 1, 2] if k + 1 < len(names) else None
        table.append({
            "kernel": n,
            "start_to_wait_return_us": round(float(np.mean(w1 - s0)) / 1e3, 2),
            "early_start_before_prev_end_us": round(float(np.mean(prev_end - s0)) / 1e3, 2) if k > 0 else None,
            "wait_return_after_prev_end_us": round(float(np.mean(w1 - prev_end)) / 1e3, 2) if k > 0 else None,
            "last_cta_start_after_prev_end_us": round(float(np.mean(s1 - prev_end)) / 1e3, 2) if k > 0 else None,
            "first_wait_return_after_prev_end_us": round(float(np.mean(w0 - prev_end)) / 1e3, 2) if k > 0 else None,
            "wait_return_to_stream_end_us": round(float(np.mean(np.where(st > 0, st - w1, 0.0))) / 1e3, 2),
            "stream_end_to_end_us": round(float(np.mean(np.where(st > 0, e1 - st, e1 - w1))) / 1e3, 2),
            "wait_return_to_end_us": round(float(np.mean(e1 - w1)) / 1e3, 2),
            "end_to_next_wait_return_us": round(float(np.mean(nxt - e1)) / 1e3, 2) if nxt is not None else None,
        })
    layer_us = float(np.mean(a[:, -1, 3] - a[:, 0, 2])) / 1e3
    print(json.dumps({"mode": "timeline", "config_index": idx, "name": wl.shape.name, "samples": len(rows),
                      "budget_bytes": int(wl.layers[0].get_info().prefetch_budget),
                      "precision": "bf16" + (", int8 KV-cache" if args.int8_kv else "") + (", int8 weights" if args.int8_weights else ""),
                      "first_wait_return_to_last_end_us": round(layer_us, 2), "kernels": table}), flush=True)
    wl.close()


def run_decode_loop(P, I, torch, args, stream):
    """A 32-layer model made of configs[1] layers (linked chain: layer i + 1 consumes layer i's
    results), decoding tokens with every context advancing by one per token, against the same chain
    replayed with fixed contexts: us per token with prefetch off / early launch only / on, and the
    number of graphs captured along the way."""
    idx = args.config if args.config >= 0 else 1
    n_layers, n_tokens = args.layers, max(args.steps, 64)
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    vflags = (P.FLAG_INT8_KV if args.int8_kv else 0) | (P.FLAG_INT8_WEIGHTS if args.int8_weights else 0)
    wl = Workload(P, I, torch, idx, 0, l2, rotation=n_layers, flags=vflags)
    shape = wl.shape
    # start n_tokens + 8 below the configured context so that the contexts can advance inside the cache
    start = np.maximum(wl.ctx_host - (n_tokens + 8), 1).astype(np.int32)
    ctx_host = start.copy()
    ctx_dev = torch.from_numpy(ctx_host).cuda()
    ios = []
    for L, io in zip(wl.layers, wl.ios):
        k = io._keep
        ios.append(L.make_io(shape.batch, ctx_dev, ctx_host, k[4], k[5], k[6], k[7], k[8], k[9], k[10]))
    res = {}
    for name, b in (("off", 0), ("early_launch_only", 1), ("l2_sixteenth", l2 // 16)):
        wl.set_budget(b)
        out = {}
        for advancing in (False, True):
            ctx_host[:] = start
            ctx_dev.copy_(torch.from_numpy(start))
            torch.cuda.synchronize()
            caps0 = wl.layers[0].graph_captures()
            # warm-up in the mode that is timed (the first advancing tokens of a setting pay one-off costs
            # of several milliseconds - first replay of a new graph, first launches of the context update)
            with torch.cuda.stream(stream):
                for _ in range(8):
                    P.preserve_decode_chain(wl.layers, ios, link=True, stream=stream)
                    if advancing:
                        ctx_dev += 1
                        ctx_host += 1
            torch.cuda.synchronize()
            ctx_host[:] = start
            ctx_dev.copy_(torch.from_numpy(start))
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.perf_counter()
            with torch.cuda.stream(stream):
                e0.record(stream)
                for _ in range(n_tokens):
                    P.preserve_decode_chain(wl.layers, ios, link=True, stream=stream)
                    if advancing:
                        ctx_dev += 1
                        ctx_host += 1
                e1.record(stream)
            torch.cuda.synchronize()
            wall = (time.perf_counter() - t0) * 1e6 / n_tokens
            key = "advancing" if advancing else "fixed"
            out[key + "_us_per_token"] = round(e0.elapsed_time(e1) * 1e3 / n_tokens, 2)
            out[key + "_host_wall_us_per_token"] = round(wall, 2)
            out[key + "_graph_captures"] = wl.layers[0].graph_captures() - caps0
        out["advancing_over_fixed"] = round(out["advancing_us_per_token"] / out["fixed_us_per_token"], 4)
        res[name] = out
    status = max(L.last_status() for L in wl.layers)
    print(json.dumps({"mode": "decode-loop", "layers": n_layers, "tokens": n_tokens,
                      "precision": "bf16" + (", int8 KV-cache" if args.int8_kv else "") + (", int8 weights" if args.int8_weights else ""),
                      "workload": f"{n_layers} x configs[{idx}] {shape.name} (linked chain), contexts "
                                  f"{int(start.min())}..{int(start.max())} advancing by one per token",
                      "results": res, "device_status": status}), flush=True)
    wl.close()


# ---------------------------------------------------------------------- reference
def cpu_baseline(shape, t, alg: int, budget_s: float, idx: int):
    from oracle import oracle as O
    O.build()
    fn = lambda: O.layer_step(shape, t)
    fn()
    t0 = time.perf_counter()
    n = 0
    while True:
        fn()
        n += 1
        if time.perf_counter() - t0 > budget_s or n >= 50:
            break
    dt = (time.perf_counter() - t0) / n
    return {"value": round(alg / dt / 1e9, 4), "unit": "GB/s", "us_per_layer": round(dt * 1e6, 1),
            "cores": O.num_threads(), "kind": "oracle",
            "sample": f"{n} full layer-steps of configs[{idx}] ({shape.name}), one layer instance, after one untimed run"}


def run_reference(args):
    """The CPU oracle alone, on the host cores: no CUDA library is loaded by this arm."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as O
    from paper_2501_08192_b200 import inputs as I
    O.build()
    idx = args.config if args.config >= 0 else HEADLINE_CONFIG
    shape = I.CONFIGS[idx]
    t = I.make_layers(shape, 1, nan_fill_tail=False)[0]
    alg = algorithmic_bytes(shape, int(t["ctx_len"].sum()))
    fn = lambda: O.layer_step(shape, t)
    warm = min(args.warmup, 2)
    for _ in range(warm):
        fn()
    # each step = one full layer-step; the number of steps is bounded by a time budget
    steps, t0 = 0, time.perf_counter()
    while steps < args.steps and (steps < 3 or time.perf_counter() - t0 < 90.0):
        fn()
        steps += 1
    ms = (time.perf_counter() - t0) * 1e3 / steps
    val = round(alg / (ms * 1e-3) / 1e9, 4)
    sample = f"each step = one full layer-step of configs[{idx}] ({shape.name}) on one layer instance"
    out = {"impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus,
           "steps": steps, "warmup": warm, "ms_per_step": round(ms, 3), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "fp32 values, fp64 accumulation",
           "data": "synthetic (same seeded inputs as the CUDA arm)",
           "config": {"workload": f"configs[{idx}] {shape.name}", "layers_per_step": 1,
                      "algorithmic_bytes_per_layer": alg},
           "us_per_layer": round(ms * 1e3, 1),
           "cpu_baseline": {"value": val, "unit": "GB/s", "cores": O.num_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--config", type=int, default=-1,
                    help="index into the five benchmark configurations (default: all five, configs[3] as the headline)")
    ap.add_argument("--mode", default="bench", choices=("bench", "timeline", "decode-loop", "streams", "real-window"))
    ap.add_argument("--layers", type=int, default=32, help="decode-loop mode: layers of the chain")
    ap.add_argument("--rotation", type=int, default=0, help="layer instances per step (0 = sized from L2)")
    ap.add_argument("--min-layer-steps", type=int, default=MIN_LAYER_STEPS,
                    help="timed layer-steps per setting (lower it only for profiler captures)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--int8-kv", action="store_true", help="run the main measurement over an int8 KV-cache (profiling aid)")
    ap.add_argument("--int8-weights", action="store_true",
                    help="run the main measurement with int8 weights (profiling aid)")
    ap.add_argument("--no-kernels", action="store_true", help="skip the isolated per-kernel timing")
    ap.add_argument("--budget-bytes", type=int, default=-1, help="prefetch budget per window (default: the library's)")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--no-real-window", action="store_true",
                    help="N > 1: skip the measurement of the real communication window")
    ap.add_argument("--dry-run", action="store_true", help="launch plumbing only (CPU, gloo); nothing is timed")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
        return 0
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args, sys.argv[1:])
    run_ours(args)
    return 0


if __name__ == "__main__":
    sys.exit(main())
