"""Pins of the analytical performance model (Section 5, "Performance & cost model"): closed forms of
its three linear terms, Algorithm 1's decisions against the oracle's, monotonicity and saturation in
the L2 size (the trend of the paper's L2-size study), and bounds that hold for any parameters."""
import numpy as np
import pytest

from paper_2501_08192_b200 import inputs as I
from paper_2501_08192_b200 import perf_model as M


def llama70b_ops(devices=32, batch=16, seq=8192, wbytes=1.0):
    # Llama-3-70B: hidden 8192, 64 q / 8 kv heads of 128, ffn 28672; int8 as in the paper's study
    return M.layer_ops(8192, max(64 // devices, 1), max(8 // devices, 1), 128, 28672 // devices, batch, batch * seq,
                       wbytes, wbytes, wbytes)


def test_the_three_linear_terms_have_their_closed_forms():
    hw = M.PAPER_TABLE
    # memory-bound operator: bytes over the off-chip bandwidth; the same bytes from L2 over the L2 bus bandwidth
    op = M.Op("w", "matmul", flops=1e6, prefetchable=1.84e9)
    assert M.op_time(hw, op) == pytest.approx(1e-3)
    assert M.op_time(hw, op, l2_hit_bytes=1.84e9) == pytest.approx(1.84e9 / 12e12)
    assert M.op_time(hw, op, l2_hit_bytes=0.92e9) == pytest.approx(0.5e-3 + 0.92e9 / 12e12)
    # compute-bound operator: operations over the peak throughput
    assert M.op_time(hw, M.Op("c", "matmul", flops=8e12, prefetchable=1e3)) == pytest.approx(1e-2)
    # collective on a ring of 32: 62 steps of (25 us + (size / 32) / 25 GB/s)
    assert M.allreduce_time(hw, 32 * 25e9 * 1e-6) == pytest.approx(62 * (25e-6 + 1e-6))
    assert M.allreduce_time(M.replace(hw, n_devices=1), 1e9) == 0.0


def test_prefetch_decisions_equal_the_oracles_algorithm_1(oracle):
    for s in I.CONFIGS:
        ops = M.layer_ops(s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, s.batch, s.batch * s.ctx)
        g = oracle.layer_graph(s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, s.batch * s.ctx)
        # model op indices -> oracle graph node indices
        to_graph = {0: 0, 1: 1, 2: 3, 3: 4, 4: 5, 5: 6, 6: 8}
        assert [int(ops[i].prefetchable) for i in (1, 2, 3, 5, 6)] == [g[to_graph[i]]["mem"] for i in (1, 2, 3, 5, 6)]
        for budget in (0, 1, 8 << 20, 23068672, 32 << 20, 126 << 20, 1 << 34):
            want = oracle.insert_prefetch_ops(g, budget)
            got = M.insert_prefetches(ops, budget)
            assert {to_graph[c]: sorted(to_graph[j] for j in v) for c, v in got.items()} == \
                   {c: sorted(v) for c, v in want.items() if c != 9}, (s.name, budget)


def test_latency_falls_with_l2_size_and_saturates():
    """The trend of the paper's L2-size study: more L2 -> more prefetched -> lower latency, until every
    window's prefetchable set fits (or the window is too short to fetch more); never slower than
    without prefetching; the gain is bounded by what the hidden off-chip reads cost."""
    hw = M.PAPER_TABLE
    ops = llama70b_ops()
    sizes = [8, 16, 24, 32, 48, 64, 104, 136, 144, 192, 256]
    sweep = M.l2_size_sweep(hw, ops, sizes)
    lat = [r["latency"] for r in sweep]
    assert all(a >= b - 1e-15 for a, b in zip(lat, lat[1:]))                 # monotone
    assert lat[0] > lat[-1]                                                  # it does help
    biggest_window = max(sum(o.prefetchable for o in ops[1:4]), sum(o.prefetchable for o in ops[5:7]))
    flat_from = next(i for i, m in enumerate(sizes) if m * 2**20 > biggest_window)
    assert all(abs(x - lat[flat_from]) < 1e-12 for x in lat[flat_from:])     # saturation
    off = M.predict(hw, ops, budget=0)["on"]
    assert off == pytest.approx(M.predict(hw, ops)["off"])                   # C = 0 is vanilla execution
    hidden = sum(o.prefetchable for o in ops) * (1 / hw.hbm_bw - 1 / hw.l2_bw)
    assert 0 < off - lat[-1] <= hidden + 1e-12
    # with the paper's parameters the windows (62 ring steps of >= 25 us) are long enough to fetch everything
    r = M.predict(M.replace(hw, l2_bytes=1 << 30), ops)
    assert r["prefetched_bytes"] == pytest.approx(r["planned_bytes"])
    # a short window limits the prefetch to what the memory delivers meanwhile
    r = M.predict(M.replace(hw, l2_bytes=1 << 30), ops, window_time=1e-6)
    assert r["prefetched_bytes"] == pytest.approx(2 * 1e-6 * hw.hbm_bw)


def test_speedup_grows_with_link_bandwidth_as_in_the_papers_study():
    """Section 5's link-bandwidth study: a faster link shortens the collectives, so the same hidden
    memory time is a larger share of the layer."""
    ops = llama70b_ops(devices=128, batch=16, seq=8192)
    sp = []
    for gbit in (200, 400, 600, 800, 1000):
        hw = M.replace(M.PAPER_TABLE, link_bw=gbit * 1e9 / 8, n_devices=128)
        sp.append(M.predict(hw, ops)["speedup_on_vs_off"])
    assert all(b > a for a, b in zip(sp, sp[1:])) and sp[0] > 1.0


def test_gpu_extension_terms():
    hw = M.b200_measured()
    s = I.CONFIGS[3]
    ops = M.layer_ops(s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, s.batch, s.batch * 2304)
    r = M.predict(hw, ops, budget=1, window_time=3e-6)
    n_kernels = sum(1 for o in ops if o.kind != "comm")
    assert r["off"] - r["early_launch_only"] == pytest.approx(n_kernels * hw.early_launch_hides)
    assert r["on"] == pytest.approx(r["early_launch_only"])                  # one byte plans nothing
    # the bytes term alone reproduces the roofline floor: ~598 MB at 6.9 TB/s
    floor = sum(o.prefetchable + o.other_bytes for o in ops if o.kind != "comm") / hw.hbm_bw
    assert 80e-6 < floor < 95e-6
    big = M.predict(hw, ops, budget=hw.l2_bytes, truncate=True, window_time=20e-6)
    assert big["on"] < big["early_launch_only"]
