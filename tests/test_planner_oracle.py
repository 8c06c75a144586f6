"""Pins for the prefetch-insertion oracle (Algorithm 1): hand-worked cases,
graph-walk behaviour on small explicit graphs, and invariants.  CPU only."""
import os

import numpy as np
import pytest

from paper_2501_08192_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "planner_cases.txt")
NAMES = {1: "Wqkv", 3: "KV", 4: "Wo", 6: "Wgu", 8: "Wdown"}


def golden_cases():
    cases = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            nums, a, b = [s.strip() for s in line.split("|")]
            vals = [int(v) for v in nums.split()]
            cases.append((vals, [] if a == "-" else a.split(), [] if b == "-" else b.split()))
    return cases


@pytest.mark.parametrize("vals,win_a,win_b", golden_cases())
def test_hand_worked_cases(oracle, vals, win_a, win_b):
    H, nq, nkv, d, F, kv_tokens, C = vals
    g = oracle.layer_graph(H, nq, nkv, d, F, kv_tokens)
    plan = oracle.insert_prefetch_ops(g, C)
    assert [NAMES[n] for n in plan[0]] == win_a
    assert [NAMES[n] for n in plan[5]] == win_b
    assert plan[9] == []                      # closing comm op has no successors


def test_byte_table_of_the_graph(oracle):
    # node sizes against the shapes' closed forms
    s = I.CONFIGS[2]
    g = oracle.layer_graph(s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, s.batch * s.ctx)
    assert [g[i]["mem"] for i in (1, 3, 4, 6, 8)] == [20971520, 67108864, 16777216, 117440512, 58720256]
    assert sum(g[i]["mem"] for i in (1, 4, 6, 8)) == s.weight_bytes() == 213909504


def test_walk_is_breadth_first_and_stops_at_comm(oracle):
    # comm0 -> {m1, m2}; m1 -> m3; m2 -> comm4 -> m5.  BFS order: m1, m2, m3, comm4.
    g = [
        {"kind": "comm", "mem": 0, "children": [1, 2]},
        {"kind": "matmul", "mem": 10, "children": [3]},
        {"kind": "matmul", "mem": 20, "children": [4]},
        {"kind": "matmul", "mem": 40, "children": []},
        {"kind": "comm", "mem": 0, "children": [5]},
        {"kind": "matmul", "mem": 5, "children": []},
    ]
    assert oracle.insert_prefetch_ops(g, 1000) == {0: [1, 2, 3], 4: [5]}
    # budget 31: 10, 30 fit; 70 does not -> stop (depth-first order would have taken m3 before m2)
    assert oracle.insert_prefetch_ops(g, 31) == {0: [1, 2], 4: [5]}
    assert oracle.insert_prefetch_ops(g, 30) == {0: [1], 4: [5]}
    # the comm op ends the walk: m5 is never prefetched for comm0 however large C is
    assert 5 not in oracle.insert_prefetch_ops(g, 10 ** 9)[0]


def test_comm_reached_before_later_siblings_ends_the_walk(oracle):
    # children in BFS order: comm first -> nothing after it is visited
    g = [
        {"kind": "comm", "mem": 0, "children": [1, 2]},
        {"kind": "comm", "mem": 0, "children": []},
        {"kind": "matmul", "mem": 1, "children": []},
    ]
    assert oracle.insert_prefetch_ops(g, 100)[0] == []


def test_other_nodes_cost_nothing_and_overflow_skips_smaller_later_nodes(oracle):
    g = [
        {"kind": "comm", "mem": 0, "children": [1]},
        {"kind": "other", "mem": 10 ** 12, "children": [2]},
        {"kind": "matmul", "mem": 50, "children": [3]},
        {"kind": "attention", "mem": 100, "children": [4]},
        {"kind": "matmul", "mem": 1, "children": []},
    ]
    assert oracle.insert_prefetch_ops(g, 1000)[0] == [2, 3, 4]
    assert oracle.insert_prefetch_ops(g, 150)[0] == [2]      # 150 is not < 150; node 4 never considered
    assert oracle.insert_prefetch_ops(g, 151)[0] == [2, 3]   # 151 is not < 151 at node 4
    assert oracle.insert_prefetch_ops(g, 152)[0] == [2, 3, 4]


def test_invariants_over_random_budgets(oracle):
    rng = np.random.default_rng(0)
    for s in I.CONFIGS:
        g = oracle.layer_graph(s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, s.batch * s.ctx, n_layers=2)
        prev = None
        for C in sorted(int(c) for c in rng.integers(0, 2 * 10 ** 9, size=40)):
            plan = oracle.insert_prefetch_ops(g, C)
            sizes = {op: sum(g[n]["mem"] for n in ns) for op, ns in plan.items()}
            for op, ns in plan.items():
                assert sizes[op] < C or sizes[op] == 0
                # prefix property: the inserted nodes are the first eligible successors, in order
                elig = []
                for n in range(op + 1, len(g)):
                    if g[n]["kind"] == "comm":
                        break
                    if g[n]["kind"] in ("matmul", "attention"):
                        elig.append(n)
                assert ns == elig[:len(ns)]
            if prev is not None:
                assert all(sizes[op] >= prev[op] for op in sizes)   # monotone in C
            prev = sizes
        # both layers of the chain plan identically
        assert [n - 9 for n in plan[9]] == plan[0] and [n - 9 for n in plan[14]] == plan[5]


def test_truncate_mode_by_its_definition(oracle):
    nb = [6291456, 536870912, 4194304]
    assert oracle.truncate_plan(nb, 0) == [0, 0, 0]
    assert oracle.truncate_plan(nb, 6291456) == [6291456, 0, 0]
    # C = 100 MiB: Wqkv whole, then the first 104857600 - 6291456 bytes of KV (a multiple of 128), nothing after
    assert oracle.truncate_plan(nb, 104857600) == [6291456, 98566144, 0]
    # C large enough for everything (strictly): all whole
    assert oracle.truncate_plan(nb, sum(nb) + 1) == nb
    # exactly equal: the last node is cut to what is left, rounded down to 128 B -> the whole node
    assert oracle.truncate_plan(nb, sum(nb)) == nb
    # rounding down to the granule
    assert oracle.truncate_plan([1000, 1000], 1300) == [1000, 256]
    assert oracle.truncate_plan([1000], 999) == [896]
