"""Host-side checks that need no GPU: the C-ABI library loads and exports every
symbol the header declares, the library's prefetch planner agrees with the
oracle's restatement of Algorithm 1, byte accounting, and error codes."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2501_08192_b200 import binding as P
from paper_2501_08192_b200 import build as B
from paper_2501_08192_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return P.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "preserve.h")).read()
    return re.findall(r"PRESERVE_API\s+[\w\s\*]+?\b(preserve_\w+)\s*\(", text)


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert len(names) >= 14 and set(names) == set(P.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_strerror_covers_all_codes(lib):
    texts = {P.preserve_strerror(c) for c in range(0, -8, -1)}
    assert len(texts) == 8 and "unknown error" not in texts
    assert P.preserve_strerror(-99) == "unknown error"


def layer_nodes(s, sum_ctx):
    d = s.head_dim
    a = [2 * s.hidden * (s.n_q_heads + 2 * s.n_kv_heads) * d, 2 * 2 * sum_ctx * s.n_kv_heads * d,
         2 * s.n_q_heads * d * s.hidden]
    b = [2 * s.hidden * 2 * s.ffn, 2 * s.ffn * s.hidden]
    return a, b


def test_planner_matches_algorithm_1_oracle(lib, oracle):
    rng = np.random.default_rng(7)
    for s in I.CONFIGS:
        sum_ctx = s.batch * s.ctx
        g = oracle.layer_graph(s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, sum_ctx)
        na, nb = layer_nodes(s, sum_ctx)
        assert [g[i]["mem"] for i in (1, 3, 4)] == na and [g[i]["mem"] for i in (6, 8)] == nb
        budgets = [0, 1, na[0], na[0] + 1, na[0] + na[1], na[0] + na[1] + 1, sum(na), sum(na) + 1, nb[0], nb[0] + 1,
                   sum(nb), sum(nb) + 1, 126 << 20] + [int(x) for x in rng.integers(0, 2 * sum(na + nb), 30)]
        for Cb in budgets:
            plan = oracle.insert_prefetch_ops(g, Cb)
            want_a = [na[i] if n in plan[0] else 0 for i, n in enumerate((1, 3, 4))]
            want_b = [nb[i] if n in plan[5] else 0 for i, n in enumerate((6, 8))]
            assert P.preserve_plan_window(na, Cb, P.PLAN_WHOLE_NODE) == want_a, (s.name, Cb)
            assert P.preserve_plan_window(nb, Cb, P.PLAN_WHOLE_NODE) == want_b, (s.name, Cb)
            assert P.preserve_plan_window(na, Cb, P.PLAN_TRUNCATE) == oracle.truncate_plan(na, Cb)
            assert P.preserve_plan_window(nb, Cb, P.PLAN_TRUNCATE) == oracle.truncate_plan(nb, Cb)


def test_planner_edge_cases(lib):
    assert P.preserve_plan_window([], 100) == []
    assert P.preserve_plan_window([0, 0], 1) == [0, 0]
    assert P.preserve_plan_window([10], 10) == [0] and P.preserve_plan_window([10], 11) == [10]
    out = (C.c_uint64 * 1)()
    assert lib.preserve_plan_window(None, 1, 5, 0, out) == P.PRESERVE_EINVAL
    assert lib.preserve_plan_window(out, 1, 5, 7, out) == P.PRESERVE_EINVAL


def test_algorithmic_bytes_closed_form(lib):
    # Llama-3-8B TP=8 shard, batch 8, ctx 4096: weights 54,525,952 + K/V 16,777,216 + activations
    s = I.CONFIGS[1]
    cfg = P.make_config(s)
    BH = s.batch * s.hidden * 2
    act = 2 * ((s.tp_degree + 1) * BH + s.hidden * 2 + 2 * BH)          # both windows
    act += BH + s.batch * (s.n_q_heads + 2 * s.n_kv_heads) * 128 * 2     # QKV: x in, q/k/v out
    act += 2 * s.batch * s.n_q_heads * 128 * 2                           # attention: q in, o out
    act += s.batch * s.n_q_heads * 128 * 2 + BH                          # O projection
    act += BH + s.batch * s.ffn * 2 + s.batch * s.ffn * 2 + BH           # gate/up, down
    assert s.weight_bytes() == 54525952
    assert P.preserve_algorithmic_bytes(cfg, s.batch, s.batch * s.ctx) == 54525952 + 16777216 + act
    assert abs(P.preserve_algorithmic_bytes(cfg, s.batch, s.batch * s.ctx) - 73.18e6) < 0.2e6
    for i, total in ((2, 288.48e6), (4, 598.87e6)):
        s = I.CONFIGS[i]
        got = P.preserve_algorithmic_bytes(P.make_config(s), s.batch, s.batch * s.ctx)
        assert abs(got - total) / total < 0.005
    bad = P.make_config(s)
    bad.head_dim = 64
    assert P.preserve_algorithmic_bytes(bad, 1, 1) == 0


def test_init_without_a_device_fails_cleanly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    cfg = P.make_config(I.small_shape())
    buf = (C.c_uint8 * 64)()
    addr = (C.addressof(buf) + 15) & ~15
    w = P.LayerWeights(*([addr] * 9))
    h = C.c_void_p(1)
    rc = lib.preserve_layer_init(C.byref(cfg), C.byref(w), C.byref(h))
    assert rc in (P.PRESERVE_EARCH, P.PRESERVE_ECUDA) and not h.value
    assert lib.preserve_layer_init(None, C.byref(w), C.byref(h)) == P.PRESERVE_EINVAL
    cfg.head_dim = 96
    assert lib.preserve_layer_init(C.byref(cfg), C.byref(w), C.byref(h)) == P.PRESERVE_ESHAPE
    lib.preserve_layer_destroy(None)     # allowed


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(P, "_lib", None)
    monkeypatch.setattr(P, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        P.lib()


def test_input_recipe_is_stable():
    """Seeded draws: a checksum of the first values of config 1 pins the draw order."""
    t = I.make_layers(I.CONFIGS[0], 1)[0]
    assert t["w_q"].shape == (1024, 512) and t["k_cache"].shape == (1, 4, 513, 128)
    assert t["ctx_len"].tolist() == [512]
    assert (t["k_cache"][:, :, 512] == I.BF16_NAN).all()
    r = I.make_layers(I.CONFIGS[3], 1, nan_fill_tail=True)[0]["ctx_len"]
    assert r.min() >= 512 and r.max() <= 4096 and len(set(r.tolist())) > 32
    again = I.make_layers(I.CONFIGS[0], 1)[0]
    assert all(np.array_equal(t[k], again[k]) for k in ("w_q", "w_down", "k_cache", "partials_in"))


# ---------------------------------------------------------------- Algorithm 1 as a graph pass
_KIND = {"comm": P.NODE_COMM, "matmul": P.NODE_MATMUL, "attention": P.NODE_ATTENTION, "other": P.NODE_OTHER}


def _run_graph_pass(g, budget, mode=P.PLAN_WHOLE_NODE):
    hits = P.preserve_plan_graph([_KIND[n["kind"]] for n in g], [int(n["mem"]) for n in g],
                                 [n["children"] for n in g], budget, mode)
    plan = {i: [] for i, n in enumerate(g) if n["kind"] == "comm"}
    for comm, node, nbytes in hits:
        plan[comm].append((node, nbytes))
    return plan


def test_graph_pass_matches_the_oracle_on_whole_models(lib, oracle):
    """32- and 80-layer operator chains of the Llama-shaped shards: the library's pass inserts the
    same prefetches, beside the same communication operators, in the same order, as the oracle's
    restatement of Algorithm 1."""
    for s, n_layers in ((I.CONFIGS[1], 32), (I.CONFIGS[2], 80), (I.CONFIGS[3], 80), (I.CONFIGS[4], 32)):
        g = oracle.layer_graph(s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, s.batch * s.ctx, n_layers)
        for budget in (0, 1, 8 << 20, 32 << 20, 126 << 20, 1 << 30, 1 << 40):
            want = oracle.insert_prefetch_ops(g, budget)
            got = _run_graph_pass(g, budget)
            assert {k: [n for n, _ in v] for k, v in got.items()} == want, (s.name, budget)
            assert all(b == g[n]["mem"] for v in got.values() for n, b in v)


def test_graph_pass_matches_the_oracle_on_random_dags(lib, oracle):
    rng = np.random.default_rng(11)
    kinds = ("comm", "matmul", "attention", "other")
    for trial in range(200):
        n = int(rng.integers(1, 40))
        g = []
        for i in range(n):
            later = list(range(i + 1, n))
            k = int(rng.integers(0, min(4, len(later)) + 1))
            ch = sorted(rng.choice(later, size=k, replace=False).tolist()) if k else []
            g.append({"kind": kinds[int(rng.choice(4, p=(0.2, 0.4, 0.15, 0.25)))],
                      "mem": int(rng.integers(0, 1000)), "children": [int(c) for c in ch]})
        total = sum(x["mem"] for x in g)
        for budget in (0, 1, int(rng.integers(0, total + 2)), total + 1):
            want = oracle.insert_prefetch_ops(g, budget)
            got = _run_graph_pass(g, budget)
            assert {k: [nn for nn, _ in v] for k, v in got.items()} == want, (trial, budget)


def test_graph_pass_truncate_mode_and_errors(lib, oracle):
    # on a chain the TRUNCATE pass equals the ordered-list form, window by window
    s = I.CONFIGS[2]
    g = oracle.layer_graph(s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, s.batch * s.ctx, 2)
    na, nb = layer_nodes(s, s.batch * s.ctx)
    for budget in (0, 100, 64 << 20, 126 << 20, 1 << 29):
        got = _run_graph_pass(g, budget, P.PLAN_TRUNCATE)
        for base, comm_a, comm_b in ((0, 0, 5), (9, 9, 14)):
            a = {n - base: b for n, b in got[comm_a]}
            b_ = {n - base: b for n, b in got[comm_b]}
            assert [a.get(i, 0) for i in (1, 3, 4)] == oracle.truncate_plan(na, budget)
            assert [b_.get(i, 0) for i in (6, 8)] == oracle.truncate_plan(nb, budget)
    # a cycle is walked once; bad arguments are refused
    assert P.preserve_plan_graph([0, 1, 1], [0, 5, 5], [[1], [2], [1]], 100) == [(0, 1, 5), (0, 2, 5)]
    assert P.preserve_plan_graph([], [], [], 10) == []
    with pytest.raises(P.PreserveError):
        P.preserve_plan_graph([0, 9], [0, 1], [[1], []], 10)
    with pytest.raises(P.PreserveError):
        P.preserve_plan_graph([0, 1], [0, 1], [[5], []], 10)
    n_out = C.c_int32()
    k = (C.c_int32 * 2)(0, 1)
    m = (C.c_uint64 * 2)(0, 5)
    so = (C.c_int32 * 3)(0, 1, 1)
    su = (C.c_int32 * 1)(1)
    assert lib.preserve_plan_graph(2, k, m, so, su, 10, 0, 0, None, None, None, C.byref(n_out)) == P.PRESERVE_ETOOBIG
    assert n_out.value == 1


def test_no_process_wide_switches_in_the_kernels_sources():
    """Distinct handles are independent: the sources keep no mutable process-wide switch (the early-launch
    flag, the prefetch mechanism and chunk size are per handle and travel as launch arguments), read no
    environment variable, and the only file-scope state left is per-device bookkeeping."""
    csrc = os.path.join(ROOT, "paper_2501_08192_b200", "csrc")
    allowed_static = ("static PerDeviceSize", "static __device__ __align__(256) unsigned char g_static_scratch",
                      "static const int", "static const int32_t", "static_assert", "static_cast", "static cudaError_t",
                      "static int reset_trace", "static size_t attn_smem_bytes", "static size_t attn_kv8_smem_bytes", "static EncodeTiledFn fn",
                      "static bool tried", "static constexpr")
    for name in sorted(os.listdir(csrc)):
        text = open(os.path.join(csrc, name)).read()
        assert "getenv" not in text, name
        for bad in ("g_pdl", "g_pf_mode", "g_pf_chunk", "static bool attr", "static bool np_set"):
            assert bad not in text, (name, bad)
        for line in text.splitlines():
            st = line.strip()
            if st.startswith("static ") and not st.startswith(allowed_static):
                raise AssertionError(f"{name}: unexpected file-scope or function-scope static: {st}")
