"""GPU tests of the runtime around the kernels, through the C ABI: a decode loop whose contexts
advance (graph reuse), layers wired output to input inside one call, the give-up paths of the
bounded waits, the prefetch mechanisms and path-forcing flags, and the prefetch kernel's own
evaluation of Algorithm 1.  Parity bar as in test_gpu_parity.py (gpu_util.tolerance_ok)."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2501_08192_b200 import binding as P
from paper_2501_08192_b200 import inputs as I

import gpu_util as G

pytestmark = pytest.mark.gpu


def _append_to_host_cache(t, ref):
    """What the step did to the cache, replayed on the host copy: slot ctx_len[b] takes the new
    key / value as bf16, ctx_len advances by one."""
    for b in range(t["ctx_len"].shape[0]):
        n = int(t["ctx_len"][b])
        t["k_cache"][b, :, n] = I.f32_to_bf16_bits(ref["k_new"][b])
        t["v_cache"][b, :, n] = I.f32_to_bf16_bits(ref["v_new"][b])
    t["ctx_len"] = t["ctx_len"] + 1


@pytest.mark.parametrize("batch,hidden,ffn", [(3, 512, 384), (20, 512, 384)], ids=["gemv", "tensor"])
def test_decode_loop_with_advancing_context_reuses_one_graph(oracle, batch, hidden, ffn):
    """84 consecutive tokens: every sequence grows by one per step (ragged start, crossing 64-key
    tile boundaries), each step compared with the oracle stepped the same way, while the library
    keeps replaying cached graphs instead of capturing one per token."""
    steps = 84
    shape = I.small_shape(name="loop", batch=batch, hidden=hidden, ffn=ffn, ctx=40 + steps + 60, ctx_min=30, seed=71)
    t = I.make_layers(shape, 1)[0]
    # start well below capacity so the contexts can grow: keep the drawn lengths within [30, 100]
    t["ctx_len"] = (30 + (t["ctx_len"] - 30) % 71).astype(np.int32)
    for b in range(batch):
        t["k_cache"][b, :, int(t["ctx_len"][b]):] = I.BF16_NAN
        t["v_cache"][b, :, int(t["ctx_len"][b]):] = I.BF16_NAN
    dl = G.DeviceLayer(shape, t)
    stream = torch.cuda.Stream()
    rng = np.random.default_rng(5)
    try:
        for step in range(steps):
            # a new residual every token (host -> device copy on the step's stream)
            resid = I.f32_to_bf16_bits(rng.standard_normal((batch, hidden), dtype=np.float32))
            t["residual_in"] = resid
            with torch.cuda.stream(stream):
                dl.residual.copy_(G.bits_to_cuda(resid), non_blocking=False)
                dl.run(stream)
            ref = oracle.layer_step(shape, t)
            stream.synchronize()
            out = dl.outputs()
            for name in ("attn_partial", "h2", "mlp_partial"):
                G.assert_close(out[name], ref[name], f"token {step}:{name}")
            k_new, v_new = dl.appended_kv()
            G.assert_close(k_new, ref["k_new"], f"token {step}:k_new")
            _append_to_host_cache(t, ref)
            with torch.cuda.stream(stream):
                dl.ctx_dev += 1
            dl.ctx_host += 1          # the host copy the library plans with (same array the io points at)
            stream.synchronize()
        assert dl.layer.last_status() == P.PRESERVE_OK
        assert 1 <= dl.layer.graph_captures() <= 4, dl.layer.graph_captures()
        # the whole cache now equals the host replay (bit compare of the live slots)
        kc = G.cuda_to_bits(dl.k_cache)
        for b in range(batch):
            n = int(t["ctx_len"][b])
            want = t["k_cache"][b, :, :n]
            got = kc[b, :, :n]
            assert np.mean(want == got) > 0.99      # appended entries may differ by one bf16 ulp from the oracle's
    finally:
        dl.close()


def test_graph_replay_equals_direct_launches_bit_for_bit(oracle):
    shape = I.small_shape(name="graph_vs_direct", batch=6, ctx=300, ctx_min=20, seed=72)
    t = I.make_layers(shape, 1)[0]
    base = None
    stream = torch.cuda.Stream()
    for flags, s in ((0, stream), (0, None), (P.FLAG_NO_GRAPH, stream)):
        dl = G.DeviceLayer(shape, t, flags=flags)
        try:
            for _ in range(3):
                if s is None:
                    dl.run()
                else:
                    with torch.cuda.stream(s):
                        dl.run(s)
                bits = dl.output_bits()
                if base is None:
                    base = bits
                for k in base:
                    assert np.array_equal(base[k], bits[k]), (flags, k)
            caps = dl.layer.graph_captures()
            assert caps == (1 if (flags == 0 and s is not None) else 0)
        finally:
            dl.close()


@pytest.mark.parametrize("batch", [4, 24], ids=["gemv", "tensor"])
def test_layers_wired_output_to_input_without_link(oracle, batch):
    """Two layers in one call, layer 1's partials_in[0] / residual_in being layer 0's bf16 output
    buffers (link = 0): layer 1 must see layer 0's finished results although its window kernel is
    launched early."""
    shape = I.small_shape(name="wired", batch=batch, hidden=2048, ffn=256, ctx=90, ctx_min=5, seed=73)
    layers = I.make_layers(replace(shape, layers=2))
    dls = [G.DeviceLayer(shape, t) for t in layers]
    stream = torch.cuda.Stream()
    try:
        d0, d1 = dls
        # poison layer 0's outputs so that a premature read is far off
        d0.mlp_out.t.fill_(1000.0)
        d0.residual_out.t.fill_(-1000.0)
        d1.io = d1.layer.make_io(batch, d1.ctx_dev, d1.ctx_host, [d0.mlp_out.t] + d1.partials[1:], d1.peers,
                                 d0.residual_out.t, d1.k_cache, d1.v_cache, d1.residual_out.t, d1.mlp_out.t,
                                 d1.attn_out.t)
        for rep in range(3):
            torch.cuda.synchronize()
            d0.mlp_out.t.fill_(1000.0)
            d0.residual_out.t.fill_(-1000.0)
            torch.cuda.synchronize()
            with torch.cuda.stream(stream):
                P.preserve_decode_chain([d0.layer, d1.layer], [d0.io, d1.io], link=False, stream=stream)
            stream.synchronize()
            ref0 = oracle.layer_step(shape, layers[0])
            out0 = d0.outputs()
            for name in ("attn_partial", "h2", "mlp_partial"):
                G.assert_close(out0[name], ref0[name], f"layer 0:{name}")
            # layer 1 against the oracle fed with exactly what layer 0 wrote (its bf16 buffers)
            parts = I.bf16_bits_to_f32(layers[1]["partials_in"]).copy()
            parts[0] = out0["mlp_partial"]
            ref1 = oracle.layer_step(shape, layers[1], partials_in=parts, residual_in=out0["h2"])
            out1 = d1.outputs()
            for name in ("attn_partial", "h2", "mlp_partial"):
                G.assert_close(out1[name], ref1[name], f"layer 1 (rep {rep}):{name}")
            # restore layer caches for the next repetition (the step appended)
        assert d0.layer.last_status() == P.PRESERVE_OK and d1.layer.last_status() == P.PRESERVE_OK
    finally:
        for d in dls:
            d.close()


WITHHOLD_CASES = [
    ("window", P.WITHHOLD_WINDOW, dict(batch=3, hidden=2048, ffn=256), 0),
    ("gemv", P.WITHHOLD_GEMV, dict(batch=4), 0),
    ("tensor", P.WITHHOLD_TENSOR, dict(batch=20), 0),
    # batch 64: the split-K hand-over by bulk copies out of the senders' shared memory
    ("tensor_wide", P.WITHHOLD_TENSOR, dict(batch=64), 0),
    ("attention", P.WITHHOLD_ATTENTION, dict(batch=4), 0),
    # int8 weights: the GEMV ring of codes, and the tcgen05 ring in front of the widening warps
    ("gemv_int8", P.WITHHOLD_GEMV, dict(batch=4), P.FLAG_INT8_WEIGHTS),
    ("tensor_int8", P.WITHHOLD_TENSOR, dict(batch=20), P.FLAG_INT8_WEIGHTS),
]


@pytest.mark.parametrize("name,what,kw,flags", WITHHOLD_CASES, ids=[c[0] for c in WITHHOLD_CASES])
def test_a_wait_that_runs_out_is_reported_and_the_handle_survives(oracle, name, what, kw, flags):
    """One producer withholds one issue; the consumer's wait (limit shortened to 2^21 SM cycles,
    about a millisecond) runs out, the kernels give up and return, the status says so, and after
    clearing it the same handle computes the right result again."""
    shape = I.small_shape(name="timeout_" + name, ctx=150, ctx_min=9, seed=74, **kw)
    t = I.make_layers(shape, 1)[0]
    ref = oracle.layer_step(shape, t, int8_weights=bool(flags & P.FLAG_INT8_WEIGHTS))
    dl = G.DeviceLayer(shape, t, flags=flags)
    stream = torch.cuda.Stream()
    try:
        dl.layer.debug_set(P.DEBUG_WAIT_LIMIT_CYCLES, 1 << 21)
        dl.layer.debug_set(P.DEBUG_WITHHOLD, what)
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            t0.record(stream)
            dl.run(stream)
            t1.record(stream)
        stream.synchronize()
        assert t0.elapsed_time(t1) < 200.0          # milliseconds: a few expired waits, not a second each
        assert dl.layer.last_status() == P.PRESERVE_ETIMEOUT
        assert dl.layer.last_status() == P.PRESERVE_ETIMEOUT      # sticky until cleared
        # back to normal: same handle, same buffers
        dl.layer.debug_set(P.DEBUG_WITHHOLD, 0)
        dl.layer.clear_status()
        dl.k_cache.copy_(G.bits_to_cuda(t["k_cache"]))
        dl.v_cache.copy_(G.bits_to_cuda(t["v_cache"]))
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            dl.run(stream)
        stream.synchronize()
        assert dl.layer.last_status() == P.PRESERVE_OK
        out = dl.outputs()
        for n in ("attn_partial", "h2", "mlp_partial"):
            G.assert_close(out[n], ref[n], f"{name} after recovery:{n}")
        # a fresh handle works too
        d2 = G.DeviceLayer(shape, t, flags=flags)
        try:
            d2.run()
            assert d2.layer.last_status() == P.PRESERVE_OK
            G.assert_close(d2.outputs()["mlp_partial"], ref["mlp_partial"], "fresh handle")
        finally:
            d2.close()
    finally:
        dl.close()


def test_prefetch_mechanisms_flags_and_forced_paths_keep_results(oracle):
    """Prefetch by bulk L2 prefetch, per-line hints or plain loads, with or without a persisting
    access-policy window: bit-identical outputs.  Forcing the GEMV kernels at batch 20 or the
    tcgen05 kernels at batch 6: within tolerance of the oracle."""
    shape = I.small_shape(name="mech", batch=6, ctx=400, ctx_min=30, seed=75)
    t = I.make_layers(shape, 1)[0]
    stream = torch.cuda.Stream()
    base = None
    for flags in (0, P.FLAG_PERSIST_L2):
        dl = G.DeviceLayer(shape, t, flags=flags)
        try:
            l2 = int(dl.layer.get_info().l2_bytes)
            for mech, chunk, ctas in ((0, 4096, 128), (1, 2048, 32), (2, 4096, 16), (0, 128, 1), (2, 1 << 20, 8)):
                dl.layer.set_prefetch_mechanism(mech, chunk, ctas)
                for budget in (l2 // 8, l2):
                    dl.layer.set_prefetch_bytes(budget)
                    with torch.cuda.stream(stream):
                        dl.run(stream)
                    bits = dl.output_bits()
                    if base is None:
                        base = bits
                    for k in base:
                        assert np.array_equal(base[k], bits[k]), (flags, mech, chunk, ctas, budget, k)
            assert dl.layer.last_status() == P.PRESERVE_OK
        finally:
            dl.close()
    dl = G.DeviceLayer(shape, t)
    try:
        for bad in ((3, 4096, 8), (0, 100, 8), (0, 4096, 0)):
            with pytest.raises(P.PreserveError):
                dl.layer.set_prefetch_mechanism(*bad)
    finally:
        dl.close()
    for batch, flag, tensor in ((20, P.FLAG_FORCE_GEMV, 0), (6, P.FLAG_FORCE_TENSOR, 1)):
        s2 = I.small_shape(name="forced", batch=batch, ctx=120, ctx_min=4, seed=76)
        t2 = I.make_layers(s2, 1)[0]
        ref = oracle.layer_step(s2, t2)
        dl = G.DeviceLayer(s2, t2, flags=flag)
        try:
            assert int(dl.layer.get_info().uses_tensor_path) == tensor
            dl.run()
            assert dl.layer.last_status() == P.PRESERVE_OK
            out = dl.outputs()
            for n in ("attn_partial", "h2", "mlp_partial"):
                G.assert_close(out[n], ref[n], f"forced path {flag}:{n}")
        finally:
            dl.close()


def test_prefetch_kernel_evaluates_the_same_plan_as_the_host(oracle):
    """The side-stream kernel walks the window's nodes itself with the device copy of the lengths;
    what it decides equals the host plan (and the oracle's Algorithm 1) for every budget and mode."""
    shape = I.small_shape(name="devplan", batch=5, ctx=700, ctx_min=100, n_q_heads=4, n_kv_heads=2, seed=77)
    t = I.make_layers(shape, 1)[0]
    dl = G.DeviceLayer(shape, t)
    stream = torch.cuda.Stream()
    try:
        info = dl.layer.get_info()
        w = [int(x) for x in info.weight_bytes]
        kv = 2 * int(t["ctx_len"].sum()) * shape.n_kv_heads * shape.head_dim * 2
        na, nb = [w[0], kv, w[1]], [w[2], w[3]]
        buf = torch.zeros(6, dtype=torch.int64, device="cuda")
        budgets = [1, 200, w[0], w[0] + 1, w[0] + kv // 2, w[0] + kv, w[0] + kv + 1, sum(na) + 1, w[2] + 130,
                   sum(nb) + 1, 1 << 40]
        for mode in (P.PLAN_WHOLE_NODE, P.PLAN_TRUNCATE):
            dl.layer.set_plan_mode(mode)
            for budget in budgets:
                dl.layer.set_prefetch_bytes(budget)
                with torch.cuda.stream(stream):
                    buf.zero_()
                    dl.run(stream)
                    dl.layer.debug_copy(6, buf, stream)
                stream.synchronize()
                host = [list(r) for r in dl.layer.get_info().planned_bytes]
                if mode == P.PLAN_TRUNCATE:
                    want_a, want_b = oracle.truncate_plan(na, budget), oracle.truncate_plan(nb, budget)
                else:
                    want_a = P.preserve_plan_window(na, budget)
                    want_b = P.preserve_plan_window(nb, budget)
                assert host == [want_a, want_b + [0]], (mode, budget)
                dev = buf.cpu().numpy().reshape(2, 3).tolist()
                # (a window with an empty host plan launches no prefetch kernel: its slots keep old values)
                if sum(want_a):
                    assert dev[0] == want_a, (mode, budget, dev)
                if sum(want_b):
                    assert dev[1] == want_b + [0], (mode, budget, dev)
        assert dl.layer.last_status() == P.PRESERVE_OK
    finally:
        dl.close()


def test_device_lengths_beyond_the_host_copy_are_reported_not_written(oracle):
    """ctx_len on the device describing far more attention work than the host copy the step was
    planned with: the surplus work items are dropped (no write beyond the partial buffers) and the
    status reports the mismatch."""
    shape = I.small_shape(name="ctx_mismatch", batch=4, n_q_heads=4, n_kv_heads=4, ctx=60000, seed=78)
    cap = shape.kv_capacity
    z = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device="cuda")
    q_hi, q_lo = z(4, 4, 128), z(4, 4, 128)
    kc, vc = z(4, 4, cap, 128), z(4, 4, cap, 128)
    o_hi, o_lo = z(4, 4, 128), z(4, 4, 128)
    host = np.full(4, 10, np.int32)                     # planned: one tile per stream
    dev = torch.full((4,), 59999, dtype=torch.int32, device="cuda")     # device: 938 tiles per stream
    rc = P.preserve_attention_static(q_hi, q_lo, kc, vc, dev, host, 4, 4, o_hi, o_lo)
    assert rc == P.PRESERVE_OK
    assert P.preserve_attention_static_status() == P.PRESERVE_ESHAPE
    # the next call clears the word again
    dev2 = torch.from_numpy(host).cuda()
    assert P.preserve_attention_static(q_hi, q_lo, kc, vc, dev2, host, 4, 4, o_hi, o_lo) == P.PRESERVE_OK
    assert P.preserve_attention_static_status() == P.PRESERVE_OK
