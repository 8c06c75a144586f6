"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on
the same seeded inputs.  Tolerance (written in gpu_util.tolerance_ok):
|gpu - ref| <= 2e-2 * min(1, rms(ref)) + 1e-2 * |ref| per element."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2501_08192_b200 import binding as P
from paper_2501_08192_b200 import inputs as I

import gpu_util as G

pytestmark = pytest.mark.gpu


def full_check(oracle, shape, flags=0, budget=None):
    t = I.make_layers(shape, 1)[0]
    ref = oracle.layer_step(shape, t, int8_weights=bool(flags & P.FLAG_INT8_WEIGHTS))
    dl = G.DeviceLayer(shape, t, flags=flags)
    try:
        if budget is not None:
            dl.layer.set_prefetch_bytes(budget)
        k_before, v_before = G.cuda_to_bits(dl.k_cache), G.cuda_to_bits(dl.v_cache)
        dl.run()
        assert dl.layer.last_status() == P.PRESERVE_OK
        out, inter = dl.outputs(), dl.intermediates()
        k_new, v_new = dl.appended_kv()
        for name in ("h", "x", "q", "o", "x2", "a"):
            G.assert_close(inter[name], ref[name], f"{shape.name}:{name}")
        G.assert_close(k_new, ref["k_new"], f"{shape.name}:k_new")
        G.assert_close(v_new, ref["v_new"], f"{shape.name}:v_new")
        for name in ("attn_partial", "h2", "mlp_partial"):
            G.assert_close(out[name], ref[name], f"{shape.name}:{name}")
        for g in (dl.residual_out, dl.mlp_out, dl.attn_out):
            assert g.guards_intact(), "write outside an output buffer"
        # append: exactly one slot per (sequence, kv head) changed in each cache
        k_after, v_after = G.cuda_to_bits(dl.k_cache), G.cuda_to_bits(dl.v_cache)
        mask = np.ones(k_before.shape, bool)
        for b in range(shape.batch):
            mask[b, :, int(t["ctx_len"][b])] = False
        assert np.array_equal(k_before[mask], k_after[mask]) and np.array_equal(v_before[mask], v_after[mask])
        assert not np.isnan(I.bf16_bits_to_f32(k_after[~mask])).any()
        return dl.output_bits()
    finally:
        dl.close()


SMALL = [
    I.small_shape(name="b1_mha", batch=1, tp_degree=1, ctx=37, n_q_heads=2, n_kv_heads=2, seed=12),
    I.small_shape(name="b2", batch=2, ctx=64, seed=40),
    I.small_shape(name="b3", batch=3, ctx=200, seed=11),
    I.small_shape(name="b4_g4", batch=4, ctx=63, n_q_heads=4, n_kv_heads=1, seed=41),
    I.small_shape(name="b5", batch=5, ctx=127, seed=42),
    I.small_shape(name="b8_ragged", batch=8, ctx=300, ctx_min=10, tp_degree=4, seed=13),
    I.small_shape(name="b12_g8", batch=12, ctx=130, n_q_heads=8, n_kv_heads=1, seed=14),
    I.small_shape(name="b15_g16", batch=15, ctx=65, n_q_heads=16, n_kv_heads=1, tp_degree=16, seed=43),
    I.small_shape(name="b16", batch=16, ctx=100, seed=15),
    I.small_shape(name="b33_ragged_g8", batch=33, ctx=300, ctx_min=1, n_q_heads=8, n_kv_heads=1, tp_degree=3, seed=16),
    I.small_shape(name="b64", batch=64, hidden=1024, ffn=1152, ctx=64, seed=17),
    I.small_shape(name="b128", batch=128, hidden=256, ffn=128, ctx=20, n_q_heads=2, n_kv_heads=2, seed=44),
    I.small_shape(name="no_rope", batch=3, ctx=90, rope_theta=0.0, seed=45),
    I.small_shape(name="ctx0", batch=2, ctx=0, seed=46),
    I.small_shape(name="ctx63", batch=2, ctx=63, seed=47),     # 64 keys: exactly one tile
    I.small_shape(name="long_multi_tile_items", batch=2, n_q_heads=4, n_kv_heads=2, ctx=20000, seed=18),
    # gate/up with more row-block groups than CTAs (a CTA loops over several groups)
    I.small_shape(name="wide_ffn_b8", batch=8, hidden=256, ffn=5120, ctx=70, seed=48),
    # 24 / 28 row blocks: one row block per warp, k split over a cluster with the one-sided reduction
    I.small_shape(name="h384_b7", batch=7, hidden=384, ffn=224, ctx=33, seed=49),
    # window rows split over a cluster of CTAs
    I.small_shape(name="h2048_b3", batch=3, hidden=2048, ffn=256, ctx=40, tp_degree=5, seed=50),
    # 40 rows x 8 CTAs: the window kernel's big-batch form (inputs loaded after the wait); tensor path with a
    # 48-column batch tile, two weight tiles per CTA and the bulk split-K hand-over
    I.small_shape(name="h8192_b40", batch=40, hidden=8192, ffn=256, ctx=50, ctx_min=3, n_q_heads=2, n_kv_heads=2,
                  tp_degree=3, seed=57),
]


@pytest.mark.parametrize("shape", SMALL, ids=[s.name for s in SMALL])
def test_small_shapes_match_oracle(oracle, shape):
    full_check(oracle, shape)


@pytest.mark.parametrize("idx", [0, 1, 3, 4])
def test_benchmark_configs_match_oracle(oracle, idx):
    # (with the side-stream L2 prefetch running: a budget of 16 MiB per window; the library's default
    # plans nothing for L2 and is what the small shapes above run with)
    full_check(oracle, I.CONFIGS[idx], budget=16 << 20)


W8_SHAPES = [
    I.small_shape(name="w8_b1", batch=1, tp_degree=1, ctx=37, n_q_heads=2, n_kv_heads=2, seed=112),
    I.small_shape(name="w8_b2", batch=2, ctx=64, seed=140),
    I.small_shape(name="w8_b3", batch=3, ctx=200, seed=111),
    I.small_shape(name="w8_b4_g4", batch=4, ctx=63, n_q_heads=4, n_kv_heads=1, seed=141),
    I.small_shape(name="w8_b8_ragged", batch=8, ctx=300, ctx_min=10, tp_degree=4, seed=113),
    I.small_shape(name="w8_b15_g16", batch=15, ctx=65, n_q_heads=16, n_kv_heads=1, tp_degree=16, seed=143),
    I.small_shape(name="w8_wide_ffn_b8", batch=8, hidden=256, ffn=5120, ctx=70, seed=148),
    I.small_shape(name="w8_h384_b7", batch=7, hidden=384, ffn=192, ctx=33, seed=149),
    I.small_shape(name="w8_h2048_b3", batch=3, hidden=2048, ffn=256, ctx=40, tp_degree=5, seed=150),
    # tensor path: the int8 tiles are widened in shared memory in front of the tcgen05 MMA
    I.small_shape(name="w8_b16", batch=16, ctx=100, seed=115),
    I.small_shape(name="w8_b33_ragged_g8", batch=33, ctx=300, ctx_min=1, n_q_heads=8, n_kv_heads=1, tp_degree=3, seed=116),
    I.small_shape(name="w8_b64", batch=64, hidden=1024, ffn=1152, ctx=64, seed=117),
    I.small_shape(name="w8_b128", batch=128, hidden=256, ffn=128, ctx=20, n_q_heads=2, n_kv_heads=2, seed=144),
    I.small_shape(name="w8_h8192_b40", batch=40, hidden=8192, ffn=256, ctx=50, ctx_min=3, n_q_heads=2, n_kv_heads=2,
                  tp_degree=3, seed=157),
]


@pytest.mark.parametrize("shape", W8_SHAPES, ids=[s.name for s in W8_SHAPES])
def test_int8_weights_match_the_quantised_oracle(oracle, shape):
    """int8 weights (per-output-channel scales) on the split-K GEMV path and on the tcgen05 path against
    the oracle that quantises the same way: every intermediate and output, same tolerance."""
    full_check(oracle, shape, flags=P.FLAG_INT8_WEIGHTS)


@pytest.mark.parametrize("idx", [0, 1, 3, 4])
def test_int8_weights_on_benchmark_configs(oracle, idx):
    bits = full_check(oracle, I.CONFIGS[idx], flags=P.FLAG_INT8_WEIGHTS, budget=16 << 20)
    again = full_check(oracle, I.CONFIGS[idx], flags=P.FLAG_INT8_WEIGHTS, budget=0)
    for k in bits:
        assert np.array_equal(bits[k], again[k]), k          # prefetch never changes results, int8 included


def test_int8_weights_on_either_path_report_one_byte_per_weight():
    for flags, tensor in ((P.FLAG_INT8_WEIGHTS, 1), (P.FLAG_INT8_WEIGHTS | P.FLAG_FORCE_GEMV, 0)):
        s = I.small_shape(batch=20, ctx=50, seed=151)
        dl = G.DeviceLayer(s, I.make_layers(s, 1)[0], flags=flags)
        try:
            info = dl.layer.get_info()
            assert info.uses_tensor_path == tensor
            assert list(info.weight_bytes) == [512 * 1024, 512 * 512, 512 * 768, 384 * 512]   # one byte per weight
        finally:
            dl.close()
    # the GEMV path's int8 tiles cover 64 k: an ffn that is not a multiple of 64 is refused
    s = I.small_shape(batch=2, ffn=96, ctx=10)
    with pytest.raises(P.PreserveError) as e:
        G.DeviceLayer(s, I.make_layers(s, 1)[0], flags=P.FLAG_INT8_WEIGHTS)
    assert e.value.code == P.PRESERVE_ESHAPE


def test_config3_chain_of_four_matches_oracle(oracle):
    shape = I.CONFIGS[2]
    layers = I.make_layers(shape)
    refs = oracle.layer_chain(shape, layers)
    dls = [G.DeviceLayer(shape, t) for t in layers]
    try:
        P.preserve_decode_chain([d.layer for d in dls], [d.io for d in dls], link=True)
        for i, (dl, ref) in enumerate(zip(dls, refs)):
            assert dl.layer.last_status() == P.PRESERVE_OK
            out = dl.outputs()
            for name in ("attn_partial", "h2", "mlp_partial"):
                G.assert_close(out[name], ref[name], f"chain layer {i}:{name}")
    finally:
        for d in dls:
            d.close()


def test_prefetch_never_changes_results(oracle):
    """Outputs are bit-identical across prefetch off, on, every swept budget, both planning
    modes, graph replay vs direct launches, and repeated runs."""
    for shape in (I.small_shape(name="det_gemv", batch=8, ctx=500, ctx_min=20, seed=50),
                  I.small_shape(name="det_tc", batch=32, ctx=700, ctx_min=5, hidden=1024, ffn=512, seed=51),
                  I.CONFIGS[1]):
        t = I.make_layers(shape, 1)[0]
        base = None
        stream = torch.cuda.Stream()      # (on the legacy default stream every step is launched directly)
        for flags in (0, P.FLAG_NO_GRAPH):
            dl = G.DeviceLayer(shape, t, flags=flags)
            try:
                l2 = int(dl.layer.get_info().l2_bytes)
                for mode in (P.PLAN_TRUNCATE, P.PLAN_WHOLE_NODE):
                    dl.layer.set_plan_mode(mode)
                    for frac in (0.0, 1 / 16, 1 / 4, 1 / 2, 1.0, 2.0):
                        dl.layer.set_prefetch_bytes(int(frac * l2))
                        for _ in range(2):
                            with torch.cuda.stream(stream):
                                dl.run(stream)
                            bits = dl.output_bits()
                            if base is None:
                                base = bits
                            for k in base:
                                assert np.array_equal(base[k], bits[k]), (shape.name, flags, mode, frac, k)
            finally:
                dl.close()


def test_schedule_variants_do_not_change_results(oracle):
    """Early launch off (ablation flag), a modelled window latency and the timeline trace change
    when kernels run, never what they compute."""
    shape = I.small_shape(name="sched", batch=7, ctx=400, ctx_min=9, seed=55)
    t = I.make_layers(shape, 1)[0]
    ref = oracle.layer_step(shape, t)
    base = None
    for flags in (0, P.FLAG_NO_EARLY_LAUNCH, P.FLAG_NO_GRAPH | P.FLAG_NO_EARLY_LAUNCH):
        dl = G.DeviceLayer(shape, t, flags=flags)
        try:
            for delay, trace in ((0, False), (5000, False), (0, True)):
                dl.layer.set_window_delay_ns(delay)
                dl.layer.set_trace(trace)
                dl.run()
                bits = dl.output_bits()
                if base is None:
                    base = bits
                    for name in ("attn_partial", "h2", "mlp_partial"):
                        G.assert_close(dl.outputs()[name], ref[name], name)
                for k in base:
                    assert np.array_equal(base[k], bits[k]), (flags, delay, trace, k)
                if trace:
                    tr = dl.layer.read_trace()
                    assert len(tr) == len(P.KERNEL_NAMES)
                    assert all(len(r) == P.TRACE_SLOTS for r in tr)
                    ends = [r[3] for r in tr]
                    assert all(s <= w1 <= w2 <= e and s <= s2 <= e and e1 <= e
                               for (s, w1, w2, e, s2, _, e1, _) in tr)
                    assert ends == sorted(ends)            # the main-stream kernels finish in order
            assert dl.layer.last_status() == P.PRESERVE_OK
        finally:
            dl.close()


def test_single_kernel_entry_point_reproduces_the_step(oracle):
    shape = I.small_shape(name="single", batch=4, ctx=120, seed=56)
    t = I.make_layers(shape, 1)[0]
    dl = G.DeviceLayer(shape, t)
    try:
        dl.run()
        want = dl.output_bits()
        dl.mlp_out.t.zero_()
        for k in range(len(P.KERNEL_NAMES)):
            dl.layer.run_kernel(dl.io, k)
        got = dl.output_bits()
        for name in want:
            assert np.array_equal(want[name], got[name]), name
        ms = dl.layer.profile_step(dl.io)
        assert len(ms) == len(P.KERNEL_NAMES) and all(v >= 0 for v in ms)
    finally:
        dl.close()


def test_host_buffer_entry_point_matches_device_path(oracle):
    shape = I.small_shape(name="host_io", batch=6, ctx=150, ctx_min=3, seed=52)
    t = I.make_layers(shape, 1)[0]
    dl = G.DeviceLayer(shape, t)
    try:
        dl.run()
        want = dl.output_bits()
        # restore the caches (the step appended), then run from pinned host buffers
        dl.k_cache.copy_(G.bits_to_cuda(t["k_cache"]))
        dl.v_cache.copy_(G.bits_to_cuda(t["v_cache"]))
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
        parts = [pin(t["partials_in"][p]) for p in range(shape.tp_degree)]
        peers = [pin(t["attn_peer_partials"][p]) for p in range(shape.tp_degree - 1)]
        resid = pin(t["residual_in"])
        r_out = torch.zeros((shape.batch, shape.hidden), dtype=torch.int16).pin_memory()
        m_out = torch.zeros((shape.batch, shape.hidden), dtype=torch.int16).pin_memory()
        hio = P.make_host_io(dl.cfg, shape.batch, dl.ctx_host, parts, peers, resid, dl.k_cache, dl.v_cache,
                             r_out, m_out)
        dl.layer.decode_step_host(hio)
        torch.cuda.synchronize()
        assert np.array_equal(r_out.numpy().view(np.uint16), want["h2"])
        assert np.array_equal(m_out.numpy().view(np.uint16), want["mlp_partial"])
        # twice in a row on one layer (the second call's gather must wait for the first call's step),
        # then from pageable buffers (copy calls instead of the gather kernel and the direct stores)
        for pinned in (True, True, False):
            dl.k_cache.copy_(G.bits_to_cuda(t["k_cache"]))
            dl.v_cache.copy_(G.bits_to_cuda(t["v_cache"]))
            mk = pin if pinned else (lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16).copy()))
            parts2 = [mk(t["partials_in"][p]) for p in range(shape.tp_degree)]
            peers2 = [mk(t["attn_peer_partials"][p]) for p in range(shape.tp_degree - 1)]
            resid2 = mk(t["residual_in"])
            r2 = torch.zeros((shape.batch, shape.hidden), dtype=torch.int16)
            m2 = torch.zeros((shape.batch, shape.hidden), dtype=torch.int16)
            if pinned:
                r2, m2 = r2.pin_memory(), m2.pin_memory()
            hio2 = P.make_host_io(dl.cfg, shape.batch, dl.ctx_host, parts2, peers2, resid2, dl.k_cache, dl.v_cache,
                                  r2, m2)
            dl.layer.decode_step_host(hio2)
            torch.cuda.synchronize()
            assert np.array_equal(r2.numpy().view(np.uint16), want["h2"]), f"pinned={pinned}"
            assert np.array_equal(m2.numpy().view(np.uint16), want["mlp_partial"]), f"pinned={pinned}"
    finally:
        dl.close()


def test_smaller_batch_than_max_batch(oracle):
    shape = I.small_shape(name="b5_of_12", batch=5, ctx=77, seed=53)
    t = I.make_layers(shape, 1)[0]
    ref = oracle.layer_step(shape, t)
    for max_batch in (12, 40):                     # GEMV path and tensor path
        dl = G.DeviceLayer(shape, t, max_batch=max_batch)
        try:
            # caches are [max_batch, ...] for the library: rebuild them at that size
            cap, d, nkv = shape.kv_capacity, shape.head_dim, shape.n_kv_heads
            kc = torch.zeros((max_batch, nkv, cap, d), dtype=torch.bfloat16, device="cuda")
            vc = torch.zeros_like(kc)
            kc[:shape.batch] = G.bits_to_cuda(t["k_cache"])
            vc[:shape.batch] = G.bits_to_cuda(t["v_cache"])
            dl.k_cache, dl.v_cache = kc, vc
            dl.io = dl.layer.make_io(shape.batch, dl.ctx_dev, dl.ctx_host, dl.partials, dl.peers, dl.residual,
                                     kc, vc, dl.residual_out.t, dl.mlp_out.t, dl.attn_out.t)
            dl.run()
            assert dl.layer.last_status() == P.PRESERVE_OK
            out = dl.outputs()
            for name in ("attn_partial", "h2", "mlp_partial"):
                G.assert_close(out[name], ref[name], f"max_batch {max_batch}:{name}")
        finally:
            dl.close()


def test_argument_validation_on_device():
    shape = I.small_shape(name="args", batch=2, ctx=10, seed=54)
    t = I.make_layers(shape, 1)[0]
    dl = G.DeviceLayer(shape, t)
    try:
        import ctypes as C
        lib = P.lib()
        io = dl.io
        good_batch = io.batch
        io.batch = 3                                     # > max_batch
        assert lib.preserve_decode_step(dl.layer.handle, C.byref(io), 0) == P.PRESERVE_ESHAPE
        io.batch = good_batch
        keep = io.residual_in
        io.residual_in = keep + 2                        # misaligned
        assert lib.preserve_decode_step(dl.layer.handle, C.byref(io), 0) == P.PRESERVE_EALIGN
        io.residual_in = None
        assert lib.preserve_decode_step(dl.layer.handle, C.byref(io), 0) == P.PRESERVE_EINVAL
        io.residual_in = keep
        bad_ctx = np.array([5, shape.ctx + 1], np.int32)  # beyond max_ctx
        old = io.ctx_len_host
        io.ctx_len_host = bad_ctx.ctypes.data
        assert lib.preserve_decode_step(dl.layer.handle, C.byref(io), 0) == P.PRESERVE_ESHAPE
        io.ctx_len_host = old
        assert lib.preserve_decode_step(None, C.byref(io), 0) == P.PRESERVE_EINVAL
        dl.run()                                         # still usable afterwards
        assert dl.layer.last_status() == P.PRESERVE_OK
    finally:
        dl.close()
    for bad in (replace(shape, head_dim=64), replace(shape, hidden=520), replace(shape, ffn=100),
                replace(shape, n_q_heads=3), replace(shape, tp_degree=17)):
        with pytest.raises(P.PreserveError) as e:
            G.DeviceLayer(bad, t)
        assert e.value.code == P.PRESERVE_ESHAPE


def test_info_reports_plan_and_bytes():
    shape = I.CONFIGS[1]
    t = I.make_layers(shape, 1)[0]
    dl = G.DeviceLayer(shape, t)
    try:
        dl.layer.set_plan_mode(P.PLAN_WHOLE_NODE)
        dl.layer.set_prefetch_bytes(32 << 20)
        dl.run()
        torch.cuda.synchronize()
        info = dl.layer.get_info()
        assert list(info.weight_bytes) == [6291456, 4194304, 29360128, 14680064]
        assert info.kv_bytes == 16777216
        assert [list(r) for r in info.planned_bytes] == [[6291456, 16777216, 4194304], [29360128, 0, 0]]
        assert info.algorithmic_bytes == P.preserve_algorithmic_bytes(dl.cfg, shape.batch, shape.batch * shape.ctx)
        assert info.sm_count > 0 and info.l2_bytes > 0 and info.uses_tensor_path == 0
    finally:
        dl.close()
