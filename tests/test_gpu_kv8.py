"""GPU parity of the int8 KV-cache path (one fp32 scale per cached vector) against the oracle that
quantises the same way.  Same tolerance as test_gpu_parity.py.  The codes of the entry a step
appends are decided from fp32 vectors that the GPU and the oracle compute in different summation
orders, so they may differ by one unit where a value sits on a rounding boundary: the test checks
that they differ by at most one, that almost all agree, and that the stored entry is a valid
quantisation of the GPU's own vector (its largest code is +-127)."""
import numpy as np
import pytest
import torch

from paper_2501_08192_b200 import binding as P
from paper_2501_08192_b200 import inputs as I

import gpu_util as G

pytestmark = pytest.mark.gpu


def check_appended(dl, ref, name):
    kq, ks, vq, vs = dl.appended_kv8()
    for got_q, got_s, rq, rs, rv, what in ((kq, ks, ref["k_codes_new"], ref["k_scale_new"], ref["k_new"], "k"),
                                           (vq, vs, ref["v_codes_new"], ref["v_scale_new"], ref["v_new"], "v")):
        diff = np.abs(got_q.astype(np.int32) - rq.astype(np.int32))
        assert diff.max() <= 1, f"{name}:{what} codes differ by {diff.max()}"
        assert (diff != 0).mean() < 0.02, f"{name}:{what} {(diff != 0).mean():.3f} of the codes differ"
        assert np.allclose(got_s, rs, rtol=2e-3), f"{name}:{what} scales"
        assert (np.abs(got_q.astype(np.int32)).max(-1) == 127).all(), f"{name}:{what} no extreme code"
        # the stored entry is within half a quantisation step of the vector, whose own tolerance is the usual one
        rv64 = rv.astype(np.float64)
        err = np.abs(got_q.astype(np.float64) * got_s[..., None].astype(np.float64) - rv64)
        bound = 0.5 * got_s[..., None] + 2e-2 * min(1.0, float(np.sqrt((rv64 ** 2).mean()))) + 1e-2 * np.abs(rv64)
        assert (err <= bound).all(), f"{name}:{what} stored entry off by {float((err / bound).max()):.3f} of the bound"


def kv8_check(oracle, shape, flags=0, budget=None, cache_seed=0):
    t = I.make_layers(shape, 1)[0]
    kv = I.make_int8_cache(shape, t["ctx_len"], seed=cache_seed)
    ref = oracle.layer_step(shape, t, int8_weights=bool(flags & P.FLAG_INT8_WEIGHTS), kv8=kv)
    dl = G.DeviceLayer(shape, t, flags=flags, kv8=kv)
    try:
        if budget is not None:
            dl.layer.set_prefetch_bytes(budget)
        before = [b.clone() for b in (dl.k_cache, dl.v_cache)]
        dl.run()
        assert dl.layer.last_status() == P.PRESERVE_OK
        assert dl.layer.last_status_code() == 0
        out, inter = dl.outputs(), dl.intermediates()
        for name in ("h", "x", "q", "o", "x2", "a"):
            G.assert_close(inter[name], ref[name], f"{shape.name}:{name}")
        for name in ("attn_partial", "h2", "mlp_partial"):
            G.assert_close(out[name], ref[name], f"{shape.name}:{name}")
        for g in (dl.residual_out, dl.mlp_out, dl.attn_out):
            assert g.guards_intact(), "write outside an output buffer"
        check_appended(dl, ref, shape.name)
        # append: exactly one slot (its codes and its scale) per (sequence, kv head) changed in each buffer
        s = shape
        for buf, old in zip((dl.k_cache, dl.v_cache), before):
            c1, s1 = G.kv8_read(dl.cfg, buf, s.batch, s.n_kv_heads, s.kv_capacity, s.head_dim)
            c0, s0 = G.kv8_read(dl.cfg, old, s.batch, s.n_kv_heads, s.kv_capacity, s.head_dim)
            mask = np.ones(s0.shape, bool)
            for b in range(s.batch):
                mask[b, :, int(t["ctx_len"][b])] = False
            assert np.array_equal(c0[mask], c1[mask])
            assert np.array_equal(s0[mask].view(np.uint32), s1[mask].view(np.uint32))
            assert np.isfinite(s1[~mask]).all()
        return dl.output_bits()
    finally:
        dl.close()


KV8_SHAPES = [
    I.small_shape(name="kv8_b1_mha", batch=1, tp_degree=1, ctx=37, n_q_heads=2, n_kv_heads=2, seed=212),
    I.small_shape(name="kv8_b2_ctx64", batch=2, ctx=64, seed=240),          # the new key opens a second tile
    I.small_shape(name="kv8_b2_ctx63", batch=2, ctx=63, seed=247),          # the new key is the last of its tile
    I.small_shape(name="kv8_ctx0", batch=2, ctx=0, seed=246),               # nothing cached yet
    I.small_shape(name="kv8_b3", batch=3, ctx=200, seed=211),
    I.small_shape(name="kv8_b4_g4", batch=4, ctx=63, n_q_heads=4, n_kv_heads=1, seed=241),
    I.small_shape(name="kv8_b8_ragged", batch=8, ctx=300, ctx_min=10, tp_degree=4, seed=213),
    I.small_shape(name="kv8_b12_g8", batch=12, ctx=130, n_q_heads=8, n_kv_heads=1, seed=214),
    I.small_shape(name="kv8_b16", batch=16, ctx=100, seed=215),              # tensor path
    I.small_shape(name="kv8_b33_ragged_g8", batch=33, ctx=300, ctx_min=1, n_q_heads=8, n_kv_heads=1, tp_degree=3, seed=216),
    I.small_shape(name="kv8_b64", batch=64, hidden=1024, ffn=1152, ctx=64, seed=217),
    I.small_shape(name="kv8_no_rope", batch=3, ctx=90, rope_theta=0.0, seed=245),
    I.small_shape(name="kv8_long_multi_tile_items", batch=2, n_q_heads=4, n_kv_heads=2, ctx=20000, seed=218),
]


@pytest.mark.parametrize("shape", KV8_SHAPES, ids=[s.name for s in KV8_SHAPES])
def test_int8_cache_matches_the_quantised_oracle(oracle, shape):
    kv8_check(oracle, shape)


@pytest.mark.parametrize("idx", [0, 1, 3, 4])
def test_int8_cache_on_benchmark_configs(oracle, idx):
    bits = kv8_check(oracle, I.CONFIGS[idx], budget=16 << 20)
    if idx in (1, 3):
        again = kv8_check(oracle, I.CONFIGS[idx], budget=0)
        for k in bits:
            assert np.array_equal(bits[k], again[k]), k          # prefetch never changes results


def test_int8_cache_with_int8_weights(oracle):
    kv8_check(oracle, I.small_shape(name="kv8_w8_b5", batch=5, ctx=127, seed=242), flags=P.FLAG_INT8_WEIGHTS)
    kv8_check(oracle, I.CONFIGS[1], flags=P.FLAG_INT8_WEIGHTS)
    kv8_check(oracle, I.small_shape(name="kv8_w8_b24", batch=24, ctx=127, seed=243), flags=P.FLAG_INT8_WEIGHTS)   # tensor path


def test_int8_cache_groups_above_eight_are_refused():
    s = I.small_shape(batch=2, ctx=20, n_q_heads=16, n_kv_heads=1, tp_degree=1)
    t = I.make_layers(s, 1)[0]
    with pytest.raises(P.PreserveError) as e:
        G.DeviceLayer(s, t, kv8=I.make_int8_cache(s, t["ctx_len"]))
    assert e.value.code == P.PRESERVE_ESHAPE


def test_int8_cache_decode_loop_advances_over_a_tile_boundary(oracle):
    """Twelve steps with the contexts advancing (one sequence crosses from 62 to 74 keys, i.e. over a
    tile boundary): the GPU's cache evolves by its own appends, the oracle's by its own; every step's
    outputs agree, one graph serves all steps, and the device plan follows the live lengths."""
    shape = I.small_shape(name="kv8_loop", batch=3, ctx=90, seed=250)
    t = I.make_layers(shape, 1)[0]
    start = np.array([60, 5, 33], np.int32)
    first = start.copy()          # (the device layer keeps and updates its own copy of the lengths)
    kv = I.make_int8_cache(shape, first, seed=3)
    dl = G.DeviceLayer(shape, dict(t, ctx_len=first), kv8=kv)
    stream = torch.cuda.Stream()
    try:
        okv = {k: v.copy() for k, v in kv.items()}
        for step in range(12):
            ctx = start + step
            ref = oracle.layer_step(shape, dict(t, ctx_len=ctx), kv8=okv)
            for b in range(shape.batch):          # the oracle's own append
                okv["k_codes"][b, :, ctx[b]] = ref["k_codes_new"][b]
                okv["v_codes"][b, :, ctx[b]] = ref["v_codes_new"][b]
                okv["k_scales"][b, :, ctx[b]] = ref["k_scale_new"][b]
                okv["v_scales"][b, :, ctx[b]] = ref["v_scale_new"][b]
            dl.ctx_host[:] = ctx
            dl.ctx_dev.copy_(torch.from_numpy(ctx))
            torch.cuda.synchronize()
            with torch.cuda.stream(stream):
                dl.run(stream)
            stream.synchronize()
            assert dl.layer.last_status_code() == 0
            out = dl.outputs()
            for name in ("attn_partial", "h2", "mlp_partial"):
                G.assert_close(out[name], ref[name], f"step {step}: {name}")
            G.assert_close(dl.intermediates()["o"], ref["o"], f"step {step}: o")
        assert dl.layer.graph_captures() == 1
    finally:
        dl.close()


def test_int8_cache_withheld_copy_ends_with_a_status(oracle):
    """The producer of CTA 0 never fetches the key box of its first tile: the consumers' bounded wait
    gives up, the step returns with a time-out status, and the handle works again afterwards."""
    shape = I.small_shape(name="kv8_withhold", batch=2, ctx=100, seed=251)
    t = I.make_layers(shape, 1)[0]
    kv = I.make_int8_cache(shape, t["ctx_len"])
    ref = oracle.layer_step(shape, t, kv8=kv)
    dl = G.DeviceLayer(shape, t, kv8=kv)
    try:
        dl.layer.debug_set(P.DEBUG_WAIT_LIMIT_CYCLES, 1 << 21)
        dl.layer.debug_set(P.DEBUG_WITHHOLD, P.WITHHOLD_ATTENTION)
        dl.run()
        torch.cuda.synchronize()
        assert dl.layer.last_status() == P.PRESERVE_ETIMEOUT
        dl.layer.debug_set(P.DEBUG_WITHHOLD, 0)
        dl.layer.clear_status()
        dl.run()
        assert dl.layer.last_status() == P.PRESERVE_OK
        G.assert_close(dl.outputs()["mlp_partial"], ref["mlp_partial"], "after the time-out")
    finally:
        dl.close()


def test_int8_cache_layout_and_byte_accounting():
    s = I.small_shape(batch=3, ctx=100, seed=252)
    cfg = P.make_config(s, flags=P.FLAG_INT8_KV)
    off, scap, total = P.preserve_kv8_layout(cfg)
    streams, cap = s.batch * s.n_kv_heads, s.ctx + 1
    assert off == (streams * cap * 128 + 255) // 256 * 256 and scap == 128 and total == off + streams * scap * 4
    t = I.make_layers(s, 1)[0]
    dl = G.DeviceLayer(s, t, kv8=I.make_int8_cache(s, t["ctx_len"]))
    try:
        dl.layer.set_prefetch_bytes(1 << 20)
        dl.run()
        info = dl.layer.get_info()
        sum_ctx = int(t["ctx_len"].sum())
        assert info.kv_bytes == 2 * sum_ctx * s.n_kv_heads * 128          # one byte per cached value
        assert info.algorithmic_bytes == P.preserve_algorithmic_bytes(cfg, s.batch, sum_ctx)
        plan = torch.zeros(6, dtype=torch.int64, device="cuda")
        dl.layer.debug_copy(6, plan)
        torch.cuda.synchronize()
        assert plan.cpu().numpy().reshape(2, 3).tolist() == [list(r) for r in info.planned_bytes]
    finally:
        dl.close()


@pytest.mark.parametrize("batch", [6, 24], ids=["gemv", "tensor"])
def test_int8_linked_chain_matches_the_oracle_chain(oracle, batch):
    """Three layers linked output to input (fp32 hand-over inside the library), int8 weights and int8
    cache together, against the oracle stepping the same chain."""
    shape = I.small_shape(name="kv8_w8_chain", batch=batch, ctx=140, ctx_min=20, layers=3, seed=260)
    layers = I.make_layers(shape)
    kvs = [I.make_int8_cache(shape, t["ctx_len"], seed=10 + i) for i, t in enumerate(layers)]
    refs = oracle.layer_chain(shape, layers, int8_weights=True, kv8=kvs)
    dls = [G.DeviceLayer(shape, t, flags=P.FLAG_INT8_WEIGHTS, kv8=kv) for t, kv in zip(layers, kvs)]
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


def test_int8_cache_with_a_smaller_batch_than_max_batch(oracle):
    """A step of 5 sequences on handles created for 12 (GEMV path) and 40 (tensor path): the cache buffers
    have the layout of the larger batch (streams of the first sequences first), int8 weights as well."""
    shape = I.small_shape(name="kv8_b5_of_more", batch=5, ctx=77, ctx_min=3, seed=253)
    t = I.make_layers(shape, 1)[0]
    kv = I.make_int8_cache(shape, t["ctx_len"])
    ref = oracle.layer_step(shape, t, int8_weights=True, kv8=kv)
    for max_batch in (12, 40):
        dl = G.DeviceLayer(shape, t, flags=P.FLAG_INT8_WEIGHTS, max_batch=max_batch, kv8=kv)
        try:
            dl.run()
            assert dl.layer.last_status() == P.PRESERVE_OK
            out = dl.outputs()
            for name in ("attn_partial", "h2", "mlp_partial"):
                G.assert_close(out[name], ref[name], f"max_batch {max_batch}:{name}")
            check_appended(dl, ref, f"max_batch {max_batch}")
        finally:
            dl.close()


def test_int8_host_buffer_entry_point_matches_the_device_path(oracle):
    """preserve_decode_step_host over the int8 cache with int8 weights (the cache stays on the device):
    bit-identical to the device-buffer call on the same inputs."""
    shape = I.small_shape(name="kv8_host_io", batch=6, ctx=150, ctx_min=3, seed=254)
    t = I.make_layers(shape, 1)[0]
    kv = I.make_int8_cache(shape, t["ctx_len"])
    dl = G.DeviceLayer(shape, t, flags=P.FLAG_INT8_WEIGHTS, kv8=kv)
    try:
        k0, v0 = dl.k_cache.clone(), dl.v_cache.clone()
        dl.run()
        want = dl.output_bits()
        dl.k_cache.copy_(k0)
        dl.v_cache.copy_(v0)
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
        parts = [pin(t["partials_in"][p]) for p in range(shape.tp_degree)]
        peers = [pin(t["attn_peer_partials"][p]) for p in range(shape.tp_degree - 1)]
        resid = pin(t["residual_in"])
        r_out = torch.zeros((shape.batch, shape.hidden), dtype=torch.int16).pin_memory()
        m_out = torch.zeros((shape.batch, shape.hidden), dtype=torch.int16).pin_memory()
        hio = P.make_host_io(dl.cfg, shape.batch, dl.ctx_host, parts, peers, resid, dl.k_cache, dl.v_cache, r_out, m_out)
        dl.layer.decode_step_host(hio)
        torch.cuda.synchronize()
        assert dl.layer.last_status() == P.PRESERVE_OK
        assert np.array_equal(r_out.numpy().view(np.uint16), want["h2"])
        assert np.array_equal(m_out.numpy().view(np.uint16), want["mlp_partial"])
    finally:
        dl.close()
