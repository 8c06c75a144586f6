"""The allocation-free attention entry point (preserve_attention_static) against the layer
path's attention.  Collected last on purpose: if it fails, a run that stops at the first
failure has already run every other test.

Why the entry point exists: a caller that is not allowed to allocate device memory when it
needs attention (a memory-frozen serving step, a plug-in without an allocator, a caller that
is capturing a stream) cannot use a handle whose workspaces come from cudaMalloc, so this
variant keeps its split-KV partials in a fixed array inside the library image.  All calls
share that array and it keeps the previous call's contents, so the test runs two different
problems back to back and checks both."""
import numpy as np
import pytest
import torch

from paper_2501_08192_b200 import binding as P
from paper_2501_08192_b200 import inputs as I

import gpu_util as G

pytestmark = pytest.mark.gpu


def layer_attention_reference(shape):
    """Run one full step through preserve_decode_step and return what its attention consumed and
    produced: q planes, the caches after the append, ctx_len, and o planes."""
    t = I.make_layers(shape, 1)[0]
    dl = G.DeviceLayer(shape, t)
    try:
        dl.run()
        assert dl.layer.last_status() == P.PRESERVE_OK
        rows = int(dl.layer.get_info().activation_rows)
        q = torch.empty((2, rows, shape.n_q_heads, shape.head_dim), dtype=torch.bfloat16, device="cuda")
        o = torch.empty_like(q)
        dl.layer.debug_copy(2, q)
        dl.layer.debug_copy(3, o)
        torch.cuda.synchronize()
        B = shape.batch
        return (q[0, :B].contiguous(), q[1, :B].contiguous(), dl.k_cache.clone(), dl.v_cache.clone(),
                dl.ctx_dev.clone(), dl.ctx_host.copy(), o[0, :B].float() + o[1, :B].float())
    finally:
        dl.close()


def run_static(shape, q_hi, q_lo, kc, vc, ctx_dev, ctx_host):
    o_hi = torch.full_like(q_hi, float("nan"))
    o_lo = torch.full_like(q_hi, float("nan"))
    before = torch.cuda.memory_allocated()
    rc = P.preserve_attention_static(q_hi, q_lo, kc, vc, ctx_dev, ctx_host, shape.n_q_heads, shape.n_kv_heads,
                                     o_hi, o_lo)
    assert rc == P.PRESERVE_OK, P.preserve_strerror(rc)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    return o_hi.float() + o_lo.float()


def test_static_attention_matches_layer_path_twice_in_a_row():
    big = I.small_shape(name="static_big", batch=6, ctx=700, ctx_min=30, n_q_heads=8, n_kv_heads=2, seed=61)
    small = I.small_shape(name="static_small", batch=2, ctx=70, n_q_heads=4, n_kv_heads=4, seed=62)
    cases = [(s, layer_attention_reference(s)) for s in (big, small)]
    # two calls in a row on the shared scratch array: a larger problem first, then a smaller one
    for shape, (q_hi, q_lo, kc, vc, ctx_dev, ctx_host, o_ref) in cases:
        got = run_static(shape, q_hi, q_lo, kc, vc, ctx_dev, ctx_host)
        G.assert_close(got.cpu().numpy(), o_ref.cpu().numpy(), f"{shape.name}:o")
    # and once more in the opposite order, so each problem also follows the other's leftovers
    for shape, (q_hi, q_lo, kc, vc, ctx_dev, ctx_host, o_ref) in reversed(cases):
        got = run_static(shape, q_hi, q_lo, kc, vc, ctx_dev, ctx_host)
        G.assert_close(got.cpu().numpy(), o_ref.cpu().numpy(), f"{shape.name}:o (second round)")


def test_static_attention_matches_the_oracle_directly(oracle):
    """The same entry point against the CPU oracle's attention on inputs drawn here (no layer path
    in between): plain bf16 queries (zero lo plane), ragged lengths, two calls in a row."""
    rng = np.random.default_rng(63)
    for B, nq, nkv, cap, lens in ((5, 8, 2, 900, (899, 1, 64, 63, 500)), (2, 4, 4, 130, (129, 77))):
        q_bits = I.f32_to_bf16_bits(rng.standard_normal((B, nq, 128), dtype=np.float32))
        k_bits = I.f32_to_bf16_bits(rng.standard_normal((B, nkv, cap, 128), dtype=np.float32))
        v_bits = I.f32_to_bf16_bits(rng.standard_normal((B, nkv, cap, 128), dtype=np.float32))
        ctx = np.array(lens, np.int32) - 1                  # the newest entry is already in the cache
        for b in range(B):
            k_bits[b, :, lens[b]:] = I.BF16_NAN
            v_bits[b, :, lens[b]:] = I.BF16_NAN
        # oracle: attends over slots 0..ctx[b]-1 of the cache plus the "new" entry = slot ctx[b]
        k_new = np.stack([I.bf16_bits_to_f32(k_bits[b, :, ctx[b]]) for b in range(B)])
        v_new = np.stack([I.bf16_bits_to_f32(v_bits[b, :, ctx[b]]) for b in range(B)])
        want = oracle.attention(I.bf16_bits_to_f32(q_bits), k_new, v_new, k_bits, v_bits, ctx)
        q_hi = G.bits_to_cuda(q_bits)
        q_lo = torch.zeros_like(q_hi)
        kc, vc = G.bits_to_cuda(k_bits), G.bits_to_cuda(v_bits)
        ctx_dev = torch.from_numpy(ctx).cuda()
        shape = I.small_shape(name="static_direct", batch=B, n_q_heads=nq, n_kv_heads=nkv, ctx=cap - 1)
        got = run_static(shape, q_hi, q_lo, kc, vc, ctx_dev, ctx)
        assert P.preserve_attention_static_status() == P.PRESERVE_OK
        G.assert_close(got.cpu().numpy(), want, f"static vs oracle B={B}")


def test_static_attention_rejects_what_does_not_fit():
    # 16 query heads per KV head and 1024 (sequence, kv head) streams need far more than the fixed array
    B, nq, nkv, cap = 128, 128, 8, 2
    z = torch.zeros((B, nq, 128), dtype=torch.bfloat16, device="cuda")
    kc = torch.zeros((B, nkv, cap, 128), dtype=torch.bfloat16, device="cuda")
    ctx_host = np.zeros(B, np.int32)
    ctx_dev = torch.zeros(B, dtype=torch.int32, device="cuda")
    rc = P.preserve_attention_static(z, z, kc, kc, ctx_dev, ctx_host, nq, nkv, z.clone(), z.clone())
    assert rc == P.PRESERVE_ETOOBIG
    assert "scratch" in P.preserve_strerror(rc)
    # bad arguments are refused before anything is queued
    assert P.preserve_attention_static(z, z, kc, kc, ctx_dev, np.full(B, cap, np.int32), nq, nkv, z, z) == P.PRESERVE_ESHAPE
    assert P.preserve_attention_static(z, None, kc, kc, ctx_dev, ctx_host, nq, nkv, z, z) == P.PRESERVE_EINVAL
