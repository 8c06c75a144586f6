"""Pins for the CPU oracle: closed forms, invariants, brute force and library
special cases that fix every step of the layer without reference to the oracle's
own code.  CPU only."""
import math

import numpy as np
import pytest
import torch

from paper_2501_08192_b200 import inputs as I


def bits(a):
    return I.f32_to_bf16_bits(np.asarray(a, np.float32))


def widen(b):
    return I.bf16_bits_to_f32(b)


# ----------------------------------------------------------------- bf16 helpers
def test_bf16_rounding_is_nearest_even():
    # 1 + 2^-8 lies halfway between bf16 neighbours 1.0 and 1 + 2^-7: ties to even -> 1.0
    assert widen(bits([1.0 + 2.0 ** -8]))[0] == 1.0
    # 1 + 3*2^-8 is halfway between 1+2^-7 (odd) and 1+2^-6 (even) -> 1 + 2^-6
    assert widen(bits([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    x = torch.randn(4096, dtype=torch.float32)
    ref = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits(x.numpy()), ref)
    assert np.array_equal(widen(ref), x.to(torch.bfloat16).float().numpy())


# ------------------------------------------------------------------- attention
def brute_attention(q, keys, vals):
    """q [d]; keys, vals [n][d] python lists -> softmax(q.K/sqrt(d)) V with plain loops."""
    d = len(q)
    s = [sum(q[i] * k[i] for i in range(d)) / math.sqrt(d) for k in keys]
    m = max(s)
    e = [math.exp(v - m) for v in s]
    z = sum(e)
    p = [v / z for v in e]
    return [sum(p[j] * vals[j][i] for j in range(len(keys))) for i in range(d)], p


def _tiny_case(B=2, nq=4, nkv=2, d=4, cap=9, lens=(5, 8), seed=3):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, nq, d)).astype(np.float32)
    kn = rng.standard_normal((B, nkv, d)).astype(np.float32)
    vn = rng.standard_normal((B, nkv, d)).astype(np.float32)
    kc = bits(rng.standard_normal((B, nkv, cap, d)))
    vc = bits(rng.standard_normal((B, nkv, cap, d)))
    return q, kn, vn, kc, vc, np.array(lens, np.int32)


def test_attention_brute_force_tiny(oracle):
    q, kn, vn, kc, vc, lens = _tiny_case()
    o, probs = oracle.attention(q, kn, vn, kc, vc, lens, want_probs=True)
    B, nq, d = q.shape
    nkv = kn.shape[1]
    G = nq // nkv
    for b in range(B):
        t = int(lens[b])
        for hq in range(nq):
            g = hq // G
            keys = [list(map(float, widen(kc[b, g, j]))) for j in range(t)] + [list(map(float, kn[b, g]))]
            vals = [list(map(float, widen(vc[b, g, j]))) for j in range(t)] + [list(map(float, vn[b, g]))]
            ref, p = brute_attention(list(map(float, q[b, hq])), keys, vals)
            np.testing.assert_allclose(o[b, hq], ref, rtol=1e-6, atol=1e-6)
            np.testing.assert_allclose(probs[b, hq, :t + 1], p, rtol=1e-6, atol=1e-7)
            assert abs(float(probs[b, hq, :t + 1].sum()) - 1.0) < 1e-6
            assert np.all(probs[b, hq, t + 1:] == 0)


def test_attention_does_not_read_past_length(oracle):
    q, kn, vn, kc, vc, lens = _tiny_case()
    o1 = oracle.attention(q, kn, vn, kc, vc, lens)
    kc2, vc2 = kc.copy(), vc.copy()
    for b in range(len(lens)):
        kc2[b, :, lens[b]:] = I.BF16_NAN
        vc2[b, :, lens[b]:] = I.BF16_NAN
    o2 = oracle.attention(q, kn, vn, kc2, vc2, lens)
    assert np.array_equal(o1, o2) and np.isfinite(o2).all()


def test_attention_equal_keys_gives_mean_of_values(oracle):
    q, kn, vn, kc, vc, lens = _tiny_case(B=1, nq=2, nkv=1, lens=(6,))
    key = bits(np.array([0.5, -1.0, 0.25, 2.0]))
    kc[:] = key
    kn[:] = widen(key)
    o = oracle.attention(q, kn, vn, kc, vc, lens)
    mean_v = (widen(vc[0, 0, :6]).astype(np.float64).sum(0) + vn[0, 0]) / 7.0
    for hq in range(2):
        np.testing.assert_allclose(o[0, hq], mean_v, rtol=1e-6, atol=1e-6)


def test_attention_equal_values_gives_that_row(oracle):
    q, kn, vn, kc, vc, lens = _tiny_case(B=1, nq=2, nkv=1, lens=(7,))
    row = bits(np.array([1.5, -0.75, 3.0, 0.125]))
    vc[:] = row
    vn[:] = widen(row)
    o = oracle.attention(q, kn, vn, kc, vc, lens)
    for hq in range(2):
        np.testing.assert_allclose(o[0, hq], widen(row), rtol=1e-6, atol=1e-6)


def test_attention_dominant_key_selects_its_value(oracle):
    q, kn, vn, kc, vc, lens = _tiny_case(B=1, nq=1, nkv=1, lens=(8,))
    q[0, 0] = np.array([1, 0, 0, 0], np.float32)
    kc[0, 0, :, :] = bits(np.zeros(4))
    kn[:] = 0
    kc[0, 0, 3] = bits(np.array([200.0, 0, 0, 0]))     # score 100 vs 0 elsewhere
    o = oracle.attention(q, kn, vn, kc, vc, lens)
    np.testing.assert_allclose(o[0, 0], widen(vc[0, 0, 3]), rtol=0, atol=1e-6)


def test_attention_attends_to_the_new_token(oracle):
    q, kn, vn, kc, vc, lens = _tiny_case(B=1, nq=1, nkv=1, lens=(5,))
    vc[:] = bits(np.zeros(4))
    o, p = oracle.attention(q, kn, vn, kc, vc, lens, want_probs=True)
    assert p[0, 0, 5] > 0
    np.testing.assert_allclose(o[0, 0], p[0, 0, 5] * vn[0, 0], rtol=1e-5, atol=1e-7)


def test_gqa_equals_mha_with_repeated_kv_heads(oracle):
    rng = np.random.default_rng(5)
    B, nq, nkv, d, cap = 2, 8, 2, 16, 33
    G = nq // nkv
    q = rng.standard_normal((B, nq, d)).astype(np.float32)
    kn = rng.standard_normal((B, nkv, d)).astype(np.float32)
    vn = rng.standard_normal((B, nkv, d)).astype(np.float32)
    kc = bits(rng.standard_normal((B, nkv, cap, d)))
    vc = bits(rng.standard_normal((B, nkv, cap, d)))
    lens = np.array([32, 17], np.int32)
    o_gqa = oracle.attention(q, kn, vn, kc, vc, lens)
    rep = lambda a: np.ascontiguousarray(np.repeat(a, G, axis=1))
    o_mha = oracle.attention(q, rep(kn), rep(vn), rep(kc), rep(vc), lens)
    assert np.array_equal(o_gqa, o_mha)


def test_attention_split_and_merge_equals_unsplit(oracle):
    """Attention over key chunks, merged with the (max, sum, weighted output)
    rule, equals attention over the whole range; written with numpy only."""
    rng = np.random.default_rng(9)
    d, cap, t = 8, 41, 40
    q = rng.standard_normal((1, 1, d)).astype(np.float32)
    kn = rng.standard_normal((1, 1, d)).astype(np.float32)
    vn = rng.standard_normal((1, 1, d)).astype(np.float32)
    kc = bits(rng.standard_normal((1, 1, cap, d)))
    vc = bits(rng.standard_normal((1, 1, cap, d)))
    o = oracle.attention(q, kn, vn, kc, vc, np.array([t], np.int32))[0, 0]
    K = np.concatenate([widen(kc[0, 0, :t]), kn[0]]).astype(np.float64)
    V = np.concatenate([widen(vc[0, 0, :t]), vn[0]]).astype(np.float64)
    for bounds in ([0, 41], [0, 7, 41], [0, 16, 32, 40, 41], list(range(0, 42))):
        m_run, l_run, o_run = -np.inf, 0.0, np.zeros(d)
        for lo, hi in zip(bounds[:-1], bounds[1:]):
            s = K[lo:hi] @ q[0, 0].astype(np.float64) / math.sqrt(d)
            m = s.max()
            e = np.exp(s - m)
            l, oc = e.sum(), e @ V[lo:hi]
            m_new = max(m_run, m)
            o_run = o_run * math.exp(m_run - m_new) + oc * math.exp(m - m_new)
            l_run = l_run * math.exp(m_run - m_new) + l * math.exp(m - m_new)
            m_run = m_new
        np.testing.assert_allclose(o, o_run / l_run, rtol=1e-6, atol=1e-6)


def test_attention_matches_torch_sdpa(oracle):
    rng = np.random.default_rng(2)
    B, nq, nkv, d, t = 2, 4, 2, 32, 50
    cap = t + 1
    q = rng.standard_normal((B, nq, d)).astype(np.float32)
    kn = rng.standard_normal((B, nkv, d)).astype(np.float32)
    vn = rng.standard_normal((B, nkv, d)).astype(np.float32)
    kc = bits(rng.standard_normal((B, nkv, cap, d)))
    vc = bits(rng.standard_normal((B, nkv, cap, d)))
    o = oracle.attention(q, kn, vn, kc, vc, np.full(B, t, np.int32))
    Kf, Vf = widen(kc).copy(), widen(vc).copy()
    Kf[:, :, t], Vf[:, :, t] = kn, vn
    G = nq // nkv
    tq = torch.from_numpy(q).double().unsqueeze(2)                       # [B,nq,1,d]
    tk = torch.from_numpy(Kf).double().repeat_interleave(G, dim=1)
    tv = torch.from_numpy(Vf).double().repeat_interleave(G, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).squeeze(2).numpy()
    np.testing.assert_allclose(o, ref, rtol=1e-5, atol=1e-6)


# --------------------------------------------------------------------- window
def test_window_closed_forms(oracle):
    rng = np.random.default_rng(1)
    B, H, eps = 3, 64, 1e-5
    r = rng.standard_normal((B, H)).astype(np.float32)
    ones = bits(np.ones(H))
    zero_part = np.zeros((1, B, H), np.float32)
    h, x = oracle.window(zero_part, r, ones, eps)
    assert np.array_equal(h, r)                       # P = 1, zero partial: h = r
    ms = (r.astype(np.float64) ** 2).mean(1)
    np.testing.assert_allclose((x.astype(np.float64) ** 2).mean(1), ms / (ms + eps), rtol=1e-6)
    # positive rescaling leaves the output unchanged up to the eps term
    _, x4 = oracle.window(zero_part, 4 * r, ones, eps)
    np.testing.assert_allclose(x4, x, rtol=1e-4, atol=1e-6)
    # the sum really is over every partial and the residual
    parts = rng.standard_normal((5, B, H)).astype(np.float32)
    h5, _ = oracle.window(parts, r, ones, eps)
    np.testing.assert_allclose(h5, r.astype(np.float64) + parts.astype(np.float64).sum(0), rtol=1e-6, atol=1e-6)
    # a one-row hand case: h = (3, 4), mean square 12.5, eps 0 -> x = h / sqrt(12.5) * g
    g = bits(np.array([2.0, 0.5]))
    _, xh = oracle.window(np.zeros((1, 1, 2), np.float32), np.array([[3.0, 4.0]], np.float32), g, 0.0)
    np.testing.assert_allclose(xh[0], [3 / math.sqrt(12.5) * 2.0, 4 / math.sqrt(12.5) * 0.5], rtol=1e-6)


def test_window_matches_torch_rms_norm(oracle):
    rng = np.random.default_rng(4)
    B, H, P, eps = 4, 256, 3, 1e-5
    parts = widen(bits(rng.standard_normal((P, B, H))))
    r = widen(bits(rng.standard_normal((B, H))))
    g = bits(1 + 0.1 * rng.standard_normal(H))
    h, x = oracle.window(parts, r, g, eps)
    th = torch.from_numpy(r).double() + torch.from_numpy(parts).double().sum(0)
    ref = torch.nn.functional.rms_norm(th, (H,), torch.from_numpy(widen(g)).double(), eps)
    np.testing.assert_allclose(h, th.numpy(), rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(x, ref.numpy(), rtol=1e-5, atol=1e-6)


# ---------------------------------------------------------------- projections
def test_matmul_special_cases_and_library(oracle):
    rng = np.random.default_rng(6)
    B, K, N = 3, 48, 40
    x = rng.standard_normal((B, K)).astype(np.float32)
    eye = bits(np.eye(K, K))
    assert np.array_equal(oracle.matmul(x, eye), x)
    assert np.all(oracle.matmul(x, bits(np.zeros((K, N)))) == 0)
    # one-hot: output column n picks input k = perm[n]  (catches a transposed operand)
    perm = rng.permutation(K)[:N]
    sel = np.zeros((K, N), np.float32)
    sel[perm, np.arange(N)] = 1
    assert np.array_equal(oracle.matmul(x, bits(sel)), x[:, perm])
    w = bits(0.02 * rng.standard_normal((K, N)))
    ref = torch.from_numpy(x).double() @ torch.from_numpy(widen(w)).double()
    np.testing.assert_allclose(oracle.matmul(x, w), ref.numpy(), rtol=1e-6, atol=1e-7)


def test_swiglu_constants(oracle):
    up = np.ones(5, np.float32)
    z = np.array([0.0, 1.0, 30.0, -30.0, -1.0], np.float32)
    a = oracle.swiglu(z, up)
    assert a[0] == 0.0
    assert abs(a[1] - 0.7310586) < 1e-6            # silu(1) = 1 / (1 + e^-1)
    assert abs(a[2] - 30.0) < 1e-5                 # silu(z) -> z for large z
    assert abs(a[3]) < 1e-10                       # silu(z) -> 0 for very negative z
    assert abs(a[4] + 0.2689414) < 1e-6            # silu(-1) = -1 / (1 + e)
    np.testing.assert_allclose(oracle.swiglu(z, 3 * up), 3 * a, rtol=1e-6)
    ref = torch.nn.functional.silu(torch.from_numpy(z).double()).numpy()
    np.testing.assert_allclose(a, ref, rtol=1e-6, atol=1e-9)


# ----------------------------------------------------------------------- rope
def test_rope_invariants(oracle):
    rng = np.random.default_rng(8)
    n, d, theta = 3, 128, 500000.0
    u = rng.standard_normal((n, d)).astype(np.float32)
    assert np.array_equal(oracle.rope(u, 0, theta), u)              # position 0: identity
    assert np.array_equal(oracle.rope(u, 77, 0.0), u)               # theta <= 0: off
    r = oracle.rope(u, 1234, theta)
    np.testing.assert_allclose(np.linalg.norm(r, axis=1), np.linalg.norm(u, axis=1), rtol=1e-6)
    # relative-position property: <rope(q,m), rope(k,n)> depends only on m - n
    q, k = u[0:1], u[1:2]
    a = float(oracle.rope(q, 100, theta)[0] @ oracle.rope(k, 60, theta)[0])
    b = float(oracle.rope(q, 4100, theta)[0] @ oracle.rope(k, 4060, theta)[0])
    assert abs(a - b) < 2e-3 * max(1.0, abs(a))
    # pair (0, d/2) rotates by exactly t radians (frequency theta^0 = 1); the last
    # pair by t * theta^(-(d-2)/d)
    e = np.zeros((1, d), np.float32)
    e[0, 0] = 1.0
    r = oracle.rope(e, 2, theta)[0]
    assert abs(r[0] - math.cos(2.0)) < 1e-6 and abs(r[d // 2] - math.sin(2.0)) < 1e-6
    e = np.zeros((1, d), np.float32)
    e[0, d // 2 - 1] = 1.0
    ang = 1000 * theta ** (-(d - 2) / d)
    r = oracle.rope(e, 1000, theta)[0]
    assert abs(r[d // 2 - 1] - math.cos(ang)) < 1e-6 and abs(r[d - 1] - math.sin(ang)) < 1e-6


# ---------------------------------------------------------------- whole layer
def torch_quantize_rows(u):
    """Per-vector symmetric int8 with torch ops: fp32 division and round-half-even, as the reading says."""
    u = u.float()
    sc = u.abs().amax(-1, keepdim=True) / 127.0
    codes = torch.where(sc > 0, torch.round(u / sc), torch.zeros_like(u)).clamp(-127, 127)
    return codes.double(), sc.double()


def torch_layer(shape, t, parts=None, resid=None, peers=None, kv8=None):
    """Independent restatement of the layer with torch CPU ops in fp64 (kv8: over that int8 cache)."""
    W = lambda n: torch.from_numpy(widen(t[n])).double()
    P, d, nq, nkv = shape.tp_degree, shape.head_dim, shape.n_q_heads, shape.n_kv_heads
    parts = W("partials_in") if parts is None else torch.from_numpy(parts).double()
    resid = W("residual_in") if resid is None else torch.from_numpy(resid).double()
    peers = W("attn_peer_partials") if peers is None else torch.from_numpy(peers).double()
    h = resid + parts.sum(0)
    norm = lambda v, g: v * torch.rsqrt((v * v).mean(-1, keepdim=True) + shape.rms_eps) * g
    x = norm(h, W("g_attn"))
    B = h.shape[0]
    q = (x @ W("w_q")).view(B, nq, d)
    k = (x @ W("w_k")).view(B, nkv, d)
    v = (x @ W("w_v")).view(B, nkv, d)
    pos = torch.from_numpy(t["ctx_len"].astype(np.int64))

    def rot(u):
        if shape.rope_theta <= 0:
            return u
        i = torch.arange(d // 2, dtype=torch.float64)
        ang = pos.double()[:, None, None] * (shape.rope_theta ** (-2 * i / d))[None, None, :]
        u1, u2 = u[..., : d // 2], u[..., d // 2:]
        return torch.cat([u1 * ang.cos() - u2 * ang.sin(), u2 * ang.cos() + u1 * ang.sin()], -1)

    q, k = rot(q), rot(k)
    if kv8 is None:
        k_st, v_st = k.bfloat16().double(), v.bfloat16().double()     # the new entry as the bf16 cache stores it
        Kc, Vc = W("k_cache").clone(), W("v_cache").clone()
    else:
        kq, ks = torch_quantize_rows(k)                               # the new entry as the int8 cache stores it
        vq, vs = torch_quantize_rows(v)
        k_st, v_st = kq * ks, vq * vs
        deq = lambda c, s_: torch.from_numpy(kv8[c].astype(np.float64)) * torch.from_numpy(
            np.nan_to_num(kv8[s_].astype(np.float64)))[..., None]
        Kc, Vc = deq("k_codes", "k_scales"), deq("v_codes", "v_scales")
    o = torch.zeros(B, nq, d, dtype=torch.float64)
    G = nq // nkv
    for b in range(B):
        n = int(pos[b])
        Kb = torch.cat([Kc[b, :, :n], k_st[b][:, None]], 1).repeat_interleave(G, 0)   # [nq,n+1,d]
        Vb = torch.cat([Vc[b, :, :n], v_st[b][:, None]], 1).repeat_interleave(G, 0)
        p = torch.softmax(torch.einsum("hd,hjd->hj", q[b], Kb) / math.sqrt(d), -1)
        o[b] = torch.einsum("hj,hjd->hd", p, Vb)
    ap = o.reshape(B, nq * d) @ W("w_o")
    h2 = h + ap + (peers.sum(0) if P > 1 else 0)
    x2 = norm(h2, W("g_mlp"))
    a = torch.nn.functional.silu(x2 @ W("w_gate")) * (x2 @ W("w_up"))
    mp = a @ W("w_down")
    return {"h": h, "x": x, "q": q, "k_new": k, "v_new": v, "o": o, "attn_partial": ap,
            "h2": h2, "x2": x2, "a": a, "mlp_partial": mp}


@pytest.mark.parametrize("shape", [
    I.small_shape(),
    I.small_shape(name="mha", n_q_heads=2, n_kv_heads=2, batch=1, tp_degree=1, ctx=37, seed=12),
    I.small_shape(name="ragged", batch=5, ctx=300, ctx_min=10, tp_degree=4, seed=13),
    I.CONFIGS[0],
])
def test_layer_matches_torch_restatement(oracle, shape):
    t = I.make_layers(shape, 1)[0]
    got = oracle.layer_step(shape, t)
    ref = torch_layer(shape, t)
    for name, r in ref.items():
        r = r.numpy()
        np.testing.assert_allclose(got[name].reshape(r.shape), r, rtol=1e-4,
                                   atol=1e-5 * max(1.0, float(np.abs(r).max())), err_msg=name)


def test_layer_config2_matches_torch_restatement(oracle):
    shape = I.CONFIGS[1]
    t = I.make_layers(shape, 1)[0]
    got = oracle.layer_step(shape, t)
    ref = torch_layer(shape, t)
    for name in ("attn_partial", "h2", "mlp_partial", "o"):
        r = ref[name].numpy()
        np.testing.assert_allclose(got[name].reshape(r.shape), r, rtol=1e-4,
                                   atol=1e-5 * max(1.0, float(np.abs(r).max())), err_msg=name)


def test_shard_sum_equals_unsharded_layer(oracle):
    """Column-split QKV/gate/up and row-split O/down over P = 2 (Section 2,
    "Multi-device inference"): the shards' partial sums add up to the block
    outputs of the unsharded layer, given identical window inputs."""
    from dataclasses import replace
    shape = I.CONFIGS[0]
    s0 = I.make_layers(shape, 1, shard=0)[0]
    s1 = I.make_layers(shape, 1, shard=1)[0]
    full_shape = replace(shape, n_q_heads=8, n_kv_heads=8, ffn=2816)
    full = dict(s0)
    full.update({k: v for k, v in s0["full"].items() if k.startswith("w_")})
    B, cap, d = shape.batch, shape.kv_capacity, shape.head_dim
    kc = np.full((B, 8, cap, d), I.BF16_NAN, np.uint16)
    vc = kc.copy()
    kc[:, :, :shape.ctx] = s0["full"]["k"]
    vc[:, :, :shape.ctx] = s0["full"]["v"]
    full["k_cache"], full["v_cache"] = kc, vc
    assert np.array_equal(kc[:, 4:], s1["k_cache"]) and np.array_equal(kc[:, :4], s0["k_cache"])

    a0 = oracle.layer_step(shape, s0)["attn_partial"]
    a1 = oracle.layer_step(shape, s1)["attn_partial"]
    zeros = np.zeros((1, B, shape.hidden), np.float32)
    f = oracle.layer_step(full_shape, full, peer_partials=zeros)
    np.testing.assert_allclose(a0 + a1, f["attn_partial"], rtol=1e-5, atol=1e-6)
    r0 = oracle.layer_step(shape, s0, peer_partials=a1[None])
    r1 = oracle.layer_step(shape, s1, peer_partials=a0[None])
    np.testing.assert_allclose(r0["h2"], f["h2"], rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(r1["h2"], f["h2"], rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(r0["mlp_partial"] + r1["mlp_partial"], f["mlp_partial"], rtol=1e-4, atol=2e-5)


def test_layer_attends_over_the_cache_as_stored(oracle):
    """The new key/value enter attention as the bf16 cache holds them: the layer's o equals
    the attention function applied to q and the nearest-even bf16 roundings of k_new, v_new."""
    shape = I.small_shape(batch=2, ctx=40, seed=22)
    t = I.make_layers(shape, 1)[0]
    r = oracle.layer_step(shape, t)
    kr, vr = widen(bits(r["k_new"])), widen(bits(r["v_new"]))
    o = oracle.attention(r["q"], kr, vr, t["k_cache"], t["v_cache"], t["ctx_len"])
    assert np.array_equal(o, r["o"])
    o_unrounded = oracle.attention(r["q"], r["k_new"], r["v_new"], t["k_cache"], t["v_cache"], t["ctx_len"])
    assert not np.array_equal(o_unrounded, r["o"])


def test_layer_reads_only_live_cache_slots(oracle):
    shape = I.small_shape(batch=2, ctx=64, ctx_min=5, seed=21)
    t = I.make_layers(shape, 1)[0]
    ref = oracle.layer_step(shape, t)
    t2 = dict(t)
    t2["k_cache"] = t["k_cache"].copy()
    t2["v_cache"] = t["v_cache"].copy()
    for b in range(shape.batch):
        n = int(t["ctx_len"][b])
        t2["k_cache"][b, :, n:] = bits(np.full(1, 7.0))
        t2["v_cache"][b, :, n:] = bits(np.full(1, -7.0))
    got = oracle.layer_step(shape, t2)
    for k in ref:
        assert np.array_equal(ref[k], got[k]) and np.isfinite(got[k]).all(), k


def test_chain_feeds_outputs_forward(oracle):
    shape = I.small_shape(layers=3, seed=31)
    layers = I.make_layers(shape)
    outs = oracle.layer_chain(shape, layers)
    parts = widen(layers[1]["partials_in"]).copy()
    parts[0] = outs[0]["mlp_partial"]
    redo = oracle.layer_step(shape, layers[1], partials_in=parts, residual_in=outs[0]["h2"])
    assert np.array_equal(redo["mlp_partial"], outs[1]["mlp_partial"])
    ref = torch_layer(shape, layers[1], parts=parts, resid=outs[0]["h2"])
    np.testing.assert_allclose(outs[1]["mlp_partial"], ref["mlp_partial"].numpy(), rtol=1e-4, atol=1e-5)


# ---------------------------------------------------------------- int8 weights (per output channel)
def test_int8_quantiser_closed_forms(oracle):
    """Pins of oracle_quantize_weights that do not retype its loop: the column maximum maps to +-127
    and the scale is max / 127; a column that is an exact multiple pattern of its scale is
    reproduced exactly; codes stay within [-127, 127]; the dequantised weight is within half a step;
    a zero column gives scale 0 and codes 0; a hand-worked 3 x 2 case."""
    rng = np.random.default_rng(3)
    K, N = 64, 9
    w = rng.standard_normal((K, N)).astype(np.float32) * 0.02
    w[:, 3] = 0.0
    # column 4: multiples of 2^-10 from -127 to 127 -> scale 2^-10 exactly, codes = the multiples
    mult = rng.integers(-127, 128, size=K)
    mult[0], mult[1] = 127, -127
    w[:, 4] = mult * 2.0 ** -10
    bits = I.f32_to_bf16_bits(w)
    wf = I.bf16_bits_to_f32(bits)
    q, sc = oracle.quantize_weights(bits)
    assert q.dtype == np.int8 and q.min() >= -127 and q.max() <= 127
    mx = np.abs(wf).max(axis=0)
    assert np.allclose(sc, mx / 127.0, rtol=1e-6)
    for n in range(N):
        if n == 3:
            assert sc[n] == 0 and not q[:, n].any()
            continue
        assert np.abs(q[np.abs(wf[:, n]).argmax(), n]) == 127
        assert np.abs(q[:, n].astype(np.float64) * sc[n] - wf[:, n]).max() <= 0.5000001 * sc[n]
    assert sc[4] == 2.0 ** -10 and np.array_equal(q[:, 4], mult)
    # hand-worked: column (0.5, -0.25, 0.125): scale 0.5/127; codes 127, -63.5 -> -64 (ties to even), 31.75 -> 32
    hand = I.f32_to_bf16_bits(np.array([[0.5, 1.0], [-0.25, -1.0], [0.125, 0.5]], np.float32))
    qh, sh = oracle.quantize_weights(hand)
    assert qh[:, 0].tolist() == [127, -64, 32] and qh[:, 1].tolist() == [127, -127, 64]
    assert abs(sh[0] - 0.5 / 127) < 1e-9 and abs(sh[1] - 1.0 / 127) < 1e-9


def test_int8_matmul_and_layer_against_independent_restatements(oracle):
    """oracle_matmul_q8 against numpy on the dequantised matrix; the int8 layer step against the
    bf16 layer step run on weights that are already exactly representable in int8 (then both
    definitions must agree), and against a torch restatement of one projection."""
    rng = np.random.default_rng(4)
    x = rng.standard_normal((3, 40)).astype(np.float32)
    w = I.f32_to_bf16_bits(rng.standard_normal((40, 7)).astype(np.float32) * 0.05)
    q, sc = oracle.quantize_weights(w)
    want = x.astype(np.float64) @ (q.astype(np.float64) * sc.astype(np.float64))
    assert np.allclose(oracle.matmul_q8(x, q, sc), want, rtol=1e-6, atol=1e-7)
    # weights = small integers times a power of two per column: int8 quantisation is lossless on them,
    # so the quantised layer equals the plain layer
    shape = I.small_shape(name="w8_lossless", batch=2, hidden=256, ffn=128, ctx=9, seed=90)
    t = I.make_layers(shape, 1)[0]
    for name in ("w_q", "w_k", "w_v", "w_o", "w_gate", "w_up", "w_down"):
        K, N = t[name].shape
        codes = rng.integers(-127, 128, size=(K, N))
        codes[0, :] = 127                                     # every column reaches the extreme code
        t[name] = I.f32_to_bf16_bits((codes * 2.0 ** -12).astype(np.float32))
    plain = oracle.layer_step(shape, t)
    quant = oracle.layer_step(shape, t, int8_weights=True)
    for k in ("q", "o", "attn_partial", "a", "mlp_partial", "h2"):
        assert np.allclose(plain[k], quant[k], rtol=2e-6, atol=1e-6), k
    # generic weights: the quantised layer differs from the plain one, by about the quantisation noise
    t2 = I.make_layers(shape, 1)[0]
    p2, q2 = oracle.layer_step(shape, t2), oracle.layer_step(shape, t2, int8_weights=True)
    rel = np.abs(p2["mlp_partial"] - q2["mlp_partial"]).max() / np.abs(p2["mlp_partial"]).max()
    assert 1e-5 < rel < 5e-2
    # one projection restated with torch: q = x W_q with dequantised weights
    xq = torch.from_numpy(q2["x"].astype(np.float64))
    qq, ss = oracle.quantize_weights(t2["w_q"])
    wq = torch.from_numpy(qq.astype(np.float64) * ss.astype(np.float64))
    if shape.rope_theta <= 0:
        assert np.allclose((xq @ wq).numpy().reshape(q2["q"].shape), q2["q"], rtol=1e-5, atol=1e-6)
    v_ref = (torch.from_numpy(q2["x"].astype(np.float64)) @ torch.from_numpy(
        oracle.quantize_weights(t2["w_v"])[0].astype(np.float64) * oracle.quantize_weights(t2["w_v"])[1].astype(np.float64)))
    assert np.allclose(v_ref.numpy().reshape(q2["v_new"].shape), q2["v_new"], rtol=1e-5, atol=1e-6)


# ---------------------------------------------------------------- int8 KV-cache (one scale per cached vector)
def test_int8_row_quantiser_closed_forms(oracle):
    """Pins of oracle_quantize_rows that do not retype its loop: hand-worked vectors (ties go to the even
    code), the zero vector, the extreme code at the largest entry, the half-step error bound, odd
    symmetry, and exact covariance with a power-of-two factor."""
    hand = np.array([[127.0, -63.5, 0.0, 1.0], [0.5, 0.25, -0.5, 0.125], [0.0, 0.0, 0.0, 0.0]], np.float32)
    q, sc = oracle.quantize_rows(hand)
    assert q[0].tolist() == [127, -64, 0, 1] and sc[0] == 1.0
    assert q[1].tolist() == [127, 64, -127, 32] and abs(sc[1] - 0.5 / 127) < 1e-9
    assert not q[2].any() and sc[2] == 0.0
    rng = np.random.default_rng(8)
    u = (rng.standard_normal((50, 128)) * rng.uniform(0.01, 30.0, (50, 1))).astype(np.float32)
    q, sc = oracle.quantize_rows(u)
    assert q.dtype == np.int8 and q.min() >= -127 and q.max() <= 127
    assert np.allclose(sc, np.abs(u).max(-1) / 127.0, rtol=1e-6)
    assert (np.abs(q[np.arange(50), np.abs(u).argmax(-1)]) == 127).all()
    assert (np.abs(q.astype(np.float64) * sc[:, None] - u) <= 0.5000001 * sc[:, None]).all()
    qn, scn = oracle.quantize_rows(-u)
    assert np.array_equal(qn, -q) and np.array_equal(scn, sc)
    q8, sc8 = oracle.quantize_rows(u * np.float32(2.0 ** -7))
    assert np.array_equal(q8, q) and np.array_equal(sc8, sc * np.float32(2.0 ** -7))
    # shape handling: leading axes are independent vectors
    q3, sc3 = oracle.quantize_rows(u.reshape(5, 10, 128))
    assert np.array_equal(q3.reshape(50, 128), q) and np.array_equal(sc3.reshape(50), sc)


def test_int8_attention_against_brute_force_and_the_bf16_routine(oracle):
    """oracle_attention_kv8 against the brute-force softmax on the dequantised arrays, and against
    the (separately pinned) bf16 attention on a cache whose entries code * 2^-5 are exact in bf16."""
    rng = np.random.default_rng(9)
    B, nq, nkv, d, cap = 2, 4, 2, 8, 11
    lens = np.array([4, 10], np.int32)
    q = rng.standard_normal((B, nq, d)).astype(np.float32)
    codes = lambda *s: rng.integers(-127, 128, size=s).astype(np.int8)
    kc, vc = codes(B, nkv, cap, d), codes(B, nkv, cap, d)
    ks = rng.uniform(0.005, 0.02, (B, nkv, cap)).astype(np.float32)
    vs = rng.uniform(0.005, 0.02, (B, nkv, cap)).astype(np.float32)
    kqn, vqn = codes(B, nkv, d), codes(B, nkv, d)
    ksn = rng.uniform(0.005, 0.02, (B, nkv)).astype(np.float32)
    vsn = rng.uniform(0.005, 0.02, (B, nkv)).astype(np.float32)
    for b in range(B):                      # dead slots must not be read
        kc[b, :, lens[b]:], vc[b, :, lens[b]:] = -128, -128
        ks[b, :, lens[b]:], vs[b, :, lens[b]:] = np.nan, np.nan
    o, probs = oracle.attention_kv8(q, kqn, ksn, vqn, vsn, kc, ks, vc, vs, lens, want_probs=True)
    G = nq // nkv
    for b in range(B):
        n = int(lens[b])
        for h in range(nq):
            g = h // G
            keys = np.concatenate([kc[b, g, :n].astype(np.float64) * ks[b, g, :n, None].astype(np.float64),
                                   (kqn[b, g].astype(np.float64) * float(ksn[b, g]))[None]])
            vals = np.concatenate([vc[b, g, :n].astype(np.float64) * vs[b, g, :n, None].astype(np.float64),
                                   (vqn[b, g].astype(np.float64) * float(vsn[b, g]))[None]])
            want, p = brute_attention(q[b, h].astype(np.float64), keys, vals)
            assert np.allclose(o[b, h], want, rtol=1e-6, atol=1e-7)
            assert np.allclose(probs[b, h, :n + 1], p, rtol=1e-6, atol=1e-8) and abs(probs[b, h, :n + 1].sum() - 1) < 1e-6
    # power-of-two scales: every code * scale is a bf16 number, so the bf16 routine sees the same cache
    ks2 = np.full_like(ks, 2.0 ** -5)
    vs2 = np.full_like(vs, 2.0 ** -6)
    kb = I.f32_to_bf16_bits(kc.astype(np.float32) * ks2[..., None])
    vb = I.f32_to_bf16_bits(vc.astype(np.float32) * vs2[..., None])
    assert np.array_equal(I.bf16_bits_to_f32(kb), kc.astype(np.float32) * ks2[..., None])
    ksn2, vsn2 = np.full_like(ksn, 2.0 ** -5), np.full_like(vsn, 2.0 ** -6)
    o8 = oracle.attention_kv8(q, kqn, ksn2, vqn, vsn2, kc, ks2, vc, vs2, lens)
    o16 = oracle.attention(q, kqn.astype(np.float32) * ksn2[..., None], vqn.astype(np.float32) * vsn2[..., None], kb, vb, lens)
    assert np.allclose(o8, o16, rtol=1e-6, atol=1e-7)


def test_int8_kv_layer_against_torch_restatement(oracle):
    """The layer step over an int8 cache against the torch restatement (its own quantiser, its own
    dequantisation), with bf16 and with int8 weights; the stored new entry is the quantised k_new, v_new."""
    for shape in (I.small_shape(name="kv8", batch=3, ctx=90, ctx_min=4, seed=95),
                  I.small_shape(name="kv8_mha", n_q_heads=2, n_kv_heads=2, batch=1, tp_degree=1, ctx=37, seed=96)):
        t = I.make_layers(shape, 1)[0]
        kv = I.make_int8_cache(shape, t["ctx_len"])
        got = oracle.layer_step(shape, t, kv8=kv)
        ref = torch_layer(shape, t, kv8=kv)
        for name, r in ref.items():
            r = r.numpy()
            np.testing.assert_allclose(got[name].reshape(r.shape), r, rtol=1e-4,
                                       atol=1e-5 * max(1.0, float(np.abs(r).max())), err_msg=name)
        kq, ks = torch_quantize_rows(torch.from_numpy(got["k_new"]))
        vq, vs = torch_quantize_rows(torch.from_numpy(got["v_new"]))
        assert np.array_equal(got["k_codes_new"], kq.numpy().astype(np.int8))
        assert np.array_equal(got["v_codes_new"], vq.numpy().astype(np.int8))
        assert np.allclose(got["k_scale_new"], ks.numpy()[..., 0], rtol=1e-7) and np.allclose(got["v_scale_new"], vs.numpy()[..., 0], rtol=1e-7)
        # the int8 cache changes the result (it is not the bf16 path in disguise) and composes with int8 weights
        plain = oracle.layer_step(shape, t)
        assert not np.allclose(plain["o"], got["o"], rtol=1e-3, atol=1e-4)
        both = oracle.layer_step(shape, t, kv8=kv, int8_weights=True)
        w8 = oracle.layer_step(shape, t, int8_weights=True)
        assert np.array_equal(both["x"], w8["x"]) and np.array_equal(both["q"], w8["q"])
        o_again = oracle.attention_kv8(both["q"], both["k_codes_new"], both["k_scale_new"], both["v_codes_new"],
                                       both["v_scale_new"], kv["k_codes"], kv["k_scales"], kv["v_codes"], kv["v_scales"],
                                       t["ctx_len"])
        assert np.array_equal(o_again, both["o"])
