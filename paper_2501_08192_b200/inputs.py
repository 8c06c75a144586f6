"""Seeded synthetic inputs for one tensor-parallel shard's decode step.

This module holds data generation only: shapes, a seeded draw order and the
fp32 -> bf16 rounding of the drawn values.  It contains none of the layer's
arithmetic, so both the CPU oracle's tests and the CUDA path may use it.

Workloads follow the five benchmark configurations (Llama-3-shaped decoder
layers under tensor parallelism; the paper's own runs use static synthetic
batches of equal length, Section 4 "Experimental setup").  Values:
weights ~ N(0, 0.02^2), RMSNorm gains 1 + N(0, 0.1^2), partial-sum buffers,
residual and cached K/V ~ N(0, 1), each drawn in fp32 and rounded once to bf16
(round to nearest even).  All tensors are returned as numpy uint16 arrays that
hold bf16 bit patterns.

Draw order per layer instance (never reorder; stored expectations depend on
it): g_attn, g_mlp, w_q, w_k, w_v, w_o, w_gate, w_up, w_down, residual_in,
partials_in[0..P-1], attn_peer_partials[0..P-2], K, V, ctx_len (ragged only).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

BF16_NAN = np.uint16(0x7FC0)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (nearest even) and return the 16-bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        out[nan] = BF16_NAN
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class ShardShape:
    """Per-shard sizes of one decoder layer's decode step."""

    name: str
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    tp_degree: int          # P: partial-sum buffers reduced in each window
    batch: int
    ctx: int                # cached tokens per sequence (max, if ragged)
    ctx_min: Optional[int] = None   # ragged: ctx_len ~ U{ctx_min..ctx}
    layers: int = 1
    seed: int = 0
    # when set, tensors are drawn at this unsharded size and shard `shard` is
    # sliced from them (heads and FFN columns are split evenly over P)
    draw_unsharded: bool = False
    rms_eps: float = 1e-5
    rope_theta: float = 500000.0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def kv_capacity(self) -> int:
        return self.ctx + 1

    def weight_bytes(self) -> int:
        H, d = self.hidden, self.head_dim
        qkv = H * (self.n_q_heads + 2 * self.n_kv_heads) * d
        o = self.n_q_heads * d * H
        gu = H * 2 * self.ffn
        dn = self.ffn * H
        return 2 * (qkv + o + gu + dn)


# The five benchmark configurations (index 0..4 = configs 1..5).
CONFIGS: Tuple[ShardShape, ...] = (
    ShardShape("tiny_tp2", 1024, 4, 4, 128, 1408, 2, 1, 512, seed=0, draw_unsharded=True),
    ShardShape("llama3_8b_tp8", 4096, 4, 1, 128, 1792, 8, 8, 4096, seed=1),
    ShardShape("llama3_70b_tp8_chain4", 8192, 8, 1, 128, 3584, 8, 16, 8192, layers=4, seed=2),
    ShardShape("llama3_70b_tp4_ragged", 8192, 16, 2, 128, 7168, 4, 64, 4096, ctx_min=512, seed=3),
    ShardShape("llama3_8b_tp8_long", 4096, 4, 1, 128, 1792, 8, 32, 32768, seed=4),
)


def _normal_bf16(rng: np.random.Generator, shape, std: float = 1.0, mean: float = 0.0,
                 chunk: int = 1 << 24) -> np.ndarray:
    """Draw N(mean, std^2) in fp32, chunked along the flat index, round to bf16."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        v = rng.standard_normal(e - s, dtype=np.float32)
        if std != 1.0:
            v *= np.float32(std)
        if mean != 0.0:
            v += np.float32(mean)
        out[s:e] = f32_to_bf16_bits(v)
    return out.reshape(shape)


def make_layer(shape: ShardShape, rng: np.random.Generator, shard: int = 0,
               nan_fill_tail: bool = True) -> Dict[str, np.ndarray]:
    """Draw one layer instance's tensors in the documented order.

    Returns bf16 bit patterns (uint16) except ctx_len (int32).  Weights are
    [in, out] row-major.  k_cache / v_cache are [batch, n_kv, ctx+1, head_dim];
    slots at and beyond ctx_len[b] hold a NaN pattern when nan_fill_tail is
    set, so that a read past the length or a missing append shows up.
    """
    P = shape.tp_degree
    H, d, B = shape.hidden, shape.head_dim, shape.batch
    mul = P if shape.draw_unsharded else 1
    nq, nkv, F = shape.n_q_heads * mul, shape.n_kv_heads * mul, shape.ffn * mul

    t: Dict[str, np.ndarray] = {}
    t["g_attn"] = _normal_bf16(rng, (H,), 0.1, 1.0)
    t["g_mlp"] = _normal_bf16(rng, (H,), 0.1, 1.0)
    t["w_q"] = _normal_bf16(rng, (H, nq * d), 0.02)
    t["w_k"] = _normal_bf16(rng, (H, nkv * d), 0.02)
    t["w_v"] = _normal_bf16(rng, (H, nkv * d), 0.02)
    t["w_o"] = _normal_bf16(rng, (nq * d, H), 0.02)
    t["w_gate"] = _normal_bf16(rng, (H, F), 0.02)
    t["w_up"] = _normal_bf16(rng, (H, F), 0.02)
    t["w_down"] = _normal_bf16(rng, (F, H), 0.02)
    t["residual_in"] = _normal_bf16(rng, (B, H))
    t["partials_in"] = np.stack([_normal_bf16(rng, (B, H)) for _ in range(P)])
    t["attn_peer_partials"] = (np.stack([_normal_bf16(rng, (B, H)) for _ in range(P - 1)])
                               if P > 1 else np.zeros((0, B, H), np.uint16))
    k = _normal_bf16(rng, (B, nkv, shape.ctx, d))
    v = _normal_bf16(rng, (B, nkv, shape.ctx, d))
    if shape.ctx_min is not None:
        ctx_len = rng.integers(shape.ctx_min, shape.ctx + 1, size=B).astype(np.int32)
    else:
        ctx_len = np.full(B, shape.ctx, dtype=np.int32)
    t["ctx_len"] = ctx_len

    if shape.draw_unsharded:
        s = shard
        nq_s, nkv_s, F_s = shape.n_q_heads, shape.n_kv_heads, shape.ffn
        t["full"] = {k_: t[k_] for k_ in ("w_q", "w_k", "w_v", "w_o", "w_gate", "w_up", "w_down")}
        t["full"]["k"] = k
        t["full"]["v"] = v
        t["w_q"] = np.ascontiguousarray(t["w_q"][:, s * nq_s * d:(s + 1) * nq_s * d])
        t["w_k"] = np.ascontiguousarray(t["w_k"][:, s * nkv_s * d:(s + 1) * nkv_s * d])
        t["w_v"] = np.ascontiguousarray(t["w_v"][:, s * nkv_s * d:(s + 1) * nkv_s * d])
        t["w_o"] = np.ascontiguousarray(t["w_o"][s * nq_s * d:(s + 1) * nq_s * d, :])
        t["w_gate"] = np.ascontiguousarray(t["w_gate"][:, s * F_s:(s + 1) * F_s])
        t["w_up"] = np.ascontiguousarray(t["w_up"][:, s * F_s:(s + 1) * F_s])
        t["w_down"] = np.ascontiguousarray(t["w_down"][s * F_s:(s + 1) * F_s, :])
        k = np.ascontiguousarray(k[:, s * nkv_s:(s + 1) * nkv_s])
        v = np.ascontiguousarray(v[:, s * nkv_s:(s + 1) * nkv_s])

    cap = shape.kv_capacity
    fill = BF16_NAN if nan_fill_tail else np.uint16(0)
    kc = np.full((B, shape.n_kv_heads, cap, d), fill, dtype=np.uint16)
    vc = np.full((B, shape.n_kv_heads, cap, d), fill, dtype=np.uint16)
    for b in range(B):
        n = int(ctx_len[b])
        kc[b, :, :n] = k[b, :, :n]
        vc[b, :, :n] = v[b, :, :n]
    t["k_cache"] = kc
    t["v_cache"] = vc
    return t


def make_int8_cache(shape: ShardShape, ctx_len: np.ndarray, seed: int = 0) -> Dict[str, np.ndarray]:
    """A seeded int8 KV-cache for `shape`: codes int8 [batch, n_kv, ctx+1, head_dim] and one fp32
    scale per cached vector [batch, n_kv, ctx+1], for keys and for values.  Codes are N(0, 42^2)
    rounded and clipped to [-127, 127]; scales are 0.02 + 0.01 |N(0, 1)|, so the cached values
    (code * scale) have about unit variance like the bf16 cache.  Slots at and beyond ctx_len[b]
    hold code -128 and a NaN scale, so that a read past the length or a missing append shows up.
    Draw order: K codes, K scales, V codes, V scales."""
    rng = np.random.Generator(np.random.PCG64([shape.seed, 0x6b76, seed]))
    B, nkv, cap, d = shape.batch, shape.n_kv_heads, shape.kv_capacity, shape.head_dim
    out: Dict[str, np.ndarray] = {}
    for name in ("k", "v"):
        codes = np.empty((B, nkv, cap, d), np.int8)
        for b in range(B):                                     # per sequence: bounded temporary
            v = rng.standard_normal((nkv, cap, d), dtype=np.float32) * np.float32(42.0)
            codes[b] = np.clip(np.rint(v), -127, 127).astype(np.int8)
        scales = (np.float32(0.02) + np.float32(0.01) * np.abs(rng.standard_normal((B, nkv, cap), dtype=np.float32))
                  ).astype(np.float32)
        for b in range(B):
            n = int(ctx_len[b])
            codes[b, :, n:] = -128
            scales[b, :, n:] = np.nan
        out[name + "_codes"] = codes
        out[name + "_scales"] = scales
    return out


def make_layers(shape: ShardShape, n_instances: Optional[int] = None, shard: int = 0,
                nan_fill_tail: bool = True) -> List[Dict[str, np.ndarray]]:
    """All layer instances of a configuration from one PCG64 stream seeded by shape.seed."""
    rng = np.random.Generator(np.random.PCG64(shape.seed))
    n = shape.layers if n_instances is None else n_instances
    return [make_layer(shape, rng, shard=shard, nan_fill_tail=nan_fill_tail) for _ in range(n)]


def small_shape(name: str = "small", **kw) -> ShardShape:
    """A shape the oracle finishes in well under a second; override any field."""
    base = ShardShape(name, 512, 4, 2, 128, 384, 2, 3, 200, seed=11)
    return replace(base, **kw)
