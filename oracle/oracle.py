"""Python face of the CPU oracle.  TEST INFRASTRUCTURE ONLY.

Loads the plain-C layer oracle (preserve_oracle.c, compiled with gcc) through
ctypes and holds the prefetch-insertion oracle, a direct restatement of
Algorithm 1 ("Prefetch Operator Insertion") over an explicit graph.

Nothing here may be imported by the product package; only the tests, the smoke
check and the benchmark's CPU-baseline leg use it.  It shares no code with the
CUDA path.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from collections import deque
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "preserve_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over the outermost loops only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("ffn", C.c_int32), ("tp_degree", C.c_int32),
                ("batch", C.c_int32), ("kv_capacity", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float)]


_OUT_NAMES = ("h", "x", "q", "k_new", "v_new", "o", "attn_partial", "h2", "x2", "a", "mlp_partial")


class _Out(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _OUT_NAMES]


_KV8_NAMES = ("k_codes", "v_codes", "k_scales", "v_scales", "k_codes_new", "v_codes_new", "k_scale_new", "v_scale_new")


class _Kv8(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _KV8_NAMES]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_num_threads.restype = C.c_int
        _lib.oracle_layer_step.restype = C.c_int
        _lib.oracle_layer_step_w8.restype = C.c_int
        _lib.oracle_layer_step_kv8.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def window(parts, r, g_bits, eps: float):
    """h = r + sum_p parts[p]; x = RMSNorm(h; g).  parts [n,B,H] f32, r [B,H] f32, g bf16 bits [H]."""
    parts, r, g_bits = _f32(parts), _f32(r), _u16(g_bits)
    n, B, H = parts.shape
    h = np.empty((B, H), np.float32)
    x = np.empty((B, H), np.float32)
    lib().oracle_window(C.c_int(B), C.c_int(H), C.c_int(n), _p(parts), _p(r), _p(g_bits),
                        C.c_float(eps), _p(h), _p(x))
    return h, x


def matmul(x, w_bits):
    """x [B,K] f32 times W [K,N] (bf16 bits, row-major) -> [B,N] f32."""
    x, w_bits = _f32(x), _u16(w_bits)
    B, K = x.shape
    K2, N = w_bits.shape
    assert K == K2
    y = np.empty((B, N), np.float32)
    lib().oracle_matmul(C.c_int(B), C.c_int(K), C.c_int(N), _p(x), _p(w_bits), _p(y))
    return y


def rope(u, t: int, theta: float):
    """Rotary embedding of u [n_heads, d] at position t; returns a new array."""
    u = _f32(u).copy()
    n, d = u.shape
    lib().oracle_rope(C.c_int(n), C.c_int(d), C.c_int(int(t)), C.c_float(theta), _p(u))
    return u


def attention(q, k_new, v_new, k_cache_bits, v_cache_bits, ctx_len, want_probs: bool = False):
    """Decode attention; q [B,nq,d], k_new/v_new [B,nkv,d] f32, caches bf16 bits [B,nkv,cap,d]."""
    q, k_new, v_new = _f32(q), _f32(k_new), _f32(v_new)
    kc, vc = _u16(k_cache_bits), _u16(v_cache_bits)
    ctx_len = np.ascontiguousarray(ctx_len, dtype=np.int32)
    B, nq, d = q.shape
    _, nkv, cap, _ = kc.shape
    o = np.empty((B, nq, d), np.float32)
    probs = np.zeros((B, nq, cap), np.float32) if want_probs else None
    lib().oracle_attention(C.c_int(B), C.c_int(nq), C.c_int(nkv), C.c_int(d), C.c_int(cap),
                           _p(ctx_len), _p(q), _p(k_new), _p(v_new), _p(kc), _p(vc), _p(o),
                           _p(probs) if want_probs else C.c_void_p(0))
    return (o, probs) if want_probs else o


def swiglu(gate, up):
    gate, up = _f32(gate), _f32(up)
    a = np.empty_like(gate)
    lib().oracle_swiglu(C.c_size_t(gate.size), _p(gate), _p(up), _p(a))
    return a


def quantize_weights(w_bits):
    """Per-output-channel symmetric int8 quantisation of W [K,N] (bf16 bits): (codes int8 [K,N], scale f32 [N])."""
    w_bits = _u16(w_bits)
    K, N = w_bits.shape
    q = np.empty((K, N), np.int8)
    sc = np.empty(N, np.float32)
    lib().oracle_quantize_weights(C.c_int(K), C.c_int(N), _p(w_bits), _p(q), _p(sc))
    return q, sc


def matmul_q8(x, q, scale):
    """x [B,K] f32 times int8 codes q [K,N] with per-column scale [N] -> [B,N] f32."""
    x = _f32(x)
    q = np.ascontiguousarray(q, np.int8)
    scale = _f32(scale)
    B, K = x.shape
    N = q.shape[1]
    y = np.empty((B, N), np.float32)
    lib().oracle_matmul_q8(C.c_int(B), C.c_int(K), C.c_int(N), _p(x), _p(q), _p(scale), _p(y))
    return y


def quantize_rows(u):
    """Symmetric int8 quantisation with one scale per vector (last axis): (codes int8, scale f32)."""
    u = _f32(u)
    d = u.shape[-1]
    q = np.empty(u.shape, np.int8)
    sc = np.empty(u.shape[:-1], np.float32)
    lib().oracle_quantize_rows(C.c_size_t(u.size // d), C.c_int(d), _p(u), _p(q), _p(sc))
    return q, sc


def _i8(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.int8, a.dtype
    return a


def attention_kv8(q, kq_new, ks_new, vq_new, vs_new, k_codes, k_scales, v_codes, v_scales, ctx_len,
                  want_probs: bool = False):
    """Decode attention over an int8 cache: codes int8 [B,nkv,cap,d], scales f32 [B,nkv,cap]; the new
    entry as codes [B,nkv,d] and scales [B,nkv]."""
    q = _f32(q)
    kq_new, vq_new, k_codes, v_codes = _i8(kq_new), _i8(vq_new), _i8(k_codes), _i8(v_codes)
    ks_new, vs_new, k_scales, v_scales = _f32(ks_new), _f32(vs_new), _f32(k_scales), _f32(v_scales)
    ctx_len = np.ascontiguousarray(ctx_len, dtype=np.int32)
    B, nq, d = q.shape
    _, nkv, cap, _ = k_codes.shape
    assert k_scales.shape == (B, nkv, cap) and v_scales.shape == (B, nkv, cap)
    o = np.empty((B, nq, d), np.float32)
    probs = np.zeros((B, nq, cap), np.float32) if want_probs else None
    lib().oracle_attention_kv8(C.c_int(B), C.c_int(nq), C.c_int(nkv), C.c_int(d), C.c_int(cap), _p(ctx_len),
                               _p(q), _p(kq_new), _p(ks_new), _p(vq_new), _p(vs_new), _p(k_codes), _p(k_scales),
                               _p(v_codes), _p(v_scales), _p(o), _p(probs) if want_probs else C.c_void_p(0))
    return (o, probs) if want_probs else o


def layer_step(shape, t: Dict[str, np.ndarray], partials_in=None, residual_in=None,
               peer_partials=None, int8_weights: bool = False, kv8: Optional[Dict[str, np.ndarray]] = None
               ) -> Dict[str, np.ndarray]:
    """One decode step of one shard's layer.

    kv8 = {"k_codes", "k_scales", "v_codes", "v_scales"} runs the step over that int8 KV-cache
    instead of t's bf16 cache; the result then also holds the appended entry as stored
    ("k_codes_new" int8 [B,nkv,d], "k_scale_new" f32 [B,nkv], and the same for v).

    `shape` needs hidden, n_q_heads, n_kv_heads, head_dim, ffn, tp_degree,
    rms_eps, rope_theta.  `t` holds the bf16-bit tensors of inputs.make_layer.
    partials_in / residual_in / peer_partials override t's entries with fp32
    arrays (a chain passes the previous layer's unrounded outputs).
    """
    def widen(b):
        return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)

    P = shape.tp_degree
    if kv8 is None:
        kc, vc = _u16(t["k_cache"]), _u16(t["v_cache"])
        B, nkv, cap, d = kc.shape
    else:
        B, nkv, cap, d = kv8["k_codes"].shape
    H = shape.hidden
    parts = _f32(widen(t["partials_in"]) if partials_in is None else partials_in).reshape(P, B, H)
    resid = _f32(widen(t["residual_in"]) if residual_in is None else residual_in).reshape(B, H)
    peers = _f32(widen(t["attn_peer_partials"]) if peer_partials is None else peer_partials)
    peers = np.ascontiguousarray(peers.reshape(max(P - 1, 0), B, H))
    if peers.size == 0:
        peers = np.zeros((1,), np.float32)
    ctx_len = np.ascontiguousarray(t["ctx_len"], dtype=np.int32)
    cfg = _Cfg(H, shape.n_q_heads, shape.n_kv_heads, d, shape.ffn, P, B, cap,
               shape.rms_eps, shape.rope_theta)
    nq, F = shape.n_q_heads, shape.ffn
    sizes = {"h": (B, H), "x": (B, H), "q": (B, nq, d), "k_new": (B, nkv, d), "v_new": (B, nkv, d),
             "o": (B, nq, d), "attn_partial": (B, H), "h2": (B, H), "x2": (B, H), "a": (B, F),
             "mlp_partial": (B, H)}
    res = {n: np.empty(s, np.float32) for n, s in sizes.items()}
    out = _Out(*[res[n].ctypes.data for n in _OUT_NAMES])
    w = [_u16(t[n]) for n in ("w_q", "w_k", "w_v", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")]
    if kv8 is not None:
        keep = [_i8(kv8["k_codes"]), _i8(kv8["v_codes"]), _f32(kv8["k_scales"]), _f32(kv8["v_scales"])]
        assert keep[2].shape == (B, nkv, cap) and keep[3].shape == (B, nkv, cap)
        res["k_codes_new"] = np.empty((B, nkv, d), np.int8)
        res["v_codes_new"] = np.empty((B, nkv, d), np.int8)
        res["k_scale_new"] = np.empty((B, nkv), np.float32)
        res["v_scale_new"] = np.empty((B, nkv), np.float32)
        kv = _Kv8(*[a.ctypes.data for a in keep],
                  *[res[n].ctypes.data for n in ("k_codes_new", "v_codes_new", "k_scale_new", "v_scale_new")])
        rc = lib().oracle_layer_step_kv8(C.byref(cfg), *[_p(a) for a in w], _p(ctx_len), _p(parts), _p(peers),
                                         _p(resid), C.byref(kv), C.c_int(1 if int8_weights else 0), C.byref(out))
        if rc != 0:
            raise ValueError("oracle_layer_step_kv8 rejected the configuration")
        return res
    fn = lib().oracle_layer_step_w8 if int8_weights else lib().oracle_layer_step
    rc = fn(C.byref(cfg), *[_p(a) for a in w], _p(ctx_len), _p(parts), _p(peers),
            _p(resid), _p(kc), _p(vc), C.byref(out))
    if rc != 0:
        raise ValueError("oracle_layer_step rejected the configuration")
    return res


def layer_chain(shape, layers: Sequence[Dict[str, np.ndarray]], int8_weights: bool = False,
                kv8: Optional[Sequence[Dict[str, np.ndarray]]] = None) -> List[Dict[str, np.ndarray]]:
    """A chain of layers: layer l+1 takes partials_in[0] = mlp_partial_l and residual_in = h2_l.
    kv8: one int8 cache per layer (see layer_step)."""
    outs: List[Dict[str, np.ndarray]] = []
    for i, t in enumerate(layers):
        kv = None if kv8 is None else kv8[i]
        if i == 0:
            outs.append(layer_step(shape, t, int8_weights=int8_weights, kv8=kv))
            continue
        prev = outs[-1]
        parts = (np.ascontiguousarray(t["partials_in"], np.uint16).astype(np.uint32)
                 << np.uint32(16)).view(np.float32).copy()
        parts[0] = prev["mlp_partial"]
        outs.append(layer_step(shape, t, partials_in=parts, residual_in=prev["h2"], int8_weights=int8_weights, kv8=kv))
    return outs


# --------------------------------------------------------------------------
# Prefetch operator insertion (Algorithm 1), over an explicit graph.
#
# A graph is a list of nodes; node i is a dict with
#   "kind": "comm" | "matmul" | "attention" | "other"
#   "mem":  bytes a prefetch of this node would bring in (weights, or K+V)
#   "children": list of successor node indices
# Readings where the listing and the prose leave a choice:
#   - the comparison is strict (cacheSum < C), as printed in the listing;
#   - a node that does not fit is skipped AND ends the walk for this
#     communication op (the listing sets the end flag); nothing after it is
#     considered and no tensor is prefetched in part;
#   - the walk also ends when no successors remain (the prose's "end of graph";
#     the listing omits this exit);
#   - nodes that are neither MatMul nor SelfAttention add nothing.
# --------------------------------------------------------------------------

def insert_prefetch_ops(graph: Sequence[dict], cache_size: int) -> Dict[int, List[int]]:
    """For every communication op, the nodes whose data is prefetched beside it."""
    plan: Dict[int, List[int]] = {}
    for op, node in enumerate(graph):
        if node["kind"] != "comm":
            continue
        plan[op] = []
        cache_sum = 0
        reached_end = False
        seen = {op}
        queue = deque()
        for ch in node["children"]:
            if ch not in seen:
                seen.add(ch)
                queue.append(ch)
        while not reached_end:
            if not queue:
                break
            n = queue.popleft()
            kind = graph[n]["kind"]
            if kind == "comm":
                reached_end = True
            else:
                if kind in ("matmul", "attention"):
                    cache_sum += int(graph[n]["mem"])
                    if cache_sum < cache_size:
                        plan[op].append(n)
                    else:
                        reached_end = True
                for ch in graph[n]["children"]:
                    if ch not in seen:
                        seen.add(ch)
                        queue.append(ch)
    return plan


def truncate_plan(node_bytes: Sequence[int], cache_size: int, granule: int = 128) -> List[int]:
    """Leading-bytes variant (not in the paper): same walk over an ordered node
    list, but the first node that does not fit is prefetched for its first
    (C - cacheSum_before) bytes rounded down to `granule`, then the walk stops.
    Returns prefetched bytes per node."""
    out = [0] * len(node_bytes)
    cache_sum = 0
    for i, nb in enumerate(node_bytes):
        if cache_sum + nb < cache_size:
            out[i] = nb
            cache_sum += nb
        else:
            room = max(cache_size - cache_sum, 0)
            out[i] = min(nb, (room // granule) * granule)
            break
    return out


def layer_graph(hidden: int, n_q_heads: int, n_kv_heads: int, head_dim: int, ffn: int,
                kv_tokens: int, n_layers: int = 1) -> List[dict]:
    """The op graph of n_layers decoder layers of one shard, as Algorithm 1 sees it.

    kv_tokens = sum over the batch of tokens already cached.  q/k/v and gate/up
    are fused nodes, so the order among siblings is the consumption order.
    A closing communication op stands for the next layer's first window.
    """
    g: List[dict] = []

    def add(kind, mem=0):
        g.append({"kind": kind, "mem": mem, "children": []})
        if len(g) > 1:
            g[-2]["children"].append(len(g) - 1)

    d = head_dim
    for _ in range(n_layers):
        add("comm")                                                        # window A
        add("matmul", 2 * hidden * (n_q_heads + 2 * n_kv_heads) * d)        # Wqkv
        add("other")                                                       # rope + append
        add("attention", 2 * 2 * kv_tokens * n_kv_heads * d)                # K and V
        add("matmul", 2 * n_q_heads * d * hidden)                           # Wo
        add("comm")                                                        # window B
        add("matmul", 2 * hidden * 2 * ffn)                                 # Wgate|up
        add("other")                                                       # activation
        add("matmul", 2 * ffn * hidden)                                     # Wdown
    add("comm")
    return g
