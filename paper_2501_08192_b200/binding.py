"""Thin ctypes binding over libpreserve.so (same names as include/preserve.h).

Argument marshalling only: every step of the decode path runs inside the CUDA
library.  torch is used for device memory and streams.  There is no CPU
fallback: if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpreserve.so")

PRESERVE_OK = 0
PRESERVE_EINVAL, PRESERVE_EALIGN, PRESERVE_ESHAPE, PRESERVE_ENOMEM = -1, -2, -3, -4
PRESERVE_ECUDA, PRESERVE_EARCH, PRESERVE_ETIMEOUT, PRESERVE_ETOOBIG = -5, -6, -7, -8
STATIC_SCRATCH_BYTES = 8 << 20
PLAN_WHOLE_NODE, PLAN_TRUNCATE = 0, 1
FLAG_NO_GRAPH, FLAG_PERSIST_L2, FLAG_NO_EARLY_LAUNCH, FLAG_FORCE_GEMV, FLAG_FORCE_TENSOR = 1, 2, 4, 8, 16
FLAG_INT8_WEIGHTS = 32
FLAG_INT8_KV = 64
DEBUG_WITHHOLD, DEBUG_WAIT_LIMIT_CYCLES = 0, 1
WITHHOLD_WINDOW, WITHHOLD_GEMV, WITHHOLD_TENSOR, WITHHOLD_ATTENTION = 1, 2, 3, 4

EXPORTS = (
    "preserve_layer_init", "preserve_set_prefetch_bytes", "preserve_set_plan_mode", "preserve_decode_step",
    "preserve_decode_chain", "preserve_decode_step_host", "preserve_layer_get_info", "preserve_last_status",
    "preserve_last_cuda_error", "preserve_debug_copy", "preserve_layer_destroy", "preserve_strerror",
    "preserve_plan_window", "preserve_algorithmic_bytes", "preserve_profile_step",
    "preserve_run_kernel", "preserve_set_trace", "preserve_read_trace",
    "preserve_set_window_delay_ns", "preserve_attention_static",
    "preserve_measure_read_bandwidth", "preserve_set_prefetch_mechanism", "preserve_clear_status",
    "preserve_graph_captures", "preserve_debug_set", "preserve_attention_static_status", "preserve_plan_graph", "preserve_measure_stream",
    "preserve_last_status_code", "preserve_comm_create", "preserve_comm_export", "preserve_comm_import",
    "preserve_comm_set_peer", "preserve_comm_write", "preserve_comm_debug_arrive", "preserve_comm_epoch",
    "preserve_comm_destroy", "preserve_layer_set_comm", "preserve_layer_set_external_attention_sum",
    "preserve_prefetch_window", "preserve_measure_stream_tma", "preserve_kv8_layout",
)
NODE_COMM, NODE_MATMUL, NODE_ATTENTION, NODE_OTHER = 0, 1, 2, 3
TRACE_SLOTS = 8
KERNEL_NAMES = ("window_a", "qkv_proj", "attn_splitkv", "attn_merge", "o_proj", "window_b", "gate_up_proj",
                "down_proj")


class LayerConfig(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("ffn", C.c_int32), ("tp_degree", C.c_int32),
                ("max_batch", C.c_int32), ("max_ctx", C.c_int32), ("rms_eps", C.c_float),
                ("rope_theta", C.c_float), ("flags", C.c_uint32)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_q", "w_k", "w_v", "w_o", "w_gate", "w_up", "w_down",
                                           "g_attn", "g_mlp")]


class StepIO(C.Structure):
    _fields_ = [("batch", C.c_int32), ("ctx_len", C.c_void_p), ("ctx_len_host", C.c_void_p),
                ("partials_in", C.POINTER(C.c_void_p)), ("attn_peer_partials", C.POINTER(C.c_void_p)),
                ("residual_in", C.c_void_p), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
                ("residual_out", C.c_void_p), ("mlp_partial_out", C.c_void_p),
                ("attn_partial_out", C.c_void_p)]


class HostIO(C.Structure):
    _fields_ = [("batch", C.c_int32), ("ctx_len_host", C.c_void_p),
                ("partials_in", C.POINTER(C.c_void_p)), ("attn_peer_partials", C.POINTER(C.c_void_p)),
                ("residual_in", C.c_void_p), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
                ("residual_out", C.c_void_p), ("mlp_partial_out", C.c_void_p)]


class Info(C.Structure):
    _fields_ = [("sm_count", C.c_int32), ("l2_bytes", C.c_int32), ("max_persisting_l2_bytes", C.c_int32),
                ("max_access_window_bytes", C.c_int32), ("uses_tensor_path", C.c_int32),
                ("activation_rows", C.c_int32), ("plan_mode", C.c_int32), ("normed_activations_fp16", C.c_int32),
                ("prefetch_budget", C.c_uint64),
                ("weight_bytes", C.c_uint64 * 4), ("kv_bytes", C.c_uint64),
                ("planned_bytes", (C.c_uint64 * 3) * 2), ("algorithmic_bytes", C.c_uint64)]


_lib = None


def lib() -> C.CDLL:
    """Load libpreserve.so (built by paper_2501_08192_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: run `python -m paper_2501_08192_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        L.preserve_layer_init.argtypes = [C.POINTER(LayerConfig), C.POINTER(LayerWeights), C.POINTER(C.c_void_p)]
        L.preserve_set_prefetch_bytes.argtypes = [C.c_void_p, C.c_size_t]
        L.preserve_set_plan_mode.argtypes = [C.c_void_p, C.c_int]
        L.preserve_set_window_delay_ns.argtypes = [C.c_void_p, C.c_int32]
        L.preserve_decode_step.argtypes = [C.c_void_p, C.POINTER(StepIO), C.c_void_p]
        L.preserve_decode_chain.argtypes = [C.POINTER(C.c_void_p), C.c_int32, C.POINTER(StepIO), C.c_int32,
                                            C.c_void_p]
        L.preserve_decode_step_host.argtypes = [C.c_void_p, C.POINTER(HostIO), C.c_void_p]
        L.preserve_profile_step.argtypes = [C.c_void_p, C.POINTER(StepIO), C.c_void_p, C.POINTER(C.c_float)]
        L.preserve_run_kernel.argtypes = [C.c_void_p, C.POINTER(StepIO), C.c_int32, C.c_void_p]
        L.preserve_prefetch_window.argtypes = [C.c_void_p, C.POINTER(StepIO), C.c_int32, C.c_void_p]
        L.preserve_set_trace.argtypes = [C.c_void_p, C.c_int32]
        L.preserve_read_trace.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        L.preserve_attention_static.argtypes = [C.c_void_p] * 6 + [C.c_int32] * 4 + [C.c_void_p] * 3
        L.preserve_measure_read_bandwidth.argtypes = [C.c_void_p, C.c_size_t, C.c_int32, C.c_void_p,
                                                      C.POINTER(C.c_float)]
        L.preserve_set_prefetch_mechanism.argtypes = [C.c_void_p, C.c_int32, C.c_uint32, C.c_int32]
        L.preserve_clear_status.argtypes = [C.c_void_p]
        L.preserve_graph_captures.argtypes = [C.c_void_p]
        L.preserve_graph_captures.restype = C.c_int64
        L.preserve_debug_set.argtypes = [C.c_void_p, C.c_int32, C.c_int64]
        L.preserve_attention_static_status.argtypes = []
        L.preserve_measure_stream.argtypes = [C.c_void_p, C.c_size_t, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                              C.c_uint32, C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(C.c_float)]
        L.preserve_last_status_code.argtypes = [C.c_void_p]
        L.preserve_kv8_layout.argtypes = [C.POINTER(LayerConfig), C.POINTER(C.c_uint64), C.POINTER(C.c_int32),
                                          C.POINTER(C.c_uint64)]
        L.preserve_comm_create.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_void_p)]
        L.preserve_comm_export.argtypes = [C.c_void_p, C.c_void_p]
        L.preserve_comm_import.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.preserve_comm_set_peer.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.preserve_comm_write.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]
        L.preserve_comm_debug_arrive.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_uint32]
        L.preserve_comm_epoch.argtypes = [C.c_void_p, C.c_int32]
        L.preserve_comm_epoch.restype = C.c_int64
        L.preserve_comm_destroy.argtypes = [C.c_void_p]
        L.preserve_comm_destroy.restype = None
        L.preserve_layer_set_comm.argtypes = [C.c_void_p, C.c_void_p]
        L.preserve_layer_set_external_attention_sum.argtypes = [C.c_void_p, C.c_void_p]
        L.preserve_measure_stream_tma.argtypes = [C.c_void_p, C.c_size_t, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                                  C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(C.c_float)]
        L.preserve_layer_get_info.argtypes = [C.c_void_p, C.POINTER(Info)]
        L.preserve_last_status.argtypes = [C.c_void_p]
        L.preserve_last_cuda_error.argtypes = [C.c_void_p]
        L.preserve_debug_copy.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]
        L.preserve_layer_destroy.argtypes = [C.c_void_p]
        L.preserve_layer_destroy.restype = None
        L.preserve_strerror.argtypes = [C.c_int]
        L.preserve_strerror.restype = C.c_char_p
        L.preserve_plan_window.argtypes = [C.POINTER(C.c_uint64), C.c_int32, C.c_uint64, C.c_int32,
                                           C.POINTER(C.c_uint64)]
        L.preserve_plan_graph.argtypes = [C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_uint64),
                                          C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_uint64, C.c_int32,
                                          C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                          C.POINTER(C.c_uint64), C.POINTER(C.c_int32)]
        L.preserve_algorithmic_bytes.argtypes = [C.POINTER(LayerConfig), C.c_int32, C.c_uint64]
        L.preserve_algorithmic_bytes.restype = C.c_uint64
        _lib = L
    return _lib


class PreserveError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {preserve_strerror(code)} ({code})")


def _check(code: int, what: str) -> None:
    if code != PRESERVE_OK:
        raise PreserveError(code, what)


def preserve_strerror(code: int) -> str:
    return lib().preserve_strerror(code).decode()


def preserve_plan_window(node_bytes: Sequence[int], budget: int, mode: int = PLAN_WHOLE_NODE) -> List[int]:
    n = len(node_bytes)
    src = (C.c_uint64 * max(n, 1))(*node_bytes)
    dst = (C.c_uint64 * max(n, 1))()
    _check(lib().preserve_plan_window(src, n, budget, mode, dst), "preserve_plan_window")
    return [int(dst[i]) for i in range(n)]


def preserve_plan_graph(kinds: Sequence[int], mem_bytes: Sequence[int], children: Sequence[Sequence[int]],
                        budget: int, mode: int = PLAN_WHOLE_NODE):
    """Algorithm 1 over an explicit graph; returns [(comm op, node, bytes), ...] in insertion order."""
    n = len(kinds)
    off = [0]
    flat: List[int] = []
    for ch in children:
        flat.extend(ch)
        off.append(len(flat))
    k = (C.c_int32 * max(n, 1))(*kinds)
    m = (C.c_uint64 * max(n, 1))(*mem_bytes)
    so = (C.c_int32 * (n + 1))(*off)
    su = (C.c_int32 * max(len(flat), 1))(*flat)
    cap = max(n * max(1, sum(1 for x in kinds if x == NODE_COMM)), 1)
    oc, on, ob = (C.c_int32 * cap)(), (C.c_int32 * cap)(), (C.c_uint64 * cap)()
    cnt = C.c_int32()
    _check(lib().preserve_plan_graph(n, k, m, so, su, budget, mode, cap, oc, on, ob, C.byref(cnt)),
           "preserve_plan_graph")
    return [(int(oc[i]), int(on[i]), int(ob[i])) for i in range(cnt.value)]


def make_config(shape, max_batch: Optional[int] = None, max_ctx: Optional[int] = None, flags: int = 0) -> LayerConfig:
    """LayerConfig from an inputs.ShardShape-like object."""
    return LayerConfig(shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn,
                       shape.tp_degree, shape.batch if max_batch is None else max_batch,
                       shape.ctx if max_ctx is None else max_ctx, shape.rms_eps, shape.rope_theta, flags)


def preserve_kv8_layout(cfg: LayerConfig):
    """(scale_offset_bytes, scale_capacity, buffer_bytes) of one int8 cache buffer for `cfg`."""
    off, cap, tot = C.c_uint64(), C.c_int32(), C.c_uint64()
    _check(lib().preserve_kv8_layout(C.byref(cfg), C.byref(off), C.byref(cap), C.byref(tot)), "preserve_kv8_layout")
    return int(off.value), int(cap.value), int(tot.value)


def preserve_algorithmic_bytes(cfg: LayerConfig, batch: int, sum_ctx: int) -> int:
    return int(lib().preserve_algorithmic_bytes(C.byref(cfg), batch, sum_ctx))


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _stream_ptr(stream) -> int:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


class Layer:
    """Owns one preserve_layer_t handle.  Methods mirror the C entry points."""

    def __init__(self, cfg: LayerConfig, weights: dict):
        """weights: name -> CUDA bf16 tensor ([in,out] row-major) for w_q..w_down, g_attn, g_mlp."""
        self.cfg = cfg
        for n, _ in LayerWeights._fields_:
            if not weights[n].is_contiguous():
                raise ValueError(f"weight {n} must be contiguous")
        w = LayerWeights(*[_ptr(weights[n]) for n, _ in LayerWeights._fields_])
        h = C.c_void_p()
        _check(lib().preserve_layer_init(C.byref(cfg), C.byref(w), C.byref(h)), "preserve_layer_init")
        self.handle = h
        self._keep = []

    def close(self) -> None:
        if self.handle:
            lib().preserve_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_prefetch_bytes(self, n: int) -> None:
        _check(lib().preserve_set_prefetch_bytes(self.handle, n), "preserve_set_prefetch_bytes")

    def set_window_delay_ns(self, ns: int) -> None:
        _check(lib().preserve_set_window_delay_ns(self.handle, ns), "preserve_set_window_delay_ns")

    def set_plan_mode(self, mode: int) -> None:
        _check(lib().preserve_set_plan_mode(self.handle, mode), "preserve_set_plan_mode")

    def make_io(self, batch, ctx_len_dev, ctx_len_host, partials_in, attn_peer_partials, residual_in,
                k_cache, v_cache, residual_out, mlp_partial_out, attn_partial_out=None) -> StepIO:
        """Marshal tensors into a StepIO.  ctx_len_host: int32 numpy array or CPU tensor (kept alive here)."""
        P = self.cfg.tp_degree
        parts = (C.c_void_p * P)(*[_ptr(t) for t in partials_in])
        peers = (C.c_void_p * max(P - 1, 1))(*[_ptr(t) for t in attn_peer_partials])
        host_ptr = ctx_len_host.ctypes.data if hasattr(ctx_len_host, "ctypes") else ctx_len_host.data_ptr()
        io = StepIO(batch, _ptr(ctx_len_dev), host_ptr, parts, peers, _ptr(residual_in), _ptr(k_cache),
                    _ptr(v_cache), _ptr(residual_out), _ptr(mlp_partial_out), _ptr(attn_partial_out))
        io._keep = (parts, peers, ctx_len_host, ctx_len_dev, partials_in, attn_peer_partials, residual_in,
                    k_cache, v_cache, residual_out, mlp_partial_out, attn_partial_out)
        return io

    def decode_step(self, io: StepIO, stream=None) -> None:
        _check(lib().preserve_decode_step(self.handle, C.byref(io), _stream_ptr(stream)), "preserve_decode_step")

    def decode_step_host(self, io: HostIO, stream=None) -> None:
        _check(lib().preserve_decode_step_host(self.handle, C.byref(io), _stream_ptr(stream)),
               "preserve_decode_step_host")

    def profile_step(self, io: StepIO, stream=None) -> List[float]:
        """Per-kernel milliseconds of one step (order: KERNEL_NAMES); synchronises the stream."""
        ms = (C.c_float * len(KERNEL_NAMES))()
        _check(lib().preserve_profile_step(self.handle, C.byref(io), _stream_ptr(stream), ms),
               "preserve_profile_step")
        return [float(v) for v in ms]

    def run_kernel(self, io: StepIO, which: int, stream=None) -> None:
        _check(lib().preserve_run_kernel(self.handle, C.byref(io), which, _stream_ptr(stream)), "preserve_run_kernel")

    def prefetch_window(self, io: StepIO, window: int, stream=None) -> None:
        _check(lib().preserve_prefetch_window(self.handle, C.byref(io), window, _stream_ptr(stream)),
               "preserve_prefetch_window")

    def set_trace(self, on: bool) -> None:
        _check(lib().preserve_set_trace(self.handle, 1 if on else 0), "preserve_set_trace")

    def read_trace(self):
        """Per kernel: (first start, first wait-return, last wait-return, last end, last start,
        last end of the streaming loop, first end, unused), ns of the GPU global timer."""
        buf = (C.c_int64 * (TRACE_SLOTS * len(KERNEL_NAMES)))()
        _check(lib().preserve_read_trace(self.handle, buf), "preserve_read_trace")
        return [tuple(int(buf[TRACE_SLOTS * k + i]) for i in range(TRACE_SLOTS)) for k in range(len(KERNEL_NAMES))]

    def get_info(self) -> Info:
        info = Info()
        _check(lib().preserve_layer_get_info(self.handle, C.byref(info)), "preserve_layer_get_info")
        return info

    def last_status(self) -> int:
        return int(lib().preserve_last_status(self.handle))

    def last_status_code(self) -> int:
        return int(lib().preserve_last_status_code(self.handle))

    def set_comm(self, comm) -> None:
        _check(lib().preserve_layer_set_comm(self.handle, comm.handle if comm is not None else None),
               "preserve_layer_set_comm")
        self._comm = comm

    def set_external_attention_sum(self, t) -> None:
        _check(lib().preserve_layer_set_external_attention_sum(self.handle, _ptr(t)),
               "preserve_layer_set_external_attention_sum")
        self._ext = t

    def clear_status(self) -> None:
        _check(lib().preserve_clear_status(self.handle), "preserve_clear_status")

    def graph_captures(self) -> int:
        return int(lib().preserve_graph_captures(self.handle))

    def set_prefetch_mechanism(self, mechanism: int, chunk_bytes: int = 4096, ctas: int = 128) -> None:
        _check(lib().preserve_set_prefetch_mechanism(self.handle, mechanism, chunk_bytes, ctas),
               "preserve_set_prefetch_mechanism")

    def debug_set(self, what: int, value: int) -> None:
        _check(lib().preserve_debug_set(self.handle, what, value), "preserve_debug_set")

    def last_cuda_error(self) -> int:
        return int(lib().preserve_last_cuda_error(self.handle))

    def debug_copy(self, which: int, dst, stream=None) -> None:
        _check(lib().preserve_debug_copy(self.handle, which, _ptr(dst), dst.numel() * dst.element_size(),
                                         _stream_ptr(stream)), "preserve_debug_copy")


def preserve_attention_static(q_hi, q_lo, k_cache, v_cache, ctx_len_dev, ctx_len_host, n_q_heads: int,
                              n_kv_heads: int, o_hi, o_lo, stream=None) -> int:
    """Allocation-free decode attention; returns the PRESERVE_* code (see preserve.h).

    Tensors: q_hi/q_lo/o_hi/o_lo CUDA bf16 [batch, n_q_heads, 128]; caches CUDA bf16
    [batch, n_kv_heads, capacity, 128]; ctx_len_dev CUDA int32 [batch]; ctx_len_host int32 numpy array."""
    batch, _, cap, _ = k_cache.shape
    return int(lib().preserve_attention_static(_ptr(q_hi), _ptr(q_lo), _ptr(k_cache), _ptr(v_cache),
                                               _ptr(ctx_len_dev), ctx_len_host.ctypes.data, batch, n_q_heads,
                                               n_kv_heads, cap, _ptr(o_hi), _ptr(o_lo), _stream_ptr(stream)))


class Comm:
    """Owns one preserve_comm_t: this rank's exchange block of the real communication window."""

    def __init__(self, rank: int, n_ranks: int, max_batch: int, hidden: int):
        h = C.c_void_p()
        _check(lib().preserve_comm_create(rank, n_ranks, max_batch, hidden, C.byref(h)), "preserve_comm_create")
        self.handle, self.rank, self.n_ranks = h, rank, n_ranks
        self._peers = []

    def export_handle(self) -> bytes:
        buf = (C.c_uint8 * 64)()
        _check(lib().preserve_comm_export(self.handle, buf), "preserve_comm_export")
        return bytes(buf)

    def import_handle(self, peer_rank: int, handle: bytes) -> None:
        buf = (C.c_uint8 * 64)(*handle)
        _check(lib().preserve_comm_import(self.handle, peer_rank, buf), "preserve_comm_import")

    def set_peer(self, peer: "Comm") -> None:
        _check(lib().preserve_comm_set_peer(self.handle, peer.rank, peer.handle), "preserve_comm_set_peer")
        self._peers.append(peer)

    def write(self, window: int, t, stream=None) -> None:
        _check(lib().preserve_comm_write(self.handle, window, _ptr(t), t.numel() * t.element_size(),
                                         _stream_ptr(stream)), "preserve_comm_write")

    def debug_arrive(self, window: int, from_rank: int, epoch: int) -> None:
        _check(lib().preserve_comm_debug_arrive(self.handle, window, from_rank, epoch), "preserve_comm_debug_arrive")

    def epoch(self, window: int) -> int:
        return int(lib().preserve_comm_epoch(self.handle, window))

    def close(self) -> None:
        if self.handle:
            lib().preserve_comm_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def preserve_attention_static_status() -> int:
    return int(lib().preserve_attention_static_status())


def preserve_measure_read_bandwidth(buf, reps: int = 10, stream=None) -> float:
    """GB/s of a pure 128-bit read stream over the CUDA tensor `buf` (see preserve.h)."""
    out = C.c_float()
    _check(lib().preserve_measure_read_bandwidth(_ptr(buf), buf.numel() * buf.element_size(), reps,
                                                 _stream_ptr(stream), C.byref(out)),
           "preserve_measure_read_bandwidth")
    return float(out.value)


def preserve_measure_stream(buf, n_bytes: int, passes: int, path: int, ctas: int, stages: int = 6,
                            chunk_bytes: int = 16384, status=None, stream=None, producers: int = 1) -> float:
    """GB/s of the single-launch streaming microbenchmark over the first n_bytes of `buf` (see preserve.h).
    `status`: CUDA int32 tensor of 64 zeros."""
    out = C.c_float()
    _check(lib().preserve_measure_stream(_ptr(buf), n_bytes, passes, path, ctas, stages, chunk_bytes, producers,
                                         _ptr(status), _stream_ptr(stream), C.byref(out)), "preserve_measure_stream")
    return float(out.value)


def preserve_measure_stream_tma(buf, n_bytes: int, passes: int, ctas: int, stages: int, box_rows: int,
                                producers: int, status, stream=None) -> float:
    """GB/s of 2-D tiled TMA loads (the tcgen05 GEMM's weight loads) over `buf` (see preserve.h)."""
    out = C.c_float()
    _check(lib().preserve_measure_stream_tma(_ptr(buf), n_bytes, passes, ctas, stages, box_rows, producers,
                                             _ptr(status), _stream_ptr(stream), C.byref(out)),
           "preserve_measure_stream_tma")
    return float(out.value)


def preserve_decode_chain(layers: Sequence[Layer], ios: Sequence[StepIO], link: bool, stream=None) -> None:
    n = len(layers)
    hs = (C.c_void_p * n)(*[l.handle for l in layers])
    arr = (StepIO * n)(*ios)
    _check(lib().preserve_decode_chain(hs, n, arr, 1 if link else 0, _stream_ptr(stream)), "preserve_decode_chain")


def make_host_io(cfg: LayerConfig, batch, ctx_len_host, partials_in, attn_peer_partials, residual_in,
                 k_cache, v_cache, residual_out, mlp_partial_out) -> HostIO:
    """HostIO from pinned CPU tensors (activations) and CUDA tensors (caches)."""
    P = cfg.tp_degree
    parts = (C.c_void_p * P)(*[_ptr(t) for t in partials_in])
    peers = (C.c_void_p * max(P - 1, 1))(*[_ptr(t) for t in attn_peer_partials])
    host_ptr = ctx_len_host.ctypes.data if hasattr(ctx_len_host, "ctypes") else ctx_len_host.data_ptr()
    io = HostIO(batch, host_ptr, parts, peers, _ptr(residual_in), _ptr(k_cache), _ptr(v_cache),
                _ptr(residual_out), _ptr(mlp_partial_out))
    io._keep = (parts, peers, ctx_len_host, partials_in, attn_peer_partials, residual_in, k_cache, v_cache,
                residual_out, mlp_partial_out)
    return io
