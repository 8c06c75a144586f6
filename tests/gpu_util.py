"""Helpers for the GPU parity tests: move seeded inputs to the device, run the
CUDA path through the C ABI, and compare with the CPU oracle."""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np
import torch

from paper_2501_08192_b200 import binding as P
from paper_2501_08192_b200 import inputs as I

GUARD = 64          # canary elements on each side of every output buffer
CANARY = 0x7B7B     # bf16 bit pattern written into the guard bands


def bits_to_cuda(a: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bf16 tensor with the same bits."""
    t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()
    return t.view(torch.bfloat16)


def cuda_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def cuda_to_f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


class GuardedOut:
    """A bf16 output buffer with canary bands in front and behind."""

    def __init__(self, shape):
        n = int(np.prod(shape))
        self.n = n
        self.shape = tuple(shape)
        raw = torch.full((n + 2 * GUARD,), 0, dtype=torch.int16, device="cuda")
        raw[:] = CANARY
        self.raw = raw
        self.t = raw[GUARD:GUARD + n].view(torch.bfloat16).view(*shape)

    def guards_intact(self) -> bool:
        r = self.raw.cpu().numpy().view(np.uint16)
        return bool((r[:GUARD] == CANARY).all() and (r[GUARD + self.n:] == CANARY).all())


def kv8_buffer(cfg, codes: np.ndarray, scales: np.ndarray) -> torch.Tensor:
    """One int8 cache buffer on the device in the library's layout: the codes, then the scales."""
    off, scap, total = P.preserve_kv8_layout(cfg)
    B, nkv, cap, d = codes.shape
    buf = torch.zeros(total, dtype=torch.uint8, device="cuda")
    buf[:codes.size] = torch.from_numpy(np.ascontiguousarray(codes).view(np.uint8).reshape(-1)).cuda()
    padded = np.full((B, nkv, scap), np.nan, np.float32)
    padded[:, :, :cap] = scales
    buf[off:off + padded.size * 4] = torch.from_numpy(padded.view(np.uint8).reshape(-1)).cuda()
    return buf


def kv8_read(cfg, buf: torch.Tensor, B: int, nkv: int, cap: int, d: int):
    """(codes int8 [B,nkv,cap,d], scales f32 [B,nkv,cap]) back from a device cache buffer."""
    off, scap, _ = P.preserve_kv8_layout(cfg)
    raw = buf.cpu().numpy()
    codes = raw[:B * nkv * cap * d].view(np.int8).reshape(B, nkv, cap, d)
    scales = raw[off:off + B * nkv * scap * 4].view(np.float32).reshape(B, nkv, scap)[:, :, :cap]
    return codes.copy(), scales.copy()


class DeviceLayer:
    """One layer instance on the device: library handle, inputs, outputs.  kv8 = the int8 cache of
    inputs.make_int8_cache: the layer is then created with FLAG_INT8_KV and runs over that cache."""

    def __init__(self, shape: I.ShardShape, t: Dict[str, np.ndarray], flags: int = 0,
                 max_batch: Optional[int] = None, kv8: Optional[Dict[str, np.ndarray]] = None):
        self.shape = shape
        self.t = t
        self.kv8 = kv8
        if kv8 is not None:
            flags |= P.FLAG_INT8_KV
        self.cfg = P.make_config(shape, max_batch=max_batch, flags=flags)
        names = ("w_q", "w_k", "w_v", "w_o", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")
        w = {n: bits_to_cuda(t[n]) for n in names}
        self.layer = P.Layer(self.cfg, w)
        del w
        B, H = shape.batch, shape.hidden
        self.partials = [bits_to_cuda(t["partials_in"][p]) for p in range(shape.tp_degree)]
        self.peers = [bits_to_cuda(t["attn_peer_partials"][p]) for p in range(shape.tp_degree - 1)]
        self.residual = bits_to_cuda(t["residual_in"])
        if kv8 is None:
            self.k_cache = bits_to_cuda(t["k_cache"])
            self.v_cache = bits_to_cuda(t["v_cache"])
        else:
            self.k_cache = kv8_buffer(self.cfg, kv8["k_codes"], kv8["k_scales"])
            self.v_cache = kv8_buffer(self.cfg, kv8["v_codes"], kv8["v_scales"])
        self.ctx_host = np.ascontiguousarray(t["ctx_len"], dtype=np.int32)
        self.ctx_dev = torch.from_numpy(self.ctx_host).cuda()
        self.residual_out = GuardedOut((B, H))
        self.mlp_out = GuardedOut((B, H))
        self.attn_out = GuardedOut((B, H))
        self.io = self.layer.make_io(B, self.ctx_dev, self.ctx_host, self.partials, self.peers, self.residual,
                                     self.k_cache, self.v_cache, self.residual_out.t, self.mlp_out.t,
                                     self.attn_out.t)

    def run(self, stream=None) -> None:
        self.layer.decode_step(self.io, stream)

    def outputs(self) -> Dict[str, np.ndarray]:
        torch.cuda.synchronize()
        return {"h2": cuda_to_f32(self.residual_out.t), "mlp_partial": cuda_to_f32(self.mlp_out.t),
                "attn_partial": cuda_to_f32(self.attn_out.t)}

    def output_bits(self) -> Dict[str, np.ndarray]:
        torch.cuda.synchronize()
        return {"h2": cuda_to_bits(self.residual_out.t), "mlp_partial": cuda_to_bits(self.mlp_out.t),
                "attn_partial": cuda_to_bits(self.attn_out.t)}

    def intermediates(self) -> Dict[str, np.ndarray]:
        """h, x, q, o, x2, a of the last step as fp32 (split activations are summed hi + lo)."""
        s = self.shape
        B, H, nq, d, F = s.batch, s.hidden, s.n_q_heads, s.head_dim, s.ffn
        rows = int(self.layer.get_info().activation_rows)
        out = {}
        buf = torch.empty((self.cfg.max_batch, H), dtype=torch.float32, device="cuda")
        self.layer.debug_copy(0, buf)
        torch.cuda.synchronize()
        out["h"] = buf[:B].cpu().numpy()
        spec = {"x": (1, (H,)), "q": (2, (nq, d)), "o": (3, (nq, d)), "x2": (4, (H,)), "a": (5, (F,))}
        fp16_x = bool(self.layer.get_info().normed_activations_fp16)
        for name, (which, tail) in spec.items():
            if fp16_x and name in ("o", "x2", "a"):   # one fp16 plane on the tensor path
                buf = torch.empty((rows,) + tail, dtype=torch.float16, device="cuda")
                self.layer.debug_copy(which, buf)
                torch.cuda.synchronize()
                out[name] = buf[:B].float().cpu().numpy()
                continue
            # (tensor path: x is hi + lo fp16 planes; everything else hi + lo bf16 planes)
            dt = torch.float16 if (fp16_x and name == "x") else torch.bfloat16
            buf = torch.empty((2, rows) + tail, dtype=dt, device="cuda")
            self.layer.debug_copy(which, buf)
            torch.cuda.synchronize()
            out[name] = (buf[0, :B].double() + buf[1, :B].double()).float().cpu().numpy()
        return out

    def appended_kv(self):
        """The cache slot written by the step, per sequence: (k [B,nkv,d], v [B,nkv,d]) as fp32."""
        torch.cuda.synchronize()
        kc, vc = cuda_to_f32(self.k_cache), cuda_to_f32(self.v_cache)
        idx = self.ctx_host
        k = np.stack([kc[b, :, idx[b]] for b in range(self.shape.batch)])
        v = np.stack([vc[b, :, idx[b]] for b in range(self.shape.batch)])
        return k, v

    def appended_kv8(self):
        """int8 cache: the slot written by the step, per sequence: (k codes [B,nkv,d], k scales [B,nkv],
        v codes, v scales)."""
        torch.cuda.synchronize()
        s = self.shape
        out = []
        for buf in (self.k_cache, self.v_cache):
            codes, scales = kv8_read(self.cfg, buf, s.batch, s.n_kv_heads, s.kv_capacity, s.head_dim)
            out.append(np.stack([codes[b, :, self.ctx_host[b]] for b in range(s.batch)]))
            out.append(np.stack([scales[b, :, self.ctx_host[b]] for b in range(s.batch)]))
        return tuple(out)

    def close(self) -> None:
        self.layer.close()


def tolerance_ok(got: np.ndarray, ref: np.ndarray):
    """|got - ref| <= atol + 1e-2 |ref| with atol = 2e-2 * min(1, rms(ref)).

    The absolute term is scaled by the tensor's rms because this shard's partial
    sums are small (weights ~ N(0, 0.02)): an unscaled 2e-2 would accept noise."""
    got = np.asarray(got, np.float64).reshape(-1)
    ref = np.asarray(ref, np.float64).reshape(-1)
    rms = float(np.sqrt(np.mean(ref * ref))) if ref.size else 0.0
    atol = 2e-2 * min(1.0, rms)
    err = np.abs(got - ref)
    bound = atol + 1e-2 * np.abs(ref)
    bad = ~(err <= bound)        # catches NaN too
    worst = float((err / np.maximum(bound, 1e-30)).max()) if err.size else 0.0
    return (not bad.any()), int(bad.sum()), worst, rms


def assert_close(got, ref, name: str):
    ok, nbad, worst, rms = tolerance_ok(got, ref)
    assert ok, f"{name}: {nbad} elements out of tolerance (worst err/bound {worst:.3f}, rms(ref) {rms:.4g})"
