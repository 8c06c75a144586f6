// Row orderings of the packed weights and the fused GEMM epilogues that rely on
// them.  A skinny GEMM produces, for every batch row b, pairs of outputs
// (v0, v1) that the epilogue needs together:
//   PLAIN : two independent outputs;
//   QKV   : head dims i and i + d/2 of one head (the rotary pair); q goes to the
//           query buffer, k and v are appended to the cache at slot ctx_len[b];
//   SWIGLU: gate_j and up_j  ->  silu(gate_j) * up_j.
// Packed row orders:
//   GEMV path  : 16-row blocks; rows r and r+8 (r < 8) of block rb are a pair.
//   tensor path: rows 2m and 2m+1 are a pair.
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"
#include "kernels.h"

namespace prsv {

// Logical coordinates of pair `pair` (GEMV path: pair = rb * 8 + r; tensor path: pair = m).
//   PLAIN : n0, n1 = output features of v0, v1
//   QKV   : n0 = head index over [q | k | v], n1 = i (first dim of the rotary pair)
//   SWIGLU: n0 = j
__host__ __device__ inline void pair_coords(int kind, bool tensor_path, int pair, int &n0, int &n1)
{
    if (kind == EPI_PLAIN) {
        if (tensor_path) { n0 = 2 * pair; n1 = 2 * pair + 1; }
        else { n0 = (pair >> 3) * 16 + (pair & 7); n1 = n0 + 8; }
    } else if (kind == EPI_QKV) {
        n0 = pair >> 6;          // 64 pairs per 128-dim head in either path
        n1 = pair & 63;
    } else {
        n0 = pair; n1 = 0;
    }
}

// Source matrix and column of packed row p (used by the packers).
// srcs are [K, cols_s] row-major; QKV: {w_q, w_k, w_v}; SWIGLU: {w_gate, w_up}; PLAIN: {w}.
__host__ __device__ inline void packed_row_source(int kind, bool tensor_path, int p, const int *src_cols,
                                                  int &src, int &col)
{
    int pair, member;
    if (tensor_path) { pair = p >> 1; member = p & 1; }
    else { pair = (p >> 4) * 8 + (p & 7); member = (p >> 3) & 1; }
    int n0, n1;
    pair_coords(kind, tensor_path, pair, n0, n1);
    if (kind == EPI_PLAIN) {
        src = 0; col = member ? n1 : n0;
    } else if (kind == EPI_QKV) {
        int f = n0 * kHeadDim + n1 + member * (kHeadDim / 2);
        src = 0;
        while (f >= src_cols[src]) { f -= src_cols[src]; ++src; }
        col = f;
    } else {
        src = member; col = n0;
    }
}

__device__ __forceinline__ void store_bf16(void *base, size_t idx, float v)
{
    reinterpret_cast<bf16 *>(base)[idx] = __float2bfloat16_rn(v);
}
// Activations that feed another GEMM are kept as hi + lo bf16 planes.
__device__ __forceinline__ void store_split(void *base, size_t plane, size_t idx, float v)
{
    const bf16 hi = __float2bfloat16_rn(v);
    reinterpret_cast<bf16 *>(base)[idx] = hi;
    reinterpret_cast<bf16 *>(base)[plane + idx] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// The QKV epilogue needs, per output, the sequence position and the rotary frequency of the pair.
// Both are inputs of the step (not results of earlier kernels), so a kernel copies them to shared
// memory once, before it waits for its predecessor, instead of chasing them through global memory
// for every output.
struct EpilogueTables {
    int pos[128];              // ctx_len[b0 + b], b < batch handled by the launch (at most 128)
    double inv_freq[kHeadDim / 2];
};
__device__ __forceinline__ void load_epilogue_tables(const EpilogueArgs &e, EpilogueTables &t, int b0, int nb)
{
    if (e.kind != EPI_QKV)
        return;
    for (int i = threadIdx.x; i < nb && i < 128; i += blockDim.x)
        t.pos[i] = e.ctx_len[b0 + i];
    for (int i = threadIdx.x; i < kHeadDim / 2; i += blockDim.x)
        t.inv_freq[i] = e.inv_freq ? e.inv_freq[i] : 0.0;
}

// Rotary factors (cos, sin) of rotary pair i at sequence position pos; (1, 0) for heads that are
// not rotated (values) and when the layer has no rotary embedding.
__device__ __forceinline__ float2 rope_trig(const EpilogueArgs &e, const EpilogueTables &tab, int pos, int hd, int i)
{
    if (!(hd < e.nq + e.nkv && e.inv_freq))
        return make_float2(1.f, 0.f);
    // angle = pos * theta^(-2i/d): the product and its reduction mod 2 pi need more than
    // fp32 (angles reach tens of thousands of radians); the reduced angle does not
    const double ang = (double)pos * tab.inv_freq[i];
    const double turns = rint(ang * 0.15915494309189535);
    const float red = (float)fma(-turns, 6.283185307179586, ang);
    // |red| <= pi: the hardware sine / cosine are within 2^-21 there, far inside the tolerance, and
    // cost two instructions instead of the library routine with its large-argument path
    float sf, cf;
    __sincosf(red, &sf, &cf);
    return make_float2(cf, sf);
}

// The QKV epilogue of one rotary pair with its factors given: rotate, then q to the query planes,
// k and v to the cache at slot pos.
__device__ __forceinline__ void epilogue_qkv(const EpilogueArgs &e, int pos, int b, int hd, int i, float v0, float v1,
                                             float2 cs)
{
    if (hd < e.nq + e.nkv && e.inv_freq) {
        const float r0 = v0 * cs.x - v1 * cs.y;
        const float r1 = v1 * cs.x + v0 * cs.y;
        v0 = r0; v1 = r1;
    }
    if (hd < e.nq) {
        const size_t o = ((size_t)b * e.nq + hd) * kHeadDim + i;
        store_split(e.q_out, e.q_plane, o, v0);
        store_split(e.q_out, e.q_plane, o + kHeadDim / 2, v1);
    } else {
        const bool is_k = hd < e.nq + e.nkv;
        const int kvh = is_k ? hd - e.nq : hd - e.nq - e.nkv;
        if (e.kv_new) {
            // int8 cache: the vector goes to the attention kernel unrounded, which quantises it
            float *dst = e.kv_new + (is_k ? 0 : e.kv_new_plane) + ((size_t)b * e.nkv + kvh) * kHeadDim + i;
            dst[0] = v0;
            dst[kHeadDim / 2] = v1;
            return;
        }
        const size_t o = (((size_t)b * e.nkv + kvh) * e.cap + pos) * kHeadDim + i;
        void *dst = is_k ? e.k_cache : e.v_cache;
        store_bf16(dst, o, v0);
        store_bf16(dst, o + kHeadDim / 2, v1);
    }
}

// Apply the epilogue KIND to one pair of fp32 results of batch row b (b_local = b - b0 indexes the
// tables).  The kind is a template argument so that a kernel instantiated for one kind carries only
// that kind's instructions.
template <int KIND>
__device__ __forceinline__ void apply_epilogue_t(const EpilogueArgs &e, const EpilogueTables &tab, int b_local,
                                                 bool tensor_path, int N, int b, int pair, float v0, float v1)
{
    int n0, n1;
    pair_coords(KIND, tensor_path, pair, n0, n1);
    if constexpr (KIND == EPI_PLAIN) {
        if (tensor_path) {
            // the pair's outputs are neighbours: one store per buffer
            const size_t o = (size_t)b * N + n0;
            if (e.out)
                *reinterpret_cast<uint32_t *>(reinterpret_cast<bf16 *>(e.out) + o) = pack_bf16(v0, v1);
            if (e.out2)
                *reinterpret_cast<uint32_t *>(reinterpret_cast<bf16 *>(e.out2) + o) = pack_bf16(v0, v1);
            if (e.out_f32)
                *reinterpret_cast<float2 *>(e.out_f32 + o) = make_float2(v0, v1);
            return;
        }
        if (e.out) {
            store_bf16(e.out, (size_t)b * N + n0, v0);
            store_bf16(e.out, (size_t)b * N + n1, v1);
        }
        if (e.out2) {
            store_bf16(e.out2, (size_t)b * N + n0, v0);
            store_bf16(e.out2, (size_t)b * N + n1, v1);
        }
        if (e.out_f32) {
            e.out_f32[(size_t)b * N + n0] = v0;
            e.out_f32[(size_t)b * N + n1] = v1;
        }
    } else if constexpr (KIND == EPI_SWIGLU) {
        // silu by the fast exponential and division (a few ulp; for v0 < -87 the quotient flushes to 0,
        // its true size being < 1e-36)
        const float a = __fdividef(v0, 1.f + __expf(-v0)) * v1;
        if (e.out_fp16)
            reinterpret_cast<__half *>(e.out)[(size_t)b * (N >> 1) + n0] = __float2half_rn(fminf(fmaxf(a, -65504.f), 65504.f));
        else
            store_split(e.out, e.out_plane, (size_t)b * (N >> 1) + n0, a);
    } else {
        const int pos = tab.pos[b_local];
        epilogue_qkv(e, pos, b, n0, n1, v0, v1, rope_trig(e, tab, pos, n0, n1));
    }
}
// The same with the kind read from the arguments.
__device__ __forceinline__ void apply_epilogue(const EpilogueArgs &e, const EpilogueTables &tab, int b_local,
                                               bool tensor_path, int N, int b, int pair, float v0, float v1)
{
    if (e.kind == EPI_PLAIN)
        apply_epilogue_t<EPI_PLAIN>(e, tab, b_local, tensor_path, N, b, pair, v0, v1);
    else if (e.kind == EPI_SWIGLU)
        apply_epilogue_t<EPI_SWIGLU>(e, tab, b_local, tensor_path, N, b, pair, v0, v1);
    else
        apply_epilogue_t<EPI_QKV>(e, tab, b_local, tensor_path, N, b, pair, v0, v1);
}

// Tensor path, two neighbouring pairs (pair0 even, and pair0 + 1) of batch row b at once:
// v = (v0, v1) of pair0 then (v0, v1) of pair0 + 1.  Their outputs are neighbours in every output
// buffer, so each buffer takes one vector store.  cs0 / cs1: the pairs' rotary factors when
// have_trig (QKV only), else computed here.
template <int KIND>
__device__ __forceinline__ void apply_epilogue_quad_t(const EpilogueArgs &e, const EpilogueTables &tab, int N, int b,
                                                      int pair0, float4 v, bool have_trig, float2 cs0, float2 cs1)
{
    if constexpr (KIND == EPI_PLAIN) {
        const size_t o = (size_t)b * N + 2 * (size_t)pair0;
        const uint2 packed = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
        if (e.out)
            *reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(e.out) + o) = packed;
        if (e.out2)
            *reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(e.out2) + o) = packed;
        if (e.out_f32)
            *reinterpret_cast<float4 *>(e.out_f32 + o) = v;
    } else if constexpr (KIND == EPI_SWIGLU) {
        const float a0 = __fdividef(v.x, 1.f + __expf(-v.x)) * v.y;
        const float a1 = __fdividef(v.z, 1.f + __expf(-v.z)) * v.w;
        const size_t o = (size_t)b * (N >> 1) + pair0;
        if (e.out_fp16) {
            *reinterpret_cast<__half2 *>(reinterpret_cast<__half *>(e.out) + o) =
                __floats2half2_rn(fminf(fmaxf(a0, -65504.f), 65504.f), fminf(fmaxf(a1, -65504.f), 65504.f));
            return;
        }
        uint32_t hi, lo;
        split_bf16x2(a0, a1, hi, lo);
        *reinterpret_cast<uint32_t *>(reinterpret_cast<bf16 *>(e.out) + o) = hi;
        *reinterpret_cast<uint32_t *>(reinterpret_cast<bf16 *>(e.out) + e.out_plane + o) = lo;
    } else {
        const int pos = tab.pos[b], hd = pair0 >> 6, i = pair0 & 63;
        if (!have_trig) {
            cs0 = rope_trig(e, tab, pos, hd, i);
            cs1 = rope_trig(e, tab, pos, hd, i + 1);
        }
        float a0 = v.x, a1 = v.y, c0 = v.z, c1 = v.w;     // dims i, i + d/2 and i + 1, i + 1 + d/2
        if (hd < e.nq + e.nkv && e.inv_freq) {
            a0 = v.x * cs0.x - v.y * cs0.y; a1 = v.y * cs0.x + v.x * cs0.y;
            c0 = v.z * cs1.x - v.w * cs1.y; c1 = v.w * cs1.x + v.z * cs1.y;
        }
        if (hd < e.nq) {
            const size_t o = ((size_t)b * e.nq + hd) * kHeadDim + i;
            bf16 *q = reinterpret_cast<bf16 *>(e.q_out);
            uint32_t hi, lo;
            split_bf16x2(a0, c0, hi, lo);
            *reinterpret_cast<uint32_t *>(q + o) = hi;
            *reinterpret_cast<uint32_t *>(q + e.q_plane + o) = lo;
            split_bf16x2(a1, c1, hi, lo);
            *reinterpret_cast<uint32_t *>(q + o + kHeadDim / 2) = hi;
            *reinterpret_cast<uint32_t *>(q + e.q_plane + o + kHeadDim / 2) = lo;
        } else {
            const bool is_k = hd < e.nq + e.nkv;
            const int kvh = is_k ? hd - e.nq : hd - e.nq - e.nkv;
            if (e.kv_new) {
                float *dst = e.kv_new + (is_k ? 0 : e.kv_new_plane) + ((size_t)b * e.nkv + kvh) * kHeadDim + i;
                *reinterpret_cast<float2 *>(dst) = make_float2(a0, c0);
                *reinterpret_cast<float2 *>(dst + kHeadDim / 2) = make_float2(a1, c1);
                return;
            }
            const size_t o = (((size_t)b * e.nkv + kvh) * e.cap + pos) * kHeadDim + i;
            bf16 *dst = reinterpret_cast<bf16 *>(is_k ? e.k_cache : e.v_cache);
            *reinterpret_cast<uint32_t *>(dst + o) = pack_bf16(a0, c0);
            *reinterpret_cast<uint32_t *>(dst + o + kHeadDim / 2) = pack_bf16(a1, c1);
        }
    }
}

}  // namespace prsv
