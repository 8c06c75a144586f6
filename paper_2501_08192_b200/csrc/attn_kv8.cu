// Split-KV flash-decode attention over an int8 KV-cache (the precision of the paper's
// measurements: Section 4, "Experimental setup"; the scaling is this build's reading: one fp32
// scale per cached vector, value = code * scale).
//
// Same structure as the bf16 kernel (persistent CTAs over (sequence, kv head, run of tiles) work
// items, one producer warp, four consumer warps of 16 keys each, fp32 partial per item, the same
// merge kernel), with these differences:
//   - a tile of 64 keys is ONE TMA box of 64 x 128 bytes per tensor plus the tile's 64 + 64
//     scales (two 256-byte bulk copies): 16.5 KiB per stage instead of 32 KiB, four stages;
//   - the codes are widened to fp16 in registers with one byte permute per pair: the byte with its
//     top bit flipped (code + 128) lands in the mantissa of 1024.0, which is the number
//     1152 + code exactly.  The products run on fp16 mma.sync with that offset left in: it adds
//     1152 * (sum of the other operand) to every result, a number the kernel also has (the sum
//     of q over the head dims, once per item; the sum of the weights over the keys, from one
//     extra MMA per tile against a row of ones) and subtracts at the end.  q and the softmax
//     weights are one fp16 plane each (11 significant bits);
//   - the key scale multiplies the score after the dot product; the value scale multiplies the
//     softmax weight before the P V product, normalised by a running power of two (the largest
//     value scale seen so far) so that the fp16 weights never leave [0, 2);
//   - ldmatrix delivers int8 pairs where the bf16 kernel gets single elements, so the head
//     dimension is visited in a permuted order on both operands of Q K^T and the output columns
//     of P V come out interleaved; both permutations are undone by index arithmetic only;
//   - the QKV projection leaves the step's new key and value as fp32 vectors in a staging
//     buffer; the warp that owns the sequence's last key quantises them (fp32 division and
//     round-to-nearest-even, as the definition says), patches its shared-memory tile and writes
//     codes and scales to the cache for the following steps;
//   - groups of at most 8 query heads per KV head (keys as MMA rows).
#include <cuda_fp16.h>

#include "../../include/preserve.h"
#include "attn_common.cuh"
#include "common.cuh"
#include "kernels.h"

namespace prsv {

constexpr int kStages8 = 4;
constexpr int kBox8 = kTileKeys * 128;                 // one 64-key box of int8 codes
constexpr int kScaleOff8 = 2 * kBox8;                  // K codes, V codes, then 64 K scales and 64 V scales
constexpr int kStage8Tx = 2 * kBox8 + 2 * kTileKeys * 4;
constexpr int kStage8Stride = 17 * 1024;               // boxes must start on 1 KiB boundaries (128-byte swizzle)
constexpr int kMaxGroup8 = 8;

struct AttnKv8Params {
    CUtensorMap k_map;      // uint8, dims (128, rows), box (128, 64), 128-byte swizzle
    CUtensorMap v_map;
    const float *k_scale;   // [streams][scale_cap]
    const float *v_scale;
    uint8_t *k_codes;       // the cache itself, for the appended entry
    uint8_t *v_codes;
    float *k_scale_w;
    float *v_scale_w;
    const float *kv_new;    // fp32 [2][streams][128]: the step's key (after the rotary embedding), then value
    size_t kv_new_plane;
    const bf16 *q;          // hi plane; lo plane at q + q_plane
    size_t q_plane;
    const int *ctx_len;
    int B, nq, nkv, G, cap, scale_cap;
    int tiles_per_item;
    int max_items;
    float scale_log2;
    float *part_o;
    float *part_ml;
    bf16 *o_out;
    size_t o_plane;
    int o_fp16;             // o_out is ONE fp16 plane instead of split bf16
    int *status;
    long long *trace;
    int inject;
};

struct AttnKv8Smem {
    alignas(1024) uint8_t stage[kStages8][kStage8Stride];
    float comb_o[kConsumerWarps][kMaxGroup8][kHeadDim];
    float comb_ml[kConsumerWarps][kMaxGroup8][2];
    uint64_t full[kStages8];
    uint64_t empty[kStages8];
    int item_base[kMaxStreams + 1];      // last: the launch only asks for the entries it needs
};

// D(16x8, f32) += A(16x16, f16, row) * B(16x8, f16, col)
__device__ __forceinline__ void mma_f16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                 "{%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Two int8 codes of `biased` (= the loaded word with every byte's top bit flipped, i.e. code + 128 as
// an unsigned byte) as an fp16 pair holding 1152 + code each.  SEL picks the bytes: 0x4140 = bytes
// (0, 1), 0x4342 = (2, 3), 0x4240 = (0, 2), 0x4341 = (1, 3).  The byte lands in the low mantissa
// bits of 1024.0 (0x6400), which is 1024 + byte = 1152 + code exactly.
constexpr float kCodeOffset = 1152.f;
template <uint32_t SEL>
__device__ __forceinline__ uint32_t s8x2_to_f16x2_offset(uint32_t biased)
{
    return __byte_perm(biased, 0x64646464u, SEL);
}

__device__ __forceinline__ float ex2_fast(float x)      // 2^x; -inf gives 0
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_f16(float lo, float hi)
{
    const __half2 t = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&t);
}

// float2 slot of head dims (2c, 2c + 1) of query head `row` in a combine row: the fragment stores
// (eight dim pairs x four heads per instruction) then take the minimum of two wavefronts, and the
// row reads are conflict-free
__device__ __forceinline__ int comb8_col2(int row, int c) { return c ^ (((row >> 1) & 1) << 3); }

// Symmetric int8 quantisation of one 128-vector held four values per lane: returns the packed codes
// of this lane's four values and the scale (the same in every lane).
__device__ __forceinline__ uint32_t quantize_row_128(float4 u, float &scale)
{
    float mx = fmaxf(fmaxf(fabsf(u.x), fabsf(u.y)), fmaxf(fabsf(u.z), fabsf(u.w)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float sc = __fdiv_rn(mx, 127.0f);
    scale = sc;
    auto code = [&](float x) -> uint32_t {
        float c = sc > 0.f ? rintf(__fdiv_rn(x, sc)) : 0.f;
        c = fminf(fmaxf(c, -127.f), 127.f);
        return (uint32_t)(int)c & 0xffu;
    };
    return code(u.x) | (code(u.y) << 8) | (code(u.z) << 16) | (code(u.w) << 24);
}

__global__ void __launch_bounds__(kAttnThreads, 2) k_attn_decode_splitkv_kv8(const __grid_constant__ AttnKv8Params p)
{
    extern __shared__ uint8_t smem_raw[];
    AttnKv8Smem &sm = *reinterpret_cast<AttnKv8Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int streams = p.B * p.nkv;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages8; ++i) {
            mbar_init(&sm.full[i], 1);
            mbar_init(&sm.empty[i], kConsumerWarps);
        }
        mbar_fence_init();
        tma_prefetch_desc(&p.k_map);
        tma_prefetch_desc(&p.v_map);
    }
    trace_start(p.trace);
    pdl_launch_dependents();
    build_item_table(p, sm.item_base);       // sequence lengths are inputs of the step: no dependency
    __syncthreads();
    int total_items = sm.item_base[streams];
    if (total_items > p.max_items) {         // device lengths disagree with the host copy: never write past the partials
        total_items = p.max_items;
        if (threadIdx.x == 0)
            atomicCAS(p.status, ST_OK, ST_ITEMS_OVERFLOW);
    }

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            // Cached entries are read-only during the step and the new entry does not come through the
            // cache at all, so nothing here depends on the projection before; only a sequence's last
            // tile waits for it, which keeps the order "every earlier kernel of the stream has
            // completed before the slot written one step ago is read".
            const uint64_t pol = policy_evict_first();
            uint32_t it = 0;
            bool ok = true, waited = false;
            for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
                const int sidx = find_stream(sm.item_base, streams, item);
                const int chunk = item - sm.item_base[sidx];
                const int nt = tiles_of(p.ctx_len[sidx / p.nkv]);
                const int t0 = chunk * p.tiles_per_item;
                const int t1 = min(nt, t0 + p.tiles_per_item);
                for (int tile = t0; tile < t1; ++tile, ++it) {
                    const int st = it % kStages8;
                    const uint32_t ph = (it / kStages8) & 1;
                    if (!mbar_wait(&sm.empty[st], ph ^ 1, p.status, ST_TIMEOUT_EMPTY)) { ok = false; break; }
                    if (tile == nt - 1 && !waited) {
                        pdl_wait();
                        waited = true;
                    }
                    mbar_expect_tx(&sm.full[st], kStage8Tx);
                    const int row = sidx * p.cap + tile * kTileKeys;
                    uint8_t *dst = sm.stage[st];
                    if (!(p.inject == INJECT_ATTN_RING && it == 0 && blockIdx.x == 0))
                        tma_load_2d_hint(dst, &p.k_map, 0, row, &sm.full[st], pol);
                    tma_load_2d_hint(dst + kBox8, &p.v_map, 0, row, &sm.full[st], pol);
                    const size_t so = (size_t)sidx * p.scale_cap + (size_t)tile * kTileKeys;
                    bulk_load_hint(dst + kScaleOff8, p.k_scale + so, kTileKeys * 4, &sm.full[st], pol);
                    bulk_load_hint(dst + kScaleOff8 + kTileKeys * 4, p.v_scale + so, kTileKeys * 4, &sm.full[st], pol);
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    // A failed wait poisons the rest of the kernel: `ok` stays false, no barrier is
    // waited on again, but every warp still reaches the named barriers below.
    const int g = lane >> 2, t = lane & 3;
    uint32_t it = 0;
    bool ok = true;
    pdl_wait();    // q and the new key / value come from the QKV projection
    trace_waited(p.trace);
    // this lane's ldmatrix row: matrices 0..3 of an x4 load = (keys 0-7 | 8-15) x (chunk c | c + 1)
    const int lkey = warp * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
    const int lsw = lkey & 7, lch = lane >> 4;
    for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
        const int sidx = find_stream(sm.item_base, streams, item);
        const int b = sidx / p.nkv, kvh = sidx % p.nkv;
        const int chunk = item - sm.item_base[sidx];
        const int n_keys = p.ctx_len[b] + 1;
        const int nt = tiles_of(p.ctx_len[b]);
        const int t0 = chunk * p.tiles_per_item;
        const int t1 = min(nt, t0 + p.tiles_per_item);

        // Q fragments (the B operand of S^T = K Q^T), query head g, as one fp16 plane.  The k index
        // of the MMA runs over the head dims in the order the int8 ldmatrix delivers them: for the
        // 16-dim chunk c, k = 2t, 2t + 1 are dims 16c + 4t, + 1 and k = 2t + 8, 2t + 9 are dims 16c + 4t + 2, + 3.
        uint32_t qa[8][2];
        float qoff[2];                       // 1152 * (sum over the head dims of q as the MMA sees it), heads 2t, 2t + 1
        {
            float qs = 0.f;
            const bf16 *qh = p.q + ((size_t)b * p.nq + (size_t)kvh * p.G + g) * kHeadDim;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint2 hi = make_uint2(0u, 0u), lo = make_uint2(0u, 0u);
                if (g < p.G) {
                    hi = *reinterpret_cast<const uint2 *>(qh + c * 16 + 4 * t);
                    lo = *reinterpret_cast<const uint2 *>(qh + p.q_plane + c * 16 + 4 * t);
                }
                const float q0 = bf_lo(hi.x) + bf_lo(lo.x), q1 = bf_hi(hi.x) + bf_hi(lo.x);
                const float q2 = bf_lo(hi.y) + bf_lo(lo.y), q3 = bf_hi(hi.y) + bf_hi(lo.y);
                const __half2 h01 = __floats2half2_rn(q0, q1), h23 = __floats2half2_rn(q2, q3);
                const float2 f01 = __half22float2(h01), f23 = __half22float2(h23);
                qa[c][0] = *reinterpret_cast<const uint32_t *>(&h01);
                qa[c][1] = *reinterpret_cast<const uint32_t *>(&h23);
                qs += (f01.x + f01.y) + (f23.x + f23.y);
            }
            qs += __shfl_xor_sync(0xffffffffu, qs, 1);       // the four lanes of a head hold 32 dims each
            qs += __shfl_xor_sync(0xffffffffu, qs, 2);
            qoff[0] = kCodeOffset * __shfl_sync(0xffffffffu, qs, 8 * t);
            qoff[1] = kCodeOffset * __shfl_sync(0xffffffffu, qs, 8 * t + 4);
        }
        // O^T accumulators: m-tile i holds head dims 16 i + 2 g (rows 0-7) and 16 i + 2 g + 1 (rows 8-15)
        // for the heads 2t and 2t + 1, in units of 2^(e_run - 127)
        float o[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        float psum[4] = {0.f, 0.f, 0.f, 0.f};   // [0], [1]: sum over the keys of the scaled weights, heads 2t and 2t + 1
        float m_run[2] = {-INFINITY, -INFINITY};
        float l_run[2] = {0.f, 0.f};
        int e_run = 0;                       // biased exponent of the largest value scale seen so far

        for (int tile = t0; ok && tile < t1; ++tile, ++it) {
            const int st = it % kStages8;
            const uint32_t ph = (it / kStages8) & 1;
            if (!mbar_wait(&sm.full[st], ph, p.status, ST_TIMEOUT_FULL)) { ok = false; break; }
            uint8_t *stage = sm.stage[st];
            float *ks_s = reinterpret_cast<float *>(stage + kScaleOff8);
            float *vs_s = ks_s + kTileKeys;
            const int key_w = tile * kTileKeys + warp * 16;          // first key of this warp
            const int valid = n_keys - key_w;                        // keys of this warp that exist

            if (valid >= 1 && valid <= 16) {
                // this warp owns the sequence's newest key: quantise the step's key and value, put
                // them into the tile and into the cache (slot ctx_len[b])
                const int kl = warp * 16 + valid - 1;
                const size_t slot = (size_t)sidx * p.cap + (size_t)(n_keys - 1);
                const uint32_t so = kl * 128 + ((((uint32_t)lane >> 2) ^ (kl & 7)) << 4) + (lane & 3) * 4;
#pragma unroll
                for (int kv = 0; kv < 2; ++kv) {
                    const float4 u = *reinterpret_cast<const float4 *>(p.kv_new + kv * p.kv_new_plane + (size_t)sidx * kHeadDim + 4 * lane);
                    float sc;
                    const uint32_t codes = quantize_row_128(u, sc);
                    *reinterpret_cast<uint32_t *>(stage + kv * kBox8 + so) = codes;
                    *reinterpret_cast<uint32_t *>((kv ? p.v_codes : p.k_codes) + slot * kHeadDim + 4 * lane) = codes;
                    if (lane == 0) {
                        (kv ? vs_s : ks_s)[kl] = sc;
                        (kv ? p.v_scale_w : p.k_scale_w)[(size_t)sidx * p.scale_cap + (size_t)(n_keys - 1)] = sc;
                    }
                }
                __syncwarp();
            }

            // ---- S^T = K Q^T: keys as the 16 MMA rows, heads as the 8 columns; lane (g, t) ends up with
            // the keys g and g + 8 for the heads 2t and 2t + 1
            float sT[4] = {0.f, 0.f, 0.f, 0.f};
            {
                const uint32_t krow = smem_u32(stage) + lkey * 128;
#pragma unroll
                for (int c = 0; c < 8; c += 2) {
                    uint32_t r[4];
                    ldmatrix_x4(r, krow + (((c + lch) ^ lsw) << 4));
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t w0 = r[2 * h] ^ 0x80808080u, w1 = r[2 * h + 1] ^ 0x80808080u;
                        const uint32_t a0 = s8x2_to_f16x2_offset<0x4140>(w0), a2 = s8x2_to_f16x2_offset<0x4342>(w0);
                        const uint32_t a1 = s8x2_to_f16x2_offset<0x4140>(w1), a3 = s8x2_to_f16x2_offset<0x4342>(w1);
                        mma_f16_16816(sT, a0, a1, a2, a3, qa[c + h][0], qa[c + h][1]);
                    }
                }
            }
            // key scales, softmax scale, mask, online softmax per head (a column: its 16 keys sit in the
            // lanes of equal t).  Dead keys are selected away, never multiplied: their scales may be NaN.
            const bool liveA = g < valid, liveB = g + 8 < valid;
            const float ksA = liveA ? ks_s[warp * 16 + g] : 0.f, ksB = liveB ? ks_s[warp * 16 + g + 8] : 0.f;
            float vsA = liveA ? vs_s[warp * 16 + g] : 0.f, vsB = liveB ? vs_s[warp * 16 + g + 8] : 0.f;
            float v[4], mx[2], corr[2];
            const float kA = ksA * p.scale_log2, kB = ksB * p.scale_log2;
            v[0] = liveA ? (sT[0] - qoff[0]) * kA : -INFINITY;
            v[1] = liveA ? (sT[1] - qoff[1]) * kA : -INFINITY;
            v[2] = liveB ? (sT[2] - qoff[0]) * kB : -INFINITY;
            v[3] = liveB ? (sT[3] - qoff[1]) * kB : -INFINITY;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                mx[j] = fmaxf(v[j], v[2 + j]);
                mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], 4));
                mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], 8));
                mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], 16));
                const float m_new = fmaxf(m_run[j], mx[j]);
                corr[j] = m_new == -INFINITY ? 1.f : ex2_fast(m_run[j] - m_new);
                m_run[j] = m_new;
                l_run[j] *= corr[j];
            }
            // the running power of two that keeps the scaled weights in [0, 2)
            {
                float vm = fmaxf(vsA, vsB);
                vm = fmaxf(vm, __shfl_xor_sync(0xffffffffu, vm, 4));
                vm = fmaxf(vm, __shfl_xor_sync(0xffffffffu, vm, 8));
                vm = fmaxf(vm, __shfl_xor_sync(0xffffffffu, vm, 16));
                int e_t = (int)((__float_as_uint(vm) >> 23) & 0xffu);
                e_t = e_t > 253 ? 253 : e_t;
                if (e_t > e_run) {
                    const float down = e_run == 0 ? 0.f : ex2_fast((float)(e_run - e_t));   // o is still zero while e_run is 0
                    corr[0] *= down;        // (l_run has been updated already: it is not rescaled)
                    corr[1] *= down;
                    e_run = e_t;
                }
                const float norm = __uint_as_float((uint32_t)(254 - e_run) << 23);       // 2^(127 - e_run)
                vsA *= norm;
                vsB *= norm;
            }
            uint32_t pa0, pa2;
            {
                float ph4[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float m = m_run[j & 1];
                    ph4[j] = m == -INFINITY ? 0.f : ex2_fast(v[j] - m);
                    l_run[j & 1] += ph4[j];
                }
                // P^T (keys x heads) -> (heads x keys), the B fragment of O^T = V^T P^T: two 8 x 8 transposes
                const uint32_t x0 = pack_f16(ph4[0] * vsA, ph4[1] * vsA), x1 = pack_f16(ph4[2] * vsB, ph4[3] * vsB);
                asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pa0) : "r"(x0));
                asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pa2) : "r"(x1));
            }
            // (once the running maximum and the running scale have settled the factors are all one)
            if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    o[i][0] *= corr[0]; o[i][1] *= corr[1];
                    o[i][2] *= corr[0]; o[i][3] *= corr[1];
                }
                psum[0] *= corr[0];
                psum[1] *= corr[1];
            }
            // the weights against a row of ones: what the code offset adds to every head dim
            mma_f16_16816(psum, 0x3c003c00u, 0x3c003c00u, 0x3c003c00u, 0x3c003c00u, pa0, pa2);
            // ---- O^T += V^T P^T: a transposed int8 ldmatrix hands lane (g, t) the keys 2t, 2t + 1 of the
            // head dims 2g, 2g + 1 of a chunk, so MMA row g is dim 2g and row g + 8 is dim 2g + 1
            {
                const uint32_t vrow = smem_u32(stage) + kBox8 + lkey * 128;
#pragma unroll
                for (int i = 0; i < 8; i += 2) {
                    uint32_t r[4];
                    ldmatrix_x4_trans(r, vrow + (((i + lch) ^ lsw) << 4));
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t w0 = r[2 * h] ^ 0x80808080u, w1 = r[2 * h + 1] ^ 0x80808080u;
                        const uint32_t a0 = s8x2_to_f16x2_offset<0x4240>(w0), a1 = s8x2_to_f16x2_offset<0x4341>(w0);
                        const uint32_t a2 = s8x2_to_f16x2_offset<0x4240>(w1), a3 = s8x2_to_f16x2_offset<0x4341>(w1);
                        mma_f16_16816(o[i + h], a0, a1, a2, a3, pa0, pa2);
                    }
                }
            }
            // the patch above wrote the tile through the generic proxy; the next TMA fill must come after it
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0)
                mbar_arrive(&sm.empty[st]);
        }
        trace_streamed(p.trace, threadIdx.x == 0);

        // ---- back to true units, then combine the four warps' partials
        {
            const float unit = __uint_as_float((uint32_t)e_run << 23);     // 2^(e_run - 127); 0 when every value scale was 0
            const float off0 = kCodeOffset * psum[0], off1 = kCodeOffset * psum[1];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                o[i][0] = (o[i][0] - off0) * unit; o[i][1] = (o[i][1] - off1) * unit;
                o[i][2] = (o[i][2] - off0) * unit; o[i][3] = (o[i][3] - off1) * unit;
            }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            // (max, sum) of heads 2t and 2t + 1: add the lanes' shares of the sum, lanes g == 0 write
            l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 4);
            l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 8);
            l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 16);
            const int row = 2 * t + j;              // head
            if (row < p.G) {
                if (g == 0) {
                    sm.comb_ml[warp][row][0] = m_run[j];
                    sm.comb_ml[warp][row][1] = l_run[j];
                }
                float2 *dst = reinterpret_cast<float2 *>(sm.comb_o[warp][row]);
#pragma unroll
                for (int i = 0; i < 8; ++i)         // head dims 16 i + 2 g and 16 i + 2 g + 1
                    dst[comb8_col2(row, 8 * i + g)] = make_float2(o[i][j], o[i][2 + j]);
            }
        }
        consumer_barrier();
        const int n_items_stream = sm.item_base[sidx + 1] - sm.item_base[sidx];
        // two head dims per consumer thread, the heads of one parity per half of the threads
        const int d2 = threadIdx.x & 63;
        for (int r = threadIdx.x >> 6; r < p.G; r += 2) {
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w)
                M = fmaxf(M, sm.comb_ml[w][r][0]);
            float2 acc = make_float2(0.f, 0.f);
            float lsum = 0.f;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) {
                const float mw = sm.comb_ml[w][r][0];
                const float c = mw == -INFINITY ? 0.f : exp2f(mw - M);
                const float2 v = reinterpret_cast<const float2 *>(sm.comb_o[w][r])[comb8_col2(r, d2)];
                acc.x += v.x * c;
                acc.y += v.y * c;
                lsum += sm.comb_ml[w][r][1] * c;
            }
            if (n_items_stream == 1) {
                // the item is the whole sequence: finish here
                const float o0 = acc.x / lsum, o1 = acc.y / lsum;
                const size_t oi = ((size_t)b * p.nq + (size_t)kvh * p.G + r) * kHeadDim + 2 * d2;
                if (p.o_fp16) {
                    *reinterpret_cast<__half2 *>(reinterpret_cast<__half *>(p.o_out) + oi) = __floats2half2_rn(o0, o1);
                } else {
                    uint32_t hi, lo;
                    split_bf16x2(o0, o1, hi, lo);
                    *reinterpret_cast<uint32_t *>(p.o_out + oi) = hi;
                    *reinterpret_cast<uint32_t *>(p.o_out + p.o_plane + oi) = lo;
                }
            } else {
                *reinterpret_cast<float2 *>(p.part_o + ((size_t)item * p.G + r) * kHeadDim + 2 * d2) = acc;
                if (d2 == 0)
                    *reinterpret_cast<float2 *>(p.part_ml + ((size_t)item * p.G + r) * 2) = make_float2(M, lsum);
            }
        }
        consumer_barrier();      // the combine rows are free for the next item
    }
    trace_end(p.trace);
}

static size_t attn_kv8_smem_bytes(int streams)
{
    return offsetof(AttnKv8Smem, item_base) + sizeof(int) * (size_t)(streams + 1) + 1024;
}

int attention_kv8_stages() { return kStages8; }

cudaError_t launch_attention_kv8_kernel(const AttnArgs &a, const cudaLaunchConfig_t &base_cfg)
{
    if (a.B * a.nkv > kMaxStreams || a.nq % a.nkv || a.nq / a.nkv > kMaxGroup8 || a.scale_cap % kTileKeys)
        return cudaErrorInvalidValue;
    AttnKv8Params p;
    p.k_map = a.k_map;
    p.v_map = a.v_map;
    p.k_scale = a.k_scale;
    p.v_scale = a.v_scale;
    p.k_codes = static_cast<uint8_t *>(a.k_codes);
    p.v_codes = static_cast<uint8_t *>(a.v_codes);
    p.k_scale_w = a.k_scale;
    p.v_scale_w = a.v_scale;
    p.kv_new = a.kv_new;
    p.kv_new_plane = a.kv_new_plane;
    p.q = reinterpret_cast<const bf16 *>(a.q);
    p.q_plane = a.q_plane;
    p.ctx_len = a.ctx_len;
    p.B = a.B; p.nq = a.nq; p.nkv = a.nkv; p.G = a.nq / a.nkv; p.cap = a.cap; p.scale_cap = a.scale_cap;
    p.tiles_per_item = a.tiles_per_item;
    p.max_items = a.max_items;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)kHeadDim);
    p.part_o = a.part_o;
    p.part_ml = a.part_ml;
    p.o_out = reinterpret_cast<bf16 *>(a.o_out);
    p.o_plane = a.o_plane;
    p.o_fp16 = a.o_fp16;
    p.status = a.status;
    p.trace = a.trace;
    p.inject = a.inject;
    static PerDeviceSize lim;      // per device: the attribute belongs to one device
    cudaError_t e = ensure_dynamic_smem(k_attn_decode_splitkv_kv8, lim, attn_kv8_smem_bytes(kMaxStreams));
    if (e != cudaSuccess)
        return e;
    cudaLaunchConfig_t cfg = base_cfg;
    cfg.dynamicSmemBytes = attn_kv8_smem_bytes(a.B * a.nkv);
    return cudaLaunchKernelEx(&cfg, k_attn_decode_splitkv_kv8, p);
}

}  // namespace prsv
