// Split-KV flash-decode attention for grouped-query heads, plus the merge of
// the per-split partial results.
//
// Decode attention multiplies one very narrow matrix (the G query heads that
// share a KV head) against the whole cached K and V of a sequence (Section 2,
// "LLM decoding is memory BW-limited"), so the kernel is a KV stream.  The
// cache is [sequence, kv head, slot, d] with d = 128 contiguous, so each
// (sequence, kv head) is one contiguous run and a tile of 64 keys is two TMA
// boxes of 64 x 64 bf16 (128-byte swizzle) per tensor.
//
// Persistent CTAs walk a static list of work items = (sequence, kv head, run of
// `tiles_per_item` tiles) in address order.  A short cache is cut into items of at most
// one ring fill, one per CTA, so every tile is in shared memory before the queries exist;
// otherwise one CTA per SM while the cache is a few ring fills (the kernels before and
// after can then be co-resident), two per SM for long caches (plan_attention).  Warp 4 is the producer: one lane issues the TMA loads into a
// 3-stage ring guarded by full/empty mbarriers (all waits bounded).  Warps 0-3 each
// own 16 of a tile's 64 keys: S = Q K^T with mma.sync (Q rows = query heads padded
// to 16, from registers; K via ldmatrix), online softmax in fp32 with exp2,
// O += P V (V via ldmatrix.trans).  At the end of an item the four warps combine
// their (max, sum, O) through the ring stage they consumed last and the CTA writes
// ONE fp32 partial per item (or the final o when the item is the whole sequence).
// k_attn_merge then combines the partials of a sequence in fixed order.  Nothing
// depends on timing, so results are bit-stable.
#include <cstdlib>

#include "../../include/preserve.h"
#include <cuda_fp16.h>

#include "attn_common.cuh"
#include "common.cuh"
#include "kernels.h"

namespace prsv {

constexpr int kStages = 3;                            // 96 KiB ring: two CTAs per SM
constexpr int kHalfBytes = kTileKeys * 128;            // one 64x64 bf16 box
constexpr int kStageBytes = 4 * kHalfBytes;            // K lo, K hi, V lo, V hi

struct AttnParams {
    CUtensorMap k_map;
    CUtensorMap v_map;
    const bf16 *q;          // hi plane; lo plane at q + q_plane (q = hi + lo)
    size_t q_plane;
    const int *ctx_len;
    int B, nq, nkv, G, cap;
    int tiles_per_item;
    int max_items;
    float scale_log2;       // log2(e) / sqrt(d)
    float *part_o;          // [item][G][d] CTA partials (unnormalised, relative to the item's max)
    float *part_ml;         // [item][G][2] (max, sum)
    bf16 *o_out;            // hi plane; lo plane at o_out + o_plane
    size_t o_plane;
    int o_fp16;             // o_out is ONE fp16 plane instead (an attention output is bounded by the largest value)
    int *status;
    long long *trace;
    int inject;             // test hook: the producer of CTA 0 never fetches one box of its first tile
};

struct AttnSmem {
    alignas(1024) uint8_t stage[kStages][kStageBytes];
    uint64_t full[kStages];
    uint64_t empty[kStages];
    float comb_ml[kConsumerWarps][16][2];
    int item_base[kMaxStreams + 1];      // last: the launch only asks for the entries it needs
};

// Where consumer warp w keeps row r (a query head of the group) of its O partial inside a ring
// stage: in the 16 key rows of each 64x64 box that only this warp reads, so no other warp can
// still be reading the bytes it overwrites.  512 B per row, four rows per box slice.
__device__ __forceinline__ float *comb_row(uint8_t *stage, int w, int r)
{
    return reinterpret_cast<float *>(stage + (r >> 2) * kHalfBytes + w * 2048 + (r & 3) * 512);
}
// float2 slot of head dims (2c, 2c + 1) within a row: XOR swizzle so that the fragment stores
// (eight rows x four column pairs per instruction) and the row reads are both conflict-free
__device__ __forceinline__ int comb_col2(int r, int c) { return c ^ ((r & 3) << 2); }

// NARROW: groups of up to 8 query heads (keys as MMA rows in the QK product), else up to 16.
template <bool NARROW>
__global__ void __launch_bounds__(kAttnThreads, 2) k_attn_decode_splitkv(const __grid_constant__ AttnParams p)
{
    extern __shared__ uint8_t smem_raw[];
    AttnSmem &sm = *reinterpret_cast<AttnSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int streams = p.B * p.nkv;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
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
    // The partial buffers hold max_items entries, sized from the host copy of the lengths.  Device
    // lengths that disagree with it must not write past them: the surplus items are dropped (the
    // result is then wrong, and the status word says why).
    int total_items = sm.item_base[streams];
    if (total_items > p.max_items) {
        total_items = p.max_items;
        if (threadIdx.x == 0)
            atomicCAS(p.status, ST_OK, ST_ITEMS_OVERFLOW);
    }

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            // Cached keys and values are read-only during the step, so their tiles are fetched
            // right away, even while the QKV projection is still running; only a sequence's last
            // tile (it holds the entry appended by that projection) has to wait for it.
            const uint64_t pol = policy_evict_first();   // each cached byte is read once per step
            uint32_t it = 0;
            bool ok = true, waited = false;
            for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
                const int sidx = find_stream(sm.item_base, streams, item);
                const int chunk = item - sm.item_base[sidx];
                const int nt = tiles_of(p.ctx_len[sidx / p.nkv]);
                const int t0 = chunk * p.tiles_per_item;
                const int t1 = min(nt, t0 + p.tiles_per_item);
                for (int tile = t0; tile < t1; ++tile, ++it) {
                    const int st = it % kStages;
                    const uint32_t ph = (it / kStages) & 1;
                    if (!mbar_wait(&sm.empty[st], ph ^ 1, p.status, ST_TIMEOUT_EMPTY)) { ok = false; break; }
                    if (tile == nt - 1 && !waited) {
                        pdl_wait();
                        waited = true;
                    }
                    mbar_expect_tx(&sm.full[st], kStageBytes);
                    const int row = sidx * p.cap + tile * kTileKeys;
                    uint8_t *dst = sm.stage[st];
                    if (!(p.inject == INJECT_ATTN_RING && it == 0 && blockIdx.x == 0))
                        tma_load_2d_hint(dst, &p.k_map, 0, row, &sm.full[st], pol);
                    tma_load_2d_hint(dst + kHalfBytes, &p.k_map, 64, row, &sm.full[st], pol);
                    tma_load_2d_hint(dst + 2 * kHalfBytes, &p.v_map, 0, row, &sm.full[st], pol);
                    tma_load_2d_hint(dst + 3 * kHalfBytes, &p.v_map, 64, row, &sm.full[st], pol);
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
    pdl_wait();    // q comes from the QKV projection
    trace_waited(p.trace);
    for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
        const int sidx = find_stream(sm.item_base, streams, item);
        const int b = sidx / p.nkv, kvh = sidx % p.nkv;
        const int chunk = item - sm.item_base[sidx];
        const int n_keys = p.ctx_len[b] + 1;
        const int nt = tiles_of(p.ctx_len[b]);
        const int t0 = chunk * p.tiles_per_item;
        const int t1 = min(nt, t0 + p.tiles_per_item);

        constexpr bool narrow = NARROW;
        // Q fragments: rows = query heads of the group (zero beyond G)
        // (both bf16 planes of q: the scores are (q_hi + q_lo) . k)
        uint32_t qa[2][8][4];
#pragma unroll
        for (int pl = 0; pl < 2; ++pl) {
            const bf16 *qb = p.q + pl * p.q_plane + ((size_t)b * p.nq + (size_t)kvh * p.G) * kHeadDim;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const int d0 = ks * 16 + 2 * t;
                qa[pl][ks][0] = g < p.G ? *reinterpret_cast<const uint32_t *>(qb + g * kHeadDim + d0) : 0u;
                qa[pl][ks][1] = (!narrow && g + 8 < p.G) ? *reinterpret_cast<const uint32_t *>(qb + (g + 8) * kHeadDim + d0) : 0u;
                qa[pl][ks][2] = g < p.G ? *reinterpret_cast<const uint32_t *>(qb + g * kHeadDim + d0 + 8) : 0u;
                qa[pl][ks][3] = (!narrow && g + 8 < p.G) ? *reinterpret_cast<const uint32_t *>(qb + (g + 8) * kHeadDim + d0 + 8) : 0u;
            }
        }
        // accumulators: O (heads x d) as 16 n-tiles of 8 head dims, or, for narrow groups, O^T (d x heads)
        // as 8 m-tiles of 16 head dims (lane (g, t): dims 16 i + g and 16 i + g + 8, heads 2t and 2t + 1)
        constexpr int kOT = narrow ? 8 : 16;
        float o[kOT][4];
#pragma unroll
        for (int i = 0; i < kOT; ++i)
            o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        float m_run[2] = {-INFINITY, -INFINITY};
        float l_run[2] = {0.f, 0.f};

        for (int tile = t0; ok && tile < t1; ++tile, ++it) {
            const int st = it % kStages;
            const uint32_t ph = (it / kStages) & 1;
            if (!mbar_wait(&sm.full[st], ph, p.status, ST_TIMEOUT_FULL)) { ok = false; break; }
            const uint32_t kbase = smem_u32(sm.stage[st]);
            const uint32_t vbase = kbase + 2 * kHalfBytes;
            const int key_w = tile * kTileKeys + warp * 16;          // first key of this warp
            const int valid = n_keys - key_w;                        // keys of this warp that exist

            if (valid < 16) {
                // last tile of the sequence: rows past the length may hold anything (even NaN);
                // zero this warp's dead V rows so that 0 * V stays 0
                const int first_dead = valid > 0 ? valid : 0;
                for (int i = lane; i < (16 - first_dead) * 16; i += 32) {
                    const int r = warp * 16 + first_dead + (i >> 4), c = i & 15;
                    uint8_t *dst = sm.stage[st] + 2 * kHalfBytes + (c >> 3) * kHalfBytes + r * 128 +
                                   (((c & 7) ^ (r & 7)) << 4);
                    *reinterpret_cast<uint4 *>(dst) = make_uint4(0, 0, 0, 0);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
            }

            float corr[2];
            uint32_t pa[4];
            if constexpr (narrow) {
                // ---- up to 8 query heads: S^T = K Q^T, keys as the 16 MMA rows, heads as the 8 columns -
                // half the MMAs of the other orientation.  Lane (g, t) holds keys g and g + 8 for the
                // heads 2t and 2t + 1.
                float sT[4] = {0.f, 0.f, 0.f, 0.f};
                {
                    const int key = warp * 16 + ((lane >> 4) << 3) + (lane & 7);
                    const uint32_t rowaddr = kbase + key * 128;
                    const int csel = (lane >> 3) & 1;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const int chunk16 = ((ks & 3) << 1) + csel;
                        const uint32_t addr = rowaddr + (ks >> 2) * kHalfBytes + ((chunk16 ^ (key & 7)) << 4);
                        uint32_t r[4];
                        ldmatrix_x4(r, addr);        // [keys 0-7 | 8-15] x [d 0-7 | 8-15] of this 16 x 16 block
#pragma unroll
                        for (int pl = 0; pl < 2; ++pl)
                            mma_bf16_16816(sT, r[0], r[2], r[1], r[3], qa[pl][ks][0], qa[pl][ks][2]);
                    }
                }
                // scale, mask, online softmax per head (a column: its 16 keys sit in the lanes of equal t)
                float v[4], mx[2];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    v[j] = (g + 8 * (j >> 1)) < valid ? sT[j] * p.scale_log2 : -INFINITY;
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    mx[j] = fmaxf(v[j], v[2 + j]);
                    mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], 4));
                    mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], 8));
                    mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], 16));
                    const float m_new = fmaxf(m_run[j], mx[j]);
                    corr[j] = m_new == -INFINITY ? 1.f : exp2f(m_run[j] - m_new);
                    m_run[j] = m_new;                       // (narrow: m_run / l_run belong to heads 2t, 2t + 1;
                    l_run[j] *= corr[j];                    //  l_run is this lane's share, summed at the end)
                }
                float ph[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float m = m_run[j & 1];
                    ph[j] = m == -INFINITY ? 0.f : exp2f(v[j] - m);
                    l_run[j & 1] += ph[j];
                }
                // P^T (keys x heads) -> (heads x keys), the B fragment of P^T in O^T = V^T P^T: two 8 x 8 transposes
                const uint32_t x0 = pack_bf16(ph[0], ph[1]), x1 = pack_bf16(ph[2], ph[3]);
                asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pa[0]) : "r"(x0));
                asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pa[2]) : "r"(x1));
                pa[1] = pa[3] = 0u;
            } else {
            // S = Q K^T for this warp's 16 keys
            float s[2][4];
#pragma unroll
            for (int i = 0; i < 2; ++i)
                s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
            {
                const int key = warp * 16 + ((lane >> 4) << 3) + (lane & 7);
                const uint32_t rowaddr = kbase + key * 128;
                const int csel = (lane >> 3) & 1;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const int chunk16 = ((ks & 3) << 1) + csel;
                    const uint32_t addr = rowaddr + (ks >> 2) * kHalfBytes + ((chunk16 ^ (key & 7)) << 4);
                    uint32_t r[4];
                    ldmatrix_x4(r, addr);
#pragma unroll
                    for (int pl = 0; pl < 2; ++pl) {
                        mma_bf16_16816(s[0], qa[pl][ks][0], qa[pl][ks][1], qa[pl][ks][2], qa[pl][ks][3], r[0], r[1]);
                        mma_bf16_16816(s[1], qa[pl][ks][0], qa[pl][ks][1], qa[pl][ks][2], qa[pl][ks][3], r[2], r[3]);
                    }
                }
            }
            // scale, mask, online softmax (rows g and g + 8)
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int kk = i * 8 + 2 * t + (j & 1);
                    const float v = kk < valid ? s[i][j] * p.scale_log2 : -INFINITY;
                    s[i][j] = v;
                    mx[j >> 1] = fmaxf(mx[j >> 1], v);
                }
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
                const float m_new = fmaxf(m_run[r], mx[r]);
                corr[r] = m_new == -INFINITY ? 1.f : exp2f(m_run[r] - m_new);
                m_run[r] = m_new;
                l_run[r] *= corr[r];
            }
            // P as one bf16 plane: the weights lie in [0, 1] and enter a sum of products with V, so
            // their 2^-9 relative rounding stays within a quarter of the tolerance on o (measured on
            // all five configs); q, whose rounding is amplified by the softmax, keeps both planes
            {
                float pv[2][4];
#pragma unroll
                for (int i = 0; i < 2; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float m = m_run[j >> 1];
                        pv[i][j] = m == -INFINITY ? 0.f : exp2f(s[i][j] - m);
                        l_run[j >> 1] += pv[i][j];
                    }
                pa[0] = pack_bf16(pv[0][0], pv[0][1]);
                pa[1] = pack_bf16(pv[0][2], pv[0][3]);
                pa[2] = pack_bf16(pv[1][0], pv[1][1]);
                pa[3] = pack_bf16(pv[1][2], pv[1][3]);
            }
            }
#pragma unroll
            for (int i = 0; i < kOT; ++i) {
                if constexpr (narrow) {          // columns = heads 2t, 2t + 1
                    o[i][0] *= corr[0]; o[i][1] *= corr[1];
                    o[i][2] *= corr[0]; o[i][3] *= corr[1];
                } else {                         // rows = heads g, g + 8
                    o[i][0] *= corr[0]; o[i][1] *= corr[0];
                    o[i][2] *= corr[1]; o[i][3] *= corr[1];
                }
            }
            // O += P V  (narrow: O^T += V^T P^T, the 16 head dims of a tile as MMA rows)
            {
                const int key = warp * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
                const uint32_t rowaddr = vbase + key * 128;
                const int csel = lane >> 4;
#pragma unroll
                for (int c = 0; c < 16; c += 2) {
                    const int cc = (c & 7) + csel;
                    const uint32_t addr = rowaddr + (c >> 3) * kHalfBytes + ((cc ^ (key & 7)) << 4);
                    uint32_t r[4];     // transposed 8 x 8 blocks [keys 0-7 | 8-15] x [dims 0-7 | 8-15] of 16 head dims
                    ldmatrix_x4_trans(r, addr);
                    if constexpr (narrow) {
                        mma_bf16_16816(o[c >> 1], r[0], r[2], r[1], r[3], pa[0], pa[2]);
                    } else {
                        mma_bf16_16816(o[c], pa[0], pa[1], pa[2], pa[3], r[0], r[1]);
                        mma_bf16_16816(o[c + 1], pa[0], pa[1], pa[2], pa[3], r[2], r[3]);
                    }
                }
            }
            __syncwarp();
            if (tile + 1 < t1 && lane == 0)
                mbar_arrive(&sm.empty[st]);      // the item's last stage is kept for the combine below
        }
        trace_streamed(p.trace, threadIdx.x == 0);

        // ---- combine the four warps' partials through the stage consumed last
        uint8_t *stage_last = sm.stage[(it + kStages - 1) % kStages];
        if constexpr (narrow) {
            // (max, sum) of heads 2t and 2t + 1: add the lanes' shares of the sum, lanes g == 0 write
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 4);
                l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 8);
                l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 16);
                if (g == 0 && 2 * t + j < p.G) {
                    sm.comb_ml[warp][2 * t + j][0] = m_run[j];
                    sm.comb_ml[warp][2 * t + j][1] = l_run[j];
                }
            }
        } else {
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
                l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
                if (t == 0 && g + 8 * r < p.G) {
                    sm.comb_ml[warp][g + 8 * r][0] = m_run[r];
                    sm.comb_ml[warp][g + 8 * r][1] = l_run[r];
                }
            }
        }
        if constexpr (narrow) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int row = 2 * t + j;              // head
                if (row < p.G) {
                    float *dst = comb_row(stage_last, warp, row);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int d0 = 16 * i + g, d1 = d0 + 8;
                        dst[2 * comb_col2(row, d0 >> 1) + (d0 & 1)] = o[i][j];
                        dst[2 * comb_col2(row, d1 >> 1) + (d1 & 1)] = o[i][2 + j];
                    }
                }
            }
        } else {
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int row = g + 8 * r;
                if (row < p.G) {
                    float2 *dst = reinterpret_cast<float2 *>(comb_row(stage_last, warp, row));
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        dst[comb_col2(row, i * 4 + t)] = make_float2(o[i][2 * r], o[i][2 * r + 1]);
                }
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
                const float2 v = reinterpret_cast<const float2 *>(comb_row(stage_last, w, r))[comb_col2(r, d2)];
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
        consumer_barrier();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0)
            mbar_arrive(&sm.empty[(it + kStages - 1) % kStages]);
    }
    trace_end(p.trace);
}

// Merge the item partials of one (sequence, query head).  One warp per partial (each lane four
// head dims, a single 16-byte load in flight per thread: a read spread over many warps returns in
// one L2 round trip, the same bytes requested by few warps take several times longer), then the
// warps' results are added in warp order, so the result does not depend on scheduling.
constexpr int kMergeMaxWarps = 32;
__global__ void __launch_bounds__(kMergeMaxWarps * 32) k_attn_merge(const __grid_constant__ AttnParams p)
{
    __shared__ int cnt_s[kMergeMaxWarps];
    __shared__ float m_s[kMergeMaxWarps], l_s[kMergeMaxWarps];
    __shared__ float acc_s[kMergeMaxWarps][kHeadDim];
    const int b = blockIdx.x / p.nq, hq = blockIdx.x % p.nq;
    const int kvh = hq / p.G, row = hq % p.G;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_warps = blockDim.x >> 5;
    const int sidx = b * p.nkv + kvh;
    long long *tr = p.trace ? p.trace + kTraceSlots : nullptr;
    trace_start(tr);
    pdl_launch_dependents();
    // first item of this stream: parallel count over the streams before it (lengths are inputs)
    int cnt = 0;
    for (int s2 = tid; s2 < sidx; s2 += blockDim.x) {
        const int nt = tiles_of(p.ctx_len[s2 / p.nkv]);
        cnt += (nt + p.tiles_per_item - 1) / p.tiles_per_item;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (lane == 0)
        cnt_s[warp] = cnt;
    const int n_items = (tiles_of(p.ctx_len[b]) + p.tiles_per_item - 1) / p.tiles_per_item;
    __syncthreads();
    int base = 0;
    for (int i = 0; i < n_warps; ++i)
        base += cnt_s[i];
    pdl_wait();    // the partials come from the split-KV kernel (every CTA waits, also those with nothing to do)
    trace_waited(tr);
    if (n_items > 1) {          // a single item was finished by the split-KV kernel itself
        float Mg = -INFINITY, L = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int e = warp; e < n_items && base + e < p.max_items; e += n_warps) {
            const size_t ent = (size_t)(base + e) * p.G + row;
            const float2 ml = *reinterpret_cast<const float2 *>(p.part_ml + ent * 2);
            const float4 ov = *(reinterpret_cast<const float4 *>(p.part_o + ent * kHeadDim) + lane);
            const float mb = fmaxf(Mg, ml.x);
            const float c = mb == -INFINITY ? 1.f : exp2f(Mg - mb);
            const float w = ml.x == -INFINITY ? 0.f : exp2f(ml.x - mb);
            L = L * c + ml.y * w;
            acc.x = acc.x * c + ov.x * w; acc.y = acc.y * c + ov.y * w;
            acc.z = acc.z * c + ov.z * w; acc.w = acc.w * c + ov.w * w;
            Mg = mb;
        }
        if (lane == 0)
            m_s[warp] = Mg;
        __syncthreads();
        // every warp rescales its own result to the common maximum (so the final sum is plain adds)
        float M = lane < n_warps ? m_s[lane] : -INFINITY;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
            M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        const float cw = Mg == -INFINITY ? 0.f : exp2f(Mg - M);
        *reinterpret_cast<float4 *>(&acc_s[warp][4 * lane]) = make_float4(acc.x * cw, acc.y * cw, acc.z * cw, acc.w * cw);
        if (lane == 0)
            l_s[warp] = L * cw;
        __syncthreads();
        if (tid < kHeadDim) {
            float a = 0.f, l = 0.f;
            for (int w = 0; w < n_warps; ++w) {          // warp order
                a += acc_s[w][tid];
                l += l_s[w];
            }
            const float ov = a / l;
            const size_t oi = ((size_t)b * p.nq + hq) * kHeadDim + tid;
            if (p.o_fp16) {
                reinterpret_cast<__half *>(p.o_out)[oi] = __float2half_rn(ov);
            } else {
                const bf16 hi = __float2bfloat16_rn(ov);
                p.o_out[oi] = hi;
                p.o_out[p.o_plane + oi] = __float2bfloat16_rn(ov - __bfloat162float(hi));
            }
        }
    }
    trace_end(tr);
}

static size_t attn_smem_bytes(int streams)
{
    return offsetof(AttnSmem, item_base) + sizeof(int) * (size_t)(streams + 1) + 1024;
}

void plan_attention(const int32_t *ctx_len_host, int batch, int nkv, int sm_count, int *grid, int *tiles_per_item,
                    int stages, double item_cost)
{
    uint64_t total_tiles = 0;
    int longest = 1;
    for (int b = 0; b < batch; ++b) {
        const int nt = (ctx_len_host[b] + 1 + kTileKeys - 1) / kTileKeys;
        total_tiles += (uint64_t)nkv * nt;
        longest = nt > longest ? nt : longest;
    }
    // A short cache fits the CTAs' rings whole: items of at most kStages tiles, one per CTA, are then
    // all in shared memory before the queries exist, and what remains after the wait is arithmetic.
    // The shortest such items that leave a (sequence, head) at most one partial per merge warp.
    for (int tpi = 1; tpi <= stages; ++tpi) {
        uint64_t items = 0;
        int per_stream = 0;
        for (int b = 0; b < batch; ++b) {
            const int nt = (ctx_len_host[b] + 1 + kTileKeys - 1) / kTileKeys;
            const int n = (nt + tpi - 1) / tpi;
            items += (uint64_t)nkv * n;
            per_stream = n > per_stream ? n : per_stream;
        }
        if (items <= (uint64_t)2 * sm_count && per_stream <= 32) {
            *grid = items <= (uint64_t)sm_count ? sm_count : 2 * sm_count;
            *tiles_per_item = tpi;
            return;
        }
    }
    // One CTA per SM while the whole cache is at most two ring fills per SM: the ring then holds
    // most of the CTA's share before the queries exist, and half of every SM's shared memory stays
    // free for the kernels before and after.  Longer caches are a steady stream: two CTAs per SM
    // keep twice the bytes in flight.
    const int g = total_tiles <= (uint64_t)2 * stages * sm_count ? sm_count : 2 * sm_count;
    // Work items = runs of `tpi` 64-key tiles of one sequence, dealt to the CTAs round-robin.  The
    // kernel lasts about rounds x (tpi + the per-item cost of combining and writing a partial,
    // worth ~1.5 tiles), rounds = items / CTAs rounded up: take the tpi that minimises that, between
    // a quarter of an even share (at most four items per CTA) and a whole share.
    const int tpi_hi = (int)((total_tiles + g - 1) / g) + 1;
    int tpi_lo = (int)((total_tiles + 4ull * g - 1) / (4ull * g));
    tpi_lo = tpi_lo < 1 ? 1 : tpi_lo;
    int best = tpi_lo;
    double best_cost = -1.0;
    for (int tpi = tpi_lo; tpi <= tpi_hi && tpi <= longest + 1; ++tpi) {
        uint64_t items = 0;
        for (int b = 0; b < batch; ++b) {
            const int nt = (ctx_len_host[b] + 1 + kTileKeys - 1) / kTileKeys;
            items += (uint64_t)nkv * ((nt + tpi - 1) / tpi);
        }
        const uint64_t rounds = (items + g - 1) / g;
        const double cost = (double)rounds * (tpi + item_cost);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best = tpi;
        }
    }
    *grid = g;
    *tiles_per_item = best;
}

cudaError_t launch_attention(const AttnArgs &a, cudaStream_t s)
{
    if (a.B * a.nkv > kMaxStreams || a.nq % a.nkv || a.nq / a.nkv > 16)
        return cudaErrorInvalidValue;
    AttnParams p;
    p.k_map = a.k_map;
    p.v_map = a.v_map;
    p.q = reinterpret_cast<const bf16 *>(a.q);
    p.q_plane = a.q_plane;
    p.o_plane = a.o_plane;
    p.o_fp16 = a.o_fp16;
    p.ctx_len = a.ctx_len;
    p.B = a.B; p.nq = a.nq; p.nkv = a.nkv; p.G = a.nq / a.nkv; p.cap = a.cap;
    p.tiles_per_item = a.tiles_per_item;
    p.max_items = a.max_items;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)kHeadDim);
    p.part_o = a.part_o;
    p.part_ml = a.part_ml;
    p.o_out = reinterpret_cast<bf16 *>(a.o_out);
    p.status = a.status;
    p.trace = a.trace;
    p.inject = a.inject;

    const size_t smem = attn_smem_bytes(a.B * a.nkv);
    if (!a.kv8) {
        static PerDeviceSize lim_narrow, lim_wide;      // per device: the attribute belongs to one device
        cudaError_t e = ensure_dynamic_smem(k_attn_decode_splitkv<true>, lim_narrow, attn_smem_bytes(kMaxStreams));
        if (e == cudaSuccess)
            e = ensure_dynamic_smem(k_attn_decode_splitkv<false>, lim_wide, attn_smem_bytes(kMaxStreams));
        if (e != cudaSuccess)
            return e;
    }
    cudaLaunchAttribute at[1];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.grid);
    cfg.blockDim = dim3(kAttnThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = at;
    cfg.numAttrs = pdl_attr(at, a.pdl);
    const int phases = a.phases ? a.phases : 3;
    cudaError_t e = cudaSuccess;
    if ((phases & 1) && a.kv8)
        e = launch_attention_kv8_kernel(a, cfg);
    else if (phases & 1)
        e = p.G <= 8 ? cudaLaunchKernelEx(&cfg, k_attn_decode_splitkv<true>, p)
                     : cudaLaunchKernelEx(&cfg, k_attn_decode_splitkv<false>, p);
    if (e != cudaSuccess)
        return e;
    if (a.mid_event) {
        e = cudaEventRecord(a.mid_event, s);
        if (e != cudaSuccess)
            return e;
    }
    if (!(phases & 2))
        return cudaSuccess;
    // one warp per item partial of the longest sequence (at least the four that write the head dims)
    int warps = a.max_items_per_stream < 4 ? 4 : (a.max_items_per_stream > kMergeMaxWarps ? kMergeMaxWarps
                                                                                          : a.max_items_per_stream);
    // Many merge CTAs (batch x heads >= 512: seven per SM) with eight warps each fill an SM's thread slots,
    // and the output projection's CTAs - launched early, to stage their weights during the merge - find no
    // room: four warps then (a warp takes two partials in turn; config 4: merge +0.9 us, O projection -1.1 us
    // with its hand-over, layer -0.5 us).
    if (a.B * a.nq >= 512 && warps > 4)
        warps = 4;
    cudaLaunchConfig_t cfg2 = {};
    cfg2.gridDim = dim3(a.B * a.nq);
    cfg2.blockDim = dim3(warps * 32);
    cfg2.stream = s;
    cfg2.attrs = at;
    cfg2.numAttrs = pdl_attr(at, a.pdl);
    return cudaLaunchKernelEx(&cfg2, k_attn_merge, p);
}

}  // namespace prsv

// ---------------------------------------------------------------------------------------
// Allocation-free decode attention.  Some callers cannot allocate device memory when they
// need attention (see the declaration in preserve.h), so the split-KV partials of this
// variant live in an array that is part of the library image instead of a cudaMalloc'd
// workspace.  In host code the array's name is only a handle for the runtime - not a device
// address - so the address is looked up once per device with cudaGetSymbolAddress and that
// pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[PRESERVE_STATIC_SCRATCH_BYTES];

namespace {
void *g_scratch_addr[prsv::kMaxDevices];      // per device, filled by the first call on that device
int g_scratch_sms[prsv::kMaxDevices];
}  // namespace

extern "C" int preserve_attention_static(const void *q_hi, const void *q_lo, const void *k_cache,
                                         const void *v_cache, const int32_t *ctx_len,
                                         const int32_t *ctx_len_host, int32_t batch, int32_t n_q_heads,
                                         int32_t n_kv_heads, int32_t kv_capacity, void *o_hi, void *o_lo,
                                         void *cuda_stream)
{
    using namespace prsv;
    if (!q_hi || !q_lo || !k_cache || !v_cache || !ctx_len || !ctx_len_host || !o_hi || !o_lo)
        return PRESERVE_EINVAL;
    const void *ptrs[] = {q_hi, q_lo, k_cache, v_cache, o_hi, o_lo};
    for (const void *p : ptrs)
        if (reinterpret_cast<uintptr_t>(p) & 15)
            return PRESERVE_EALIGN;
    if (batch < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads || n_q_heads / n_kv_heads > 16 ||
        kv_capacity < 1 || (long long)batch * n_kv_heads > kMaxStreams ||
        (long long)batch * n_kv_heads * kv_capacity > 0x7fffffffll)
        return PRESERVE_ESHAPE;
    uint64_t total_tiles = 0;
    for (int b = 0; b < batch; ++b) {
        if (ctx_len_host[b] < 0 || ctx_len_host[b] >= kv_capacity)
            return PRESERVE_ESHAPE;
        total_tiles += (uint64_t)n_kv_heads * ((uint64_t)(ctx_len_host[b] + 1 + kTileKeys - 1) / kTileKeys);
    }

    // ---- once per device: the array's device address (with that device current)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return PRESERVE_EARCH;
    }
    if (!g_scratch_addr[dev]) {
        void *addr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&addr, g_static_scratch);
        if (e != cudaSuccess || !addr) {
            (void)cudaGetLastError();
            return PRESERVE_ECUDA;
        }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
            (void)cudaGetLastError();
            return PRESERVE_ECUDA;
        }
        g_scratch_sms[dev] = sms;
        g_scratch_addr[dev] = addr;
    }

    // ---- carve the array: [status word, 256 B][partial O][partial (max, sum)]
    const int G = n_q_heads / n_kv_heads;
    int grid = 0, tpi = 1;
    plan_attention(ctx_len_host, batch, n_kv_heads, g_scratch_sms[dev], &grid, &tpi);
    uint64_t n_items = 0, max_items_seq = 0;
    for (int b = 0; b < batch; ++b) {
        const uint64_t nt = (uint64_t)(ctx_len_host[b] + 1 + kTileKeys - 1) / kTileKeys;
        const uint64_t ni = (nt + tpi - 1) / tpi;
        n_items += (uint64_t)n_kv_heads * ni;
        max_items_seq = ni > max_items_seq ? ni : max_items_seq;
    }
    const uint64_t o_bytes = n_items * G * kHeadDim * sizeof(float);
    const uint64_t ml_bytes = n_items * G * 2 * sizeof(float);
    if (256 + o_bytes + ml_bytes > PRESERVE_STATIC_SCRATCH_BYTES)
        return PRESERVE_ETOOBIG;
    unsigned char *base = static_cast<unsigned char *>(g_scratch_addr[dev]);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);

    AttnArgs a = {};
    const uint64_t rows = (uint64_t)batch * n_kv_heads * kv_capacity;
    if (!encode_bf16_map_2d(&a.k_map, k_cache, kHeadDim, rows, 64, 64) ||
        !encode_bf16_map_2d(&a.v_map, v_cache, kHeadDim, rows, 64, 64))
        return PRESERVE_EARCH;
    // the status word is the only part of the array that must start at zero
    if (cudaMemsetAsync(base, 0, 256, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    a.q = q_hi;
    a.q_plane = (size_t)(static_cast<const bf16 *>(q_lo) - static_cast<const bf16 *>(q_hi));
    a.ctx_len = ctx_len;
    a.B = batch; a.nq = n_q_heads; a.nkv = n_kv_heads; a.cap = kv_capacity;
    a.grid = grid;
    a.tiles_per_item = tpi;
    a.max_items = (int)n_items;
    a.max_items_per_stream = (int)max_items_seq;
    a.part_o = reinterpret_cast<float *>(base + 256);
    a.part_ml = reinterpret_cast<float *>(base + 256 + o_bytes);
    a.o_out = o_hi;
    a.o_plane = (size_t)(static_cast<bf16 *>(o_lo) - static_cast<bf16 *>(o_hi));
    a.status = reinterpret_cast<int *>(base);
    a.pdl = 1;      // (the merge kernel's prologue overlaps the split-KV kernel's tail)
    if (launch_attention(a, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    return PRESERVE_OK;
}

// The device status word of the allocation-free entry point on the current device (it lives at the
// start of the static array, where no handle can reach it).  Waits for the device, allocates nothing.
extern "C" int preserve_attention_static_status(void)
{
    using namespace prsv;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return PRESERVE_EARCH;
    }
    if (!g_scratch_addr[dev])
        return PRESERVE_OK;         // no call on this device yet
    int st = 0;
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(&st, g_scratch_addr[dev], sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    return st == ST_OK ? PRESERVE_OK : (st == ST_ITEMS_OVERFLOW ? PRESERVE_ESHAPE : PRESERVE_ETIMEOUT);
}

