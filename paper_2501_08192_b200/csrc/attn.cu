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
// Persistent CTAs (one per SM) walk a static list of work items = (sequence,
// kv head, run of `tiles_per_item` tiles) in address order.  Warp 4 is the
// producer: one lane issues the TMA loads into a 4-stage ring guarded by
// full/empty mbarriers (all waits bounded).  Warps 0-3 each own 16 of a tile's
// 64 keys: S = Q K^T with mma.sync (Q rows = query heads padded to 16, from
// registers; K via ldmatrix), online softmax in fp32 with exp2, O += P V (V via
// ldmatrix.trans).  At the end of an item the four warps' (max, sum, O) are
// combined through shared memory and written as an fp32 partial; k_attn_merge
// combines the partials of a sequence in fixed order and writes bf16 output.
// Nothing depends on timing, so results are bit-stable.
#include "common.cuh"
#include "kernels.h"

namespace prsv {

constexpr int kTileKeys = 64;
constexpr int kStages = 4;
constexpr int kConsumerWarps = 4;
constexpr int kAttnThreads = (kConsumerWarps + 1) * 32;
constexpr int kHalfBytes = kTileKeys * 128;            // one 64x64 bf16 box
constexpr int kStageBytes = 4 * kHalfBytes;            // K lo, K hi, V lo, V hi
constexpr int kMaxStreams = 2048;                      // (sequence, kv head) pairs per launch

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
    float *part_o;
    float *part_ml;
    bf16 *o_out;            // hi plane; lo plane at o_out + o_plane
    size_t o_plane;
    int *status;
};

struct AttnSmem {
    alignas(1024) uint8_t stage[kStages][kStageBytes];
    float merge_o[kConsumerWarps][16][kHeadDim];
    float merge_m[kConsumerWarps][16];
    float merge_l[kConsumerWarps][16];
    uint64_t full[kStages];
    uint64_t empty[kStages];
    int item_base[kMaxStreams + 1];
};

__device__ __forceinline__ int tiles_of(int ctx) { return (ctx + 1 + kTileKeys - 1) / kTileKeys; }

// First item index of every stream, computed identically by every CTA.
__device__ __forceinline__ void build_item_table(const AttnParams &p, int *item_base)
{
    // serial prefix over at most kMaxStreams entries by one thread; tiny next to the KV stream
    if (threadIdx.x == 0) {
        int acc = 0;
        const int streams = p.B * p.nkv;
        for (int sidx = 0; sidx < streams; ++sidx) {
            item_base[sidx] = acc;
            const int nt = tiles_of(p.ctx_len[sidx / p.nkv]);
            acc += (nt + p.tiles_per_item - 1) / p.tiles_per_item;
        }
        item_base[streams] = acc;
    }
}

__device__ __forceinline__ int find_stream(const int *item_base, int streams, int item)
{
    int lo = 0, hi = streams;     // item_base[lo] <= item < item_base[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (item_base[mid] <= item) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(kAttnThreads, 1) k_attn_decode_splitkv(const __grid_constant__ AttnParams p)
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
    pdl_wait();    // q and the appended k/v come from the QKV projection
    build_item_table(p, sm.item_base);
    __syncthreads();
    const int total_items = sm.item_base[streams];

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
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
                    mbar_expect_tx(&sm.full[st], kStageBytes);
                    const int row = sidx * p.cap + tile * kTileKeys;
                    uint8_t *dst = sm.stage[st];
                    tma_load_2d(dst, &p.k_map, 0, row, &sm.full[st]);
                    tma_load_2d(dst + kHalfBytes, &p.k_map, 64, row, &sm.full[st]);
                    tma_load_2d(dst + 2 * kHalfBytes, &p.v_map, 0, row, &sm.full[st]);
                    tma_load_2d(dst + 3 * kHalfBytes, &p.v_map, 64, row, &sm.full[st]);
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
    for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
        const int sidx = find_stream(sm.item_base, streams, item);
        const int b = sidx / p.nkv, kvh = sidx % p.nkv;
        const int chunk = item - sm.item_base[sidx];
        const int n_keys = p.ctx_len[b] + 1;
        const int nt = tiles_of(p.ctx_len[b]);
        const int t0 = chunk * p.tiles_per_item;
        const int t1 = min(nt, t0 + p.tiles_per_item);

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
                qa[pl][ks][1] = g + 8 < p.G ? *reinterpret_cast<const uint32_t *>(qb + (g + 8) * kHeadDim + d0) : 0u;
                qa[pl][ks][2] = g < p.G ? *reinterpret_cast<const uint32_t *>(qb + g * kHeadDim + d0 + 8) : 0u;
                qa[pl][ks][3] = g + 8 < p.G ? *reinterpret_cast<const uint32_t *>(qb + (g + 8) * kHeadDim + d0 + 8) : 0u;
            }
        }
        float o[16][4];
#pragma unroll
        for (int i = 0; i < 16; ++i)
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
            float corr[2];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
                const float m_new = fmaxf(m_run[r], mx[r]);
                corr[r] = m_new == -INFINITY ? 1.f : exp2f(m_run[r] - m_new);
                m_run[r] = m_new;
                l_run[r] *= corr[r];
            }
            uint32_t pa[4], pb[4];      // P as hi + lo bf16 planes
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
                split_bf16x2(pv[0][0], pv[0][1], pa[0], pb[0]);
                split_bf16x2(pv[0][2], pv[0][3], pa[1], pb[1]);
                split_bf16x2(pv[1][0], pv[1][1], pa[2], pb[2]);
                split_bf16x2(pv[1][2], pv[1][3], pa[3], pb[3]);
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                o[i][0] *= corr[0]; o[i][1] *= corr[0];
                o[i][2] *= corr[1]; o[i][3] *= corr[1];
            }
            // O += P V
            {
                const int key = warp * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
                const uint32_t rowaddr = vbase + key * 128;
                const int csel = lane >> 4;
#pragma unroll
                for (int c = 0; c < 16; c += 2) {
                    const int cc = (c & 7) + csel;
                    const uint32_t addr = rowaddr + (c >> 3) * kHalfBytes + ((cc ^ (key & 7)) << 4);
                    uint32_t r[4];
                    ldmatrix_x4_trans(r, addr);
                    mma_bf16_16816(o[c], pa[0], pa[1], pa[2], pa[3], r[0], r[1]);
                    mma_bf16_16816(o[c + 1], pa[0], pa[1], pa[2], pa[3], r[2], r[3]);
                    mma_bf16_16816(o[c], pb[0], pb[1], pb[2], pb[3], r[0], r[1]);
                    mma_bf16_16816(o[c + 1], pb[0], pb[1], pb[2], pb[3], r[2], r[3]);
                }
            }
            __syncwarp();
            if (lane == 0)
                mbar_arrive(&sm.empty[st]);
        }
        // ---- combine the four warps and write the item's partial
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
            l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
        }
        if (t == 0) {
            sm.merge_m[warp][g] = m_run[0];
            sm.merge_m[warp][g + 8] = m_run[1];
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
        float scale[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = g + 8 * r;
            float M = sm.merge_m[0][row];
#pragma unroll
            for (int w = 1; w < kConsumerWarps; ++w)
                M = fmaxf(M, sm.merge_m[w][row]);
            scale[r] = m_run[r] == -INFINITY ? 0.f : exp2f(m_run[r] - M);
        }
        if (t == 0) {
            sm.merge_l[warp][g] = l_run[0] * scale[0];
            sm.merge_l[warp][g + 8] = l_run[1] * scale[1];
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            *reinterpret_cast<float2 *>(&sm.merge_o[warp][g][i * 8 + 2 * t]) =
                make_float2(o[i][0] * scale[0], o[i][1] * scale[0]);
            *reinterpret_cast<float2 *>(&sm.merge_o[warp][g + 8][i * 8 + 2 * t]) =
                make_float2(o[i][2] * scale[1], o[i][3] * scale[1]);
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
        {
            // 128 threads: thread = head dim; loop over the group's rows
            const int d = threadIdx.x;
            for (int row = 0; row < p.G; ++row) {
                float acc = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w)
                    acc += sm.merge_o[w][row][d];
                p.part_o[((size_t)item * p.G + row) * kHeadDim + d] = acc;
                if (d == 0) {
                    float M = sm.merge_m[0][row], L = 0.f;
#pragma unroll
                    for (int w = 1; w < kConsumerWarps; ++w)
                        M = fmaxf(M, sm.merge_m[w][row]);
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w)
                        L += sm.merge_l[w][row];
                    p.part_ml[((size_t)item * p.G + row) * 2] = M;
                    p.part_ml[((size_t)item * p.G + row) * 2 + 1] = L;
                }
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
    }
    pdl_launch_dependents();
}

// Merge the partials of one (sequence, query head) in item order; thread = head dim.
__global__ void __launch_bounds__(kHeadDim) k_attn_merge(const __grid_constant__ AttnParams p)
{
    const int b = blockIdx.x / p.nq, hq = blockIdx.x % p.nq;
    const int kvh = hq / p.G, row = hq % p.G;
    const int d = threadIdx.x;
    pdl_wait();
    int base = 0;
    const int sidx = b * p.nkv + kvh;
    for (int s2 = 0; s2 < sidx; ++s2) {
        const int nt = tiles_of(p.ctx_len[s2 / p.nkv]);
        base += (nt + p.tiles_per_item - 1) / p.tiles_per_item;
    }
    const int n_items = (tiles_of(p.ctx_len[b]) + p.tiles_per_item - 1) / p.tiles_per_item;
    float M = -INFINITY;
    for (int j = 0; j < n_items; ++j)
        M = fmaxf(M, p.part_ml[((size_t)(base + j) * p.G + row) * 2]);
    float L = 0.f, acc = 0.f;
    for (int j = 0; j < n_items; ++j) {
        const size_t idx = (size_t)(base + j) * p.G + row;
        const float m = p.part_ml[idx * 2];
        const float w = m == -INFINITY ? 0.f : exp2f(m - M);
        L += p.part_ml[idx * 2 + 1] * w;
        acc += p.part_o[idx * kHeadDim + d] * w;
    }
    pdl_launch_dependents();
    const float ov = acc / L;
    const bf16 hi = __float2bfloat16_rn(ov);
    const size_t oi = ((size_t)b * p.nq + hq) * kHeadDim + d;
    p.o_out[oi] = hi;
    p.o_out[p.o_plane + oi] = __float2bfloat16_rn(ov - __bfloat162float(hi));
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
    p.ctx_len = a.ctx_len;
    p.B = a.B; p.nq = a.nq; p.nkv = a.nkv; p.G = a.nq / a.nkv; p.cap = a.cap;
    p.tiles_per_item = a.tiles_per_item;
    p.max_items = a.max_items;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)kHeadDim);
    p.part_o = a.part_o;
    p.part_ml = a.part_ml;
    p.o_out = reinterpret_cast<bf16 *>(a.o_out);
    p.status = a.status;

    const size_t smem = sizeof(AttnSmem) + 1024;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_attn_decode_splitkv, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess)
            return e;
        attr_set = true;
    }
    cudaLaunchAttribute at[1];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.grid);
    cfg.blockDim = dim3(kAttnThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = at;
    cfg.numAttrs = pdl_attr(at);
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_attn_decode_splitkv, p);
    if (e != cudaSuccess)
        return e;
    cudaLaunchConfig_t cfg2 = {};
    cfg2.gridDim = dim3(a.B * a.nq);
    cfg2.blockDim = dim3(kHeadDim);
    cfg2.stream = s;
    cfg2.attrs = at;
    cfg2.numAttrs = pdl_attr(at);
    return cudaLaunchKernelEx(&cfg2, k_attn_merge, p);
}

}  // namespace prsv
