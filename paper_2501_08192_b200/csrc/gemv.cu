// Split-K GEMV for decode batches below 16: y[b,n] = sum_k x[b,k] * W[n,k].
//
// The projection layers of the decode phase reuse each weight only `batch`
// times (Section 2, "LLM decoding is memory BW-limited"), so the kernel is a
// pure weight stream.  The packed weights are 1 KiB fragment-major tiles (16
// output rows x 32 k, see pack.cu), contiguous along k within a 16-row block.
//
// CTAs of 8 warps.  A CTA (or a cluster of up to 8 CTAs) owns one group of
// 16-row blocks at a time (further groups are loop iterations); the k range is
// split over the warps of the CTA and the CTAs of the cluster, so every warp
// streams ONE contiguous run of tiles per row block - for one or (RB = 2) two row
// blocks, which then share every activation fragment the warp loads.  Each warp is
// its own producer and consumer: lane 0 keeps a private ring of up to four 2 KiB
// slots filled with bulk async copies (cp.async.bulk -> shared memory, completion
// on per-slot mbarriers, all waits bounded) and refills a slot as soon as the warp
// has consumed it.  The ring is filled before the programmatic-dependent-launch
// wait, so weights are already streaming while the previous kernel finishes; only
// the small activation fragments are loaded after the wait (in bursts, so that
// their L2 latency is paid once per burst).  Grids never exceed what is
// co-resident (two CTAs per SM); a projection with few row-block groups is split
// further along k, which shortens the activation slice every CTA reads after the wait.
// Two arithmetic variants:
//   - CUDA cores (batch <= 4): 2 x batch fp32 accumulators per lane, finished by
//     a warp-shuffle reduction over the four lanes that share a row;
//   - mma.sync m16n8k16 (5 <= batch <= 15): at batch 8 the fp32 FMA pipe would
//     need ~8 FMAs per weight and co-limit the stream, so the 16x32 tile feeds
//     warp MMAs with the batch as the n = 8 operand.
// Activations arrive as hi + lo bf16 planes (x = hi + lo).
// Split-K partial sums are added in a fixed order, so results are bit-stable: warps
// through shared memory; cluster ranks one-sidedly - ranks 1.. store their sums
// into rank 0's shared memory (st.async + mbarrier complete_tx) and rank 0
// finishes the outputs - or, when a CTA handles several groups, through
// distributed shared memory with every rank finishing its share of the outputs.
// The fused epilogues live in epilogue.cuh.
#include <cooperative_groups.h>

#include "epilogue.cuh"

namespace cg = cooperative_groups;

namespace prsv {

constexpr int kGemvWarps = 8;
constexpr int kRingSlots = 4;
constexpr int kUnitChunks = 2;                       // tiles per ring slot (2 KiB)
constexpr int kGemvSmemBytes = kGemvWarps * kRingSlots * kUnitChunks * 1024;

struct GemvParams {
    const uint4 *w;
    const uint4 *x;      // hi plane; lo plane at x + x_plane
    size_t x_plane;      // in uint4 units
    int B, N, K;
    int b0;              // first batch row handled by this launch (x, outputs and ctx_len are indexed b0 + b)
    int row_blocks;      // N / 16
    int kchunks;         // K / 32
    int warps_k;         // warps of a CTA that split k (1, 2, 4, 8)
    int splits;          // cluster size along k
    int groups;          // row-block groups = row_blocks / (8 / warps_k)
    int slots;           // ring slots per warp actually used (1, 2 or 4): no more than the warp's run needs
    int push;            // cluster reduction by one-sided hand-over to rank 0 (else every rank reads all ranks)
    int recv_off;        // push: offset of rank 0's receive area in dynamic shared memory
    int *status;
    long long *trace;
    const uint8_t *next_w;
    uint32_t next_slice;   // bytes of next_w each CTA prefetches
    size_t next_bytes;
    int inject;            // test hook: warp 0 of CTA (0, 0) arms its first ring slot but never fills it
    const float *scales;   // W8: per packed row
    EpilogueArgs epi;
};

// two int8 codes (bytes at bit `shift` and `shift + 8` of w) as a bf16 pair: every code is exact in bf16
__device__ __forceinline__ uint32_t s8x2_to_bf16x2(uint32_t w, int shift)
{
    const int a = (int)(w << (24 - shift)) >> 24, b = (int)(w << (16 - shift)) >> 24;
    return pack_bf16((float)a, (float)b);
}
__device__ __forceinline__ float s8_to_f32(uint32_t w, int byte) { return (float)((int)(w << (24 - 8 * byte)) >> 24); }

// RB = 16-row blocks per warp: with two, every activation fragment a warp loads is used for two
// weight tiles, which halves the activation traffic from L2 (for batch 8 it is otherwise as large
// as the weight stream itself, and an SM takes in only ~50 GB/s in total).
// W8: the weights are int8 codes - a 1 KiB tile then covers 16 rows x 64 k (a lane's 16 bytes per row
// are k = 16 t .. 16 t + 15), the codes are widened to bf16 (exactly) in registers, and every output
// is multiplied by its row's scale in front of the epilogue.
template <int NB, bool MMA, int RB, bool W8 = false>
__global__ void __launch_bounds__(kGemvWarps * 32, 2) k_gemv_splitk(const __grid_constant__ GemvParams p)
{
    constexpr int NTB = MMA ? NB / 8 : 1;   // n-tiles that cover the batch
    constexpr int NT = 2 * NTB;             // hi planes then lo planes of the activations
    constexpr int XF = W8 ? 2 : 1;          // uint4 of activations per tile, lane and (batch row, plane): 8 k each
    constexpr int NX = (MMA ? NT : 2 * NB) * XF;   // activation fragments (uint4) per tile
    __shared__ float red[kGemvWarps][RB * 16][NB];       // per-warp partials
    __shared__ float cta_part[kGemvWarps * RB][16][NB];  // per-row-block CTA partials (read across the cluster)
    __shared__ uint64_t bars[kGemvWarps][kRingSlots];
    __shared__ uint64_t push_bar;
    __shared__ EpilogueTables tabs;
    __shared__ float scale_s[W8 ? kGemvWarps * RB * 16 : 1];   // W8: the scales of the group's rows
    extern __shared__ uint8_t gemv_smem_raw[];
    uint8_t *wsm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(gemv_smem_raw) + 127) & ~uintptr_t(127));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int rbs_per_cta = kGemvWarps / p.warps_k * RB;
    const int rbl = warp / p.warps_k * RB, wk = warp % p.warps_k;   // rbl: first of this warp's row blocks in the group
    const int s = blockIdx.y;                        // == cluster rank along k

    // this warp's run of k-chunks: part ki of ks = splits * warps_k equal parts (same for every group)
    const int ks = p.splits * p.warps_k, ki = s * p.warps_k + wk;
    const int c_begin = (int)((long long)p.kchunks * ki / ks);
    const int c_end = (int)((long long)p.kchunks * (ki + 1) / ks);
    uint8_t *ring = wsm + (size_t)warp * (p.slots * kUnitChunks * 1024);
    const uint32_t slot_mask = (uint32_t)p.slots - 1;

    trace_start(p.trace);
    pdl_launch_dependents();    // the next kernel may start its own weight fetch right away

    // The activation fragments of kBurst tiles are requested in one burst (their L2 latency is paid
    // once per burst) and used for the warp's RB row blocks: <= 64 registers of fragments.
    constexpr int kBurstBase = NX <= 2 ? 8 : (NX <= 4 ? 4 : 2);
    constexpr int kBurst = kBurstBase / RB >= kUnitChunks ? kBurstBase / RB : kUnitChunks;
    constexpr int kBurstUnits = kBurst / kUnitChunks;

    // ---- producer side of this warp's ring (lane 0 only): units in consumption order - per burst of
    // k, the units of row block 0, then those of row block 1
    int p_grp = blockIdx.x, p_c0 = c_begin, p_r = 0, p_u = 0;   // next unit: burst start, row block, unit in burst
    uint32_t n_issued = 0;
    const uint64_t pol = policy_evict_first();       // every weight byte is read once per step
    auto issue_next = [&]() {
        if (p_grp >= p.groups || c_begin >= c_end)
            return;
        const int p_c = p_c0 + p_u * kUnitChunks;
        const int n = min(kUnitChunks, c_end - p_c);
        const int slot = n_issued & slot_mask;
        const size_t rb = (size_t)p_grp * rbs_per_cta + rbl + p_r;
        const uint32_t bytes = (uint32_t)n * 1024u;
        mbar_expect_tx(&bars[warp][slot], bytes);
        if (!(p.inject == INJECT_GEMV_RING && n_issued == 0 && warp == 0 && blockIdx.x == 0 && blockIdx.y == 0))
            bulk_load_hint(ring + slot * (kUnitChunks * 1024),
                           reinterpret_cast<const uint8_t *>(p.w) + (rb * p.kchunks + p_c) * 1024, bytes, &bars[warp][slot], pol);
        ++n_issued;
        ++p_u;
        if (p_u == kBurstUnits || p_c0 + p_u * kUnitChunks >= c_end) {
            p_u = 0;
            if (++p_r == RB) {
                p_r = 0;
                p_c0 += kBurst;
                if (p_c0 >= c_end) {
                    p_c0 = c_begin;
                    p_grp += gridDim.x;
                }
            }
        }
    };
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kRingSlots; ++i)
            mbar_init(&bars[warp][i], 1);
        mbar_fence_init();
        for (int i = 0; i < p.slots; ++i)
            issue_next();
    }
    __syncwarp();

    const int part_floats = rbs_per_cta * 16 * NB;   // one rank's partial sums of a group
    if (p.push) {
        // rank 0 will receive the other ranks' partial sums: its barrier must exist (and expect them)
        // before anybody sends - a cluster barrier, split: arrive here, wait just before the sends, so
        // that a CTA which starts late does not spend the barrier's latency ahead of its dependency wait
        if (s == 0 && threadIdx.x == 0) {
            mbar_init(&push_bar, 1);
            mbar_fence_init();
            mbar_expect_tx(&push_bar, (uint32_t)(p.splits - 1) * part_floats * 4u);
        }
        __syncwarp();
        cluster_arrive_relaxed();
    }
    load_epilogue_tables(p.epi, tabs, p.b0, p.B);    // inputs of the step: safe before the wait
    const int xrow = p.K >> 3;                       // uint4 per activation row
    auto load_x = [&](int c, uint4 (&xq)[NX]) {
        if constexpr (MMA) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int b = (nt % NTB) * 8 + g;
                const uint4 *plane = p.x + (nt >= NTB ? p.x_plane : 0);
#pragma unroll
                for (int f = 0; f < XF; ++f)
                    xq[nt * XF + f] = b < p.B ? ld_cached(plane + (size_t)(p.b0 + b) * xrow + c * (4 * XF) + t * XF + f)
                                              : make_uint4(0, 0, 0, 0);
            }
        } else {
#pragma unroll
            for (int b = 0; b < NB; ++b)
#pragma unroll
                for (int f = 0; f < XF; ++f) {
                    const size_t o = (size_t)(p.b0 + b) * xrow + c * (4 * XF) + t * XF + f;
                    xq[b * XF + f] = b < p.B ? ld_cached(p.x + o) : make_uint4(0, 0, 0, 0);
                    xq[(NB + b) * XF + f] = b < p.B ? ld_cached(p.x + p.x_plane + o) : make_uint4(0, 0, 0, 0);
                }
        }
    };

    // W8: the scales of a group's rows are weights - fetched ahead of the stream (the first group's even
    // ahead of the wait), not behind the reduction where their memory round trip would sit on the tail
    auto load_scales = [&](int grp) {
        if constexpr (W8) {
            if (grp < p.groups)
                for (int i = threadIdx.x; i < rbs_per_cta * 16; i += blockDim.x)
                    scale_s[i] = p.scales[(size_t)grp * rbs_per_cta * 16 + i];
        }
    };
    load_scales(blockIdx.x);
    pdl_wait();   // x is produced by the previous kernel of the stream
    trace_waited(p.trace);

    uint32_t n_consumed = 0;
    bool ok = true;
    bool push_short = false;      // rank 0: the wait for the other ranks' partial sums ran out
    for (int grp = blockIdx.x; grp < p.groups; grp += gridDim.x) {
        float acc[RB][MMA ? NT : 2 * NB][MMA ? 4 : 1];
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int i = 0; i < (MMA ? NT : 2 * NB); ++i)
#pragma unroll
                for (int j = 0; j < (MMA ? 4 : 1); ++j)
                    acc[r][i][j] = 0.f;

        // eight weights of row g (wl) and of row g + 8 (wh) against the same eight k of every batch row
        auto fma8 = [&](float (&a_)[MMA ? NT : 2 * NB][MMA ? 4 : 1], const float (&l)[8], const float (&h)[8],
                        const uint4 (&xq)[NX], int f) {
            if constexpr (!MMA) {
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const uint4 &xh = xq[b * XF + f], &xl = xq[(NB + b) * XF + f];     // x = hi + lo, exact in fp32
                    const float x0 = bf_lo(xh.x) + bf_lo(xl.x), x1 = bf_hi(xh.x) + bf_hi(xl.x);
                    const float x2 = bf_lo(xh.y) + bf_lo(xl.y), x3 = bf_hi(xh.y) + bf_hi(xl.y);
                    const float x4 = bf_lo(xh.z) + bf_lo(xl.z), x5 = bf_hi(xh.z) + bf_hi(xl.z);
                    const float x6 = bf_lo(xh.w) + bf_lo(xl.w), x7 = bf_hi(xh.w) + bf_hi(xl.w);
                    float a = a_[2 * b][0], c = a_[2 * b + 1][0];
                    a = fmaf(l[0], x0, a); a = fmaf(l[1], x1, a); a = fmaf(l[2], x2, a); a = fmaf(l[3], x3, a);
                    a = fmaf(l[4], x4, a); a = fmaf(l[5], x5, a); a = fmaf(l[6], x6, a); a = fmaf(l[7], x7, a);
                    c = fmaf(h[0], x0, c); c = fmaf(h[1], x1, c); c = fmaf(h[2], x2, c); c = fmaf(h[3], x3, c);
                    c = fmaf(h[4], x4, c); c = fmaf(h[5], x5, c); c = fmaf(h[6], x6, c); c = fmaf(h[7], x7, c);
                    a_[2 * b][0] = a; a_[2 * b + 1][0] = c;
                }
            }
        };
        auto compute = [&](float (&a_)[MMA ? NT : 2 * NB][MMA ? 4 : 1], const uint4 &wl, const uint4 &wh, const uint4 (&xq)[NX]) {
            if constexpr (MMA && !W8) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    mma_bf16_16816(a_[nt], wl.x, wh.x, wl.y, wh.y, xq[nt].x, xq[nt].y);
                    mma_bf16_16816(a_[nt], wl.z, wh.z, wl.w, wh.w, xq[nt].z, xq[nt].w);
                }
            } else if constexpr (MMA && W8) {
                // word j of wl / wh = codes of k = 16 t + 4 j .. + 3: one m16n8k16 MMA per word
                const uint32_t lw[4] = {wl.x, wl.y, wl.z, wl.w}, hw[4] = {wh.x, wh.y, wh.z, wh.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t a0 = s8x2_to_bf16x2(lw[j], 0), a2 = s8x2_to_bf16x2(lw[j], 16);
                    const uint32_t a1 = s8x2_to_bf16x2(hw[j], 0), a3 = s8x2_to_bf16x2(hw[j], 16);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint4 &xv = xq[nt * 2 + (j >> 1)];
                        mma_bf16_16816(a_[nt], a0, a1, a2, a3, (j & 1) ? xv.z : xv.x, (j & 1) ? xv.w : xv.y);
                    }
                }
            } else if constexpr (!W8) {
                const float l[8] = {bf_lo(wl.x), bf_hi(wl.x), bf_lo(wl.y), bf_hi(wl.y), bf_lo(wl.z), bf_hi(wl.z), bf_lo(wl.w), bf_hi(wl.w)};
                const float h[8] = {bf_lo(wh.x), bf_hi(wh.x), bf_lo(wh.y), bf_hi(wh.y), bf_lo(wh.z), bf_hi(wh.z), bf_lo(wh.w), bf_hi(wh.w)};
                fma8(a_, l, h, xq, 0);
            } else {
                const uint32_t lw[4] = {wl.x, wl.y, wl.z, wl.w}, hw[4] = {wh.x, wh.y, wh.z, wh.w};
#pragma unroll
                for (int f = 0; f < 2; ++f) {
                    float l[8], h[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        l[i] = s8_to_f32(lw[2 * f + (i >> 2)], i & 3);
                        h[i] = s8_to_f32(hw[2 * f + (i >> 2)], i & 3);
                    }
                    fma8(a_, l, h, xq, f);
                }
            }
        };

        // ---- stream this warp's run through its ring
        for (int c0 = c_begin; ok && c0 < c_end; c0 += kBurst) {
            const int nb = min(kBurst, c_end - c0);
            uint4 xq[kBurst][NX];
#pragma unroll
            for (int u = 0; u < kBurst; ++u)
                if (u < nb)
                    load_x(c0 + u, xq[u]);
#pragma unroll
            for (int r = 0; r < RB; ++r) {
#pragma unroll
                for (int uu = 0; uu < kBurstUnits; ++uu) {
                    if (uu * kUnitChunks < nb && ok) {
                        const int slot = n_consumed & slot_mask;
                        const uint32_t ph = (n_consumed >> (p.slots == 4 ? 2 : p.slots - 1)) & 1;
                        ok = mbar_wait(&bars[warp][slot], ph, p.status, ST_TIMEOUT_FULL);
                        if (ok) {
                            const uint4 *wtile =
                                reinterpret_cast<const uint4 *>(ring + slot * (kUnitChunks * 1024)) + lane * 2;
#pragma unroll
                            for (int u = 0; u < kUnitChunks; ++u)
                                if (uu * kUnitChunks + u < nb) {
                                    const uint4 wl = wtile[u * 64], wh = wtile[u * 64 + 1];
                                    compute(acc[r], wl, wh, xq[uu * kUnitChunks + u]);
                                }
                        }
                        ++n_consumed;
                        __syncwarp();
                        if (lane == 0 && ok)
                            issue_next();       // the slot just read is free again
                    }
                }
            }
        }

        trace_streamed(p.trace, threadIdx.x == 0);
        if (p.next_slice && grp + (int)gridDim.x >= p.groups && threadIdx.x == 32) {
            // this CTA's stream is over: HBM would idle until the next kernel's late CTAs start -
            // pull its slice of that kernel's weights into L2 meanwhile
            const size_t o = (size_t)(blockIdx.y * gridDim.x + blockIdx.x) * p.next_slice;
            if (o < p.next_bytes) {
                const size_t left = p.next_bytes - o;
                bulk_prefetch_l2(p.next_w + o, (uint32_t)(left < p.next_slice ? left : p.next_slice) & ~15u);
            }
        }
        // ---- warp partial -> shared memory: red[warp][row block of the warp * 16 + row][b]
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            if constexpr (MMA) {
#pragma unroll
                for (int nt = 0; nt < NTB; ++nt) {
                    red[warp][r * 16 + g][nt * 8 + 2 * t] = acc[r][nt][0] + acc[r][NTB + nt][0];
                    red[warp][r * 16 + g][nt * 8 + 2 * t + 1] = acc[r][nt][1] + acc[r][NTB + nt][1];
                    red[warp][r * 16 + g + 8][nt * 8 + 2 * t] = acc[r][nt][2] + acc[r][NTB + nt][2];
                    red[warp][r * 16 + g + 8][nt * 8 + 2 * t + 1] = acc[r][nt][3] + acc[r][NTB + nt][3];
                }
            } else {
#pragma unroll
                for (int i = 0; i < 2 * NB; ++i) {
                    float v = acc[r][i][0];
                    v += __shfl_xor_sync(0xffffffffu, v, 1);
                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                    if (t == 0)
                        red[warp][r * 16 + g + 8 * (i & 1)][i >> 1] = v;
                }
            }
        }
        __syncthreads();

        // ---- sum over the warps that split k (fixed order) -> cta_part[rbl][row][b]
        for (int i = threadIdx.x; i < rbs_per_cta * 16 * NB; i += blockDim.x) {
            const int b = i % NB, row = (i / NB) % 16, rl = i / (16 * NB);
            const int wrow = rl / RB, r = rl % RB;       // warp row of the CTA, row block of that warp
            float v = 0.f;
            for (int k = 0; k < p.warps_k; ++k)
                v += red[wrow * p.warps_k + k][r * 16 + row][b];
            cta_part[rl][row][b] = v;
        }

        // ---- sum over the cluster ranks (fixed order)
        const int n_out = rbs_per_cta * 8 * NB;          // (row block, pair, batch row) triples of the group
        if (p.splits > 1 && p.push) {
            // One-sided: ranks 1.. store their partial sums into rank 0's shared memory, signalling its
            // barrier with the bytes, and are done; rank 0 waits for all the bytes and finishes every
            // output.  No cluster barrier on the critical path.  (One group per CTA in this mode.)
            __syncthreads();
            cluster_wait();       // (the arrival in the prologue: rank 0's barrier exists)
            float *recv = reinterpret_cast<float *>(wsm + p.recv_off);
            if (s != 0) {
                const uint32_t dst = cluster_map(recv + (size_t)(s - 1) * part_floats, 0);
                const uint32_t bar = cluster_map(&push_bar, 0);
                const float4 *src = reinterpret_cast<const float4 *>(&cta_part[0][0][0]);
                for (int i = threadIdx.x; i < part_floats / 4; i += blockDim.x)
                    st_async_v4(dst + i * 16, src[i], bar);
            } else {
                const bool got = mbar_wait(&push_bar, 0, p.status, ST_TIMEOUT_FULL);
                push_short = !got;
                ok = got && ok;
                for (int i = threadIdx.x; i < n_out; i += blockDim.x) {
                    const int b = i % NB, r = (i / NB) % 8, rl = i / (8 * NB);
                    if (b >= p.B)
                        continue;
                    float v0 = cta_part[rl][r][b], v1 = cta_part[rl][r + 8][b];
                    for (int q = 1; q < p.splits; ++q) {
                        v0 += recv[(size_t)(q - 1) * part_floats + (rl * 16 + r) * NB + b];
                        v1 += recv[(size_t)(q - 1) * part_floats + (rl * 16 + r + 8) * NB + b];
                    }
                    if constexpr (W8) {
                        v0 *= scale_s[rl * 16 + r];
                        v1 *= scale_s[rl * 16 + r + 8];
                    }
                    apply_epilogue(p.epi, tabs, b, false, p.N, p.b0 + b, (grp * rbs_per_cta + rl) * 8 + r, v0, v1);
                }
            }
        } else if (p.splits > 1) {
            // every rank finishes its share of the outputs, reading all ranks' partial sums
            cg::cluster_group cluster = cg::this_cluster();
            cluster.sync();
            const float *remote[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
                remote[q] = cluster.map_shared_rank(&cta_part[0][0][0], q < p.splits ? q : 0);
            for (int i = threadIdx.x * p.splits + s; i < n_out; i += blockDim.x * p.splits) {
                const int b = i % NB, r = (i / NB) % 8, rl = i / (8 * NB);
                if (b >= p.B)
                    continue;
                float v0 = 0.f, v1 = 0.f;
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (q < p.splits) {
                        v0 += remote[q][(rl * 16 + r) * NB + b];
                        v1 += remote[q][(rl * 16 + r + 8) * NB + b];
                    }
                if constexpr (W8) {
                    v0 *= scale_s[rl * 16 + r];
                    v1 *= scale_s[rl * 16 + r + 8];
                }
                apply_epilogue(p.epi, tabs, b, false, p.N, p.b0 + b, (grp * rbs_per_cta + rl) * 8 + r, v0, v1);
            }
            cluster.sync();   // peers' shared memory must outlive the reads; also fences red/cta_part reuse
            load_scales(grp + gridDim.x);
        } else {
            __syncthreads();
            for (int i = threadIdx.x; i < n_out; i += blockDim.x) {
                const int b = i % NB, r = (i / NB) % 8, rl = i / (8 * NB);
                if (b >= p.B)
                    continue;
                float v0 = cta_part[rl][r][b], v1 = cta_part[rl][r + 8][b];
                if constexpr (W8) {
                    v0 *= scale_s[rl * 16 + r];
                    v1 *= scale_s[rl * 16 + r + 8];
                }
                apply_epilogue(p.epi, tabs, b, false, p.N, p.b0 + b, (grp * rbs_per_cta + rl) * 8 + r, v0, v1);
            }
            __syncthreads();
            load_scales(grp + gridDim.x);
        }
    }
    if (p.push && s == 0) {
        // Rank 0 gave up waiting for a rank's partial sums: that rank may still store them into this
        // CTA's shared memory, and a store into a CTA that has exited is a fault.  Stay until every other
        // rank has left (its stores were issued before that), then give the stores in flight a bounded
        // time to land.  (The barrier counts only threads that have not exited; the other ranks never
        // wait on it.)
        if (__syncthreads_or(push_short ? 1 : 0)) {
            cluster_arrive_relaxed();
            cluster_wait();
            if (threadIdx.x == 0)
                mbar_wait(&push_bar, 0, p.status, ST_TIMEOUT_FULL);
            __syncthreads();
        }
    }
    trace_end(p.trace);
}

template <int NB, bool MMA, int RB, bool W8>
static cudaError_t launch_variant(GemvParams &p, int sm_count, int pdl, cudaStream_t s)
{
    static PerDeviceSize smem_limit;      // per instantiation and device
    {
        cudaError_t e = ensure_dynamic_smem(k_gemv_splitk<NB, MMA, RB, W8>, smem_limit, kGemvSmemBytes + 32 * 1024 + 128);
        if (e != cudaSuccess)
            return e;
    }
    // Mapping: k is split over the 8 warps of a CTA while every warp still gets at least two
    // tiles (otherwise fewer warps split k and the others take further row blocks); cluster ranks
    // add splits only while the grid stays within the co-resident CTAs; groups beyond the grid
    // become further loop iterations.  Depends only on the shapes and the SM count, never on the
    // prefetch setting.
    // (an int8 tile covers 64 k, as much as two 16-bit tiles: one per warp is the same slice of k)
    constexpr int kMinChunks = W8 ? 1 : 2;
    int wk = kGemvWarps;
    while (wk > 1 && p.kchunks / wk < kMinChunks && p.row_blocks % (2 * RB * kGemvWarps / wk) == 0) wk /= 2;
    p.warps_k = wk;
    p.groups = p.row_blocks / (kGemvWarps / wk * RB);
    // Two CTA slots per SM for every matrix (64 KiB rings, <= 128 registers).  A small projection whose
    // rows alone give few groups is split further along k instead (QKV of an 8B shard: 24 groups x 8
    // ranks): each CTA then reads a short slice of the activations after the wait, and that read - not
    // the weights, which are in the rings by then - is what such a kernel's time consists of.
    const int slots_total = 2 * sm_count;
    int splits = 1;
    while (splits < 8 && p.groups * splits * 2 <= slots_total && p.kchunks / (wk * splits * 2) >= kMinChunks) splits *= 2;
    p.splits = splits;
    int clusters = slots_total / p.splits;
    if (clusters > p.groups) clusters = p.groups;
    if (clusters < 1) clusters = 1;
    // ring depth: no deeper than a warp's whole run, so that a small projection leaves the shared
    // memory to the kernels it shares the SM with
    const int groups_per_cta = (p.groups + clusters - 1) / clusters;
    const int chunks_per_warp = (p.kchunks + p.splits * p.warps_k - 1) / (p.splits * p.warps_k);
    const int units = groups_per_cta * RB * ((chunks_per_warp + kUnitChunks - 1) / kUnitChunks);
    p.slots = units >= 4 ? 4 : (units >= 2 ? 2 : 1);
    // one-sided cluster reduction when every CTA has a single group and rank 0's receive area is small
    const size_t ring_bytes = (size_t)kGemvWarps * p.slots * kUnitChunks * 1024;
    const size_t recv_bytes = (size_t)(p.splits - 1) * (kGemvWarps / p.warps_k * RB) * 16 * NB * 4;
    p.push = p.splits > 1 && groups_per_cta == 1 && recv_bytes <= 32 * 1024;
    p.recv_off = (int)ring_bytes;
    p.next_slice = 0;
    if (p.next_w && p.next_bytes) {
        const size_t n_ctas = (size_t)clusters * p.splits;
        p.next_slice = (uint32_t)(((p.next_bytes + n_ctas - 1) / n_ctas + 127) & ~size_t(127));
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(clusters, p.splits, 1);
    cfg.blockDim = dim3(kGemvWarps * 32);
    cfg.dynamicSmemBytes = ring_bytes + (p.push ? recv_bytes : 0) + 128;
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    int n = pdl_attr(at, pdl);
    if (p.splits > 1) {
        at[n].id = cudaLaunchAttributeClusterDimension;
        at[n].val.clusterDim.x = 1;
        at[n].val.clusterDim.y = p.splits;
        at[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = at;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, k_gemv_splitk<NB, MMA, RB, W8>, p);
}

template <bool W8>
static cudaError_t launch_by_batch(GemvParams &p, int B, int sm_count, int pdl, cudaStream_t s)
{
    // two row blocks per warp whenever the matrix has enough row blocks to still fill the SMs
    const bool two = p.row_blocks % 2 == 0 && p.row_blocks >= 32;
    if (B == 1) return two ? launch_variant<1, false, 2, W8>(p, sm_count, pdl, s) : launch_variant<1, false, 1, W8>(p, sm_count, pdl, s);
    if (B == 2) return two ? launch_variant<2, false, 2, W8>(p, sm_count, pdl, s) : launch_variant<2, false, 1, W8>(p, sm_count, pdl, s);
    // (int8 weights double the activation fragments a lane holds per tile: batch 3-4 takes the MMA form there)
    if (B <= 4 && !W8) return two ? launch_variant<4, false, 2, false>(p, sm_count, pdl, s) : launch_variant<4, false, 1, false>(p, sm_count, pdl, s);
    if (B <= 8) return two ? launch_variant<8, true, 2, W8>(p, sm_count, pdl, s) : launch_variant<8, true, 1, W8>(p, sm_count, pdl, s);
    return two ? launch_variant<16, true, 2, W8>(p, sm_count, pdl, s) : launch_variant<16, true, 1, W8>(p, sm_count, pdl, s);
}

cudaError_t launch_gemv(const GemvArgs &a, int sm_count, cudaStream_t s)
{
    const int tile_k = a.w8 ? 64 : 32;       // k covered by a 1 KiB tile
    if (a.B < 1 || a.B > 16 || a.N % 16 || a.K % tile_k || (a.w8 && !a.scales))
        return cudaErrorInvalidValue;
    GemvParams p;
    p.w = reinterpret_cast<const uint4 *>(a.w);
    p.x = reinterpret_cast<const uint4 *>(a.x);
    p.x_plane = a.x_plane / 8;
    p.B = a.B; p.N = a.N; p.K = a.K; p.b0 = a.b0;
    p.row_blocks = a.N / 16;
    p.kchunks = a.K / tile_k;
    p.epi = a.epi;
    p.status = a.status;
    p.trace = a.trace;
    p.next_w = reinterpret_cast<const uint8_t *>(a.next_w);
    p.next_bytes = a.next_bytes;
    p.inject = a.inject;
    p.scales = a.scales;
    return a.w8 ? launch_by_batch<true>(p, a.B, sm_count, a.pdl, s) : launch_by_batch<false>(p, a.B, sm_count, a.pdl, s);
}

}  // namespace prsv
