// Split-K GEMV for decode batches below 16: y[b,n] = sum_k x[b,k] * W[n,k].
//
// The projection layers of the decode phase reuse each weight only `batch`
// times (Section 2, "LLM decoding is memory BW-limited"), so the kernel is a
// pure weight stream: every warp walks a contiguous run of 1 KiB fragment-major
// tiles (16 output rows x 32 k, see pack.cu) with two 128-bit loads per lane per
// tile and no shared-memory staging.  Two arithmetic variants share the loop:
//   - CUDA cores (batch <= 4): 2 x batch fp32 accumulators per lane, finished by
//     a warp-shuffle reduction over the four lanes that share a row;
//   - mma.sync m16n8k16 (5 <= batch <= 15): at batch 8 the fp32 FMA pipe would
//     need ~8 FMAs per weight and co-limit the stream, so the 16x32 tile feeds
//     two warp MMAs with the batch as the n = 8 operand.
// Split-K: the k range is divided over the warps of a CTA (summed through
// shared memory) and over the CTAs of a thread-block cluster (summed by rank 0
// through distributed shared memory), always in a fixed order, so results are
// bit-stable.  Rank 0 applies the fused epilogue (epilogue.cuh).
#include <cooperative_groups.h>

#include "epilogue.cuh"

namespace cg = cooperative_groups;

namespace prsv {

int g_pdl = 0;

constexpr int kGemvWarps = 8;
constexpr int kGemvUnroll = 4;

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
    EpilogueArgs epi;
};

template <int NB, bool MMA>
__global__ void __launch_bounds__(kGemvWarps * 32) k_gemv_splitk(const __grid_constant__ GemvParams p)
{
    constexpr int NTB = MMA ? NB / 8 : 1;   // n-tiles that cover the batch
    constexpr int NT = 2 * NTB;             // hi planes then lo planes of the activations
    __shared__ float red[kGemvWarps][16][NB];      // per-warp partials
    __shared__ float cta_part[kGemvWarps][16][NB];  // per-row-block CTA partials (read by cluster rank 0)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int rbs_per_cta = kGemvWarps / p.warps_k;
    const int rbl = warp / p.warps_k, wk = warp % p.warps_k;
    const int rb = blockIdx.x * rbs_per_cta + rbl;
    const int s = blockIdx.y;                        // == cluster rank along k
    const bool active = rb < p.row_blocks;

    // k-chunk range of this CTA, then of this warp
    const int cta_lo = (int)((long long)p.kchunks * s / p.splits);
    const int cta_hi = (int)((long long)p.kchunks * (s + 1) / p.splits);
    const int span = cta_hi - cta_lo;
    const int c_begin = cta_lo + (int)((long long)span * wk / p.warps_k);
    const int c_end = cta_lo + (int)((long long)span * (wk + 1) / p.warps_k);

    float acc[MMA ? NT : 2 * NB][MMA ? 4 : 1];
#pragma unroll
    for (int i = 0; i < (MMA ? NT : 2 * NB); ++i)
#pragma unroll
        for (int j = 0; j < (MMA ? 4 : 1); ++j)
            acc[i][j] = 0.f;

    const uint4 *wp = p.w + (size_t)rb * p.kchunks * 64 + lane * 2;
    const int xrow = p.K >> 3;                       // uint4 per activation row

    pdl_wait();   // x is produced by the previous kernel of the stream

    if (active) {
        auto compute = [&](const uint4 &wl, const uint4 &wh, const uint4 (&xq)[MMA ? NT : 2 * NB]) {
            if constexpr (MMA) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    mma_bf16_16816(acc[nt], wl.x, wh.x, wl.y, wh.y, xq[nt].x, xq[nt].y);
                    mma_bf16_16816(acc[nt], wl.z, wh.z, wl.w, wh.w, xq[nt].z, xq[nt].w);
                }
            } else {
                const float l0 = bf_lo(wl.x), l1 = bf_hi(wl.x), l2 = bf_lo(wl.y), l3 = bf_hi(wl.y);
                const float l4 = bf_lo(wl.z), l5 = bf_hi(wl.z), l6 = bf_lo(wl.w), l7 = bf_hi(wl.w);
                const float h0 = bf_lo(wh.x), h1 = bf_hi(wh.x), h2 = bf_lo(wh.y), h3 = bf_hi(wh.y);
                const float h4 = bf_lo(wh.z), h5 = bf_hi(wh.z), h6 = bf_lo(wh.w), h7 = bf_hi(wh.w);
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const uint4 &xh = xq[b], &xl = xq[NB + b];     // x = hi + lo, exact in fp32
                    const float x0 = bf_lo(xh.x) + bf_lo(xl.x), x1 = bf_hi(xh.x) + bf_hi(xl.x);
                    const float x2 = bf_lo(xh.y) + bf_lo(xl.y), x3 = bf_hi(xh.y) + bf_hi(xl.y);
                    const float x4 = bf_lo(xh.z) + bf_lo(xl.z), x5 = bf_hi(xh.z) + bf_hi(xl.z);
                    const float x6 = bf_lo(xh.w) + bf_lo(xl.w), x7 = bf_hi(xh.w) + bf_hi(xl.w);
                    float a = acc[2 * b][0], c = acc[2 * b + 1][0];
                    a = fmaf(l0, x0, a); a = fmaf(l1, x1, a); a = fmaf(l2, x2, a); a = fmaf(l3, x3, a);
                    a = fmaf(l4, x4, a); a = fmaf(l5, x5, a); a = fmaf(l6, x6, a); a = fmaf(l7, x7, a);
                    c = fmaf(h0, x0, c); c = fmaf(h1, x1, c); c = fmaf(h2, x2, c); c = fmaf(h3, x3, c);
                    c = fmaf(h4, x4, c); c = fmaf(h5, x5, c); c = fmaf(h6, x6, c); c = fmaf(h7, x7, c);
                    acc[2 * b][0] = a; acc[2 * b + 1][0] = c;
                }
            }
        };
        auto load_x = [&](int c, uint4 (&xq)[MMA ? NT : 2 * NB]) {
            if constexpr (MMA) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const int b = (nt % NTB) * 8 + g;
                    const uint4 *plane = p.x + (nt >= NTB ? p.x_plane : 0);
                    xq[nt] = b < p.B ? ld_cached(plane + (size_t)(p.b0 + b) * xrow + c * 4 + t) : make_uint4(0, 0, 0, 0);
                }
            } else {
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    xq[b] = b < p.B ? ld_cached(p.x + (size_t)(p.b0 + b) * xrow + c * 4 + t) : make_uint4(0, 0, 0, 0);
                    xq[NB + b] = b < p.B ? ld_cached(p.x + p.x_plane + (size_t)(p.b0 + b) * xrow + c * 4 + t)
                                         : make_uint4(0, 0, 0, 0);
                }
            }
        };

        int c = c_begin;
        for (; c + kGemvUnroll <= c_end; c += kGemvUnroll) {
            uint4 wl[kGemvUnroll], wh[kGemvUnroll];
            uint4 xq[kGemvUnroll][MMA ? NT : 2 * NB];
#pragma unroll
            for (int u = 0; u < kGemvUnroll; ++u) {
                wl[u] = ld_stream(wp + (size_t)(c + u) * 64);
                wh[u] = ld_stream(wp + (size_t)(c + u) * 64 + 1);
            }
#pragma unroll
            for (int u = 0; u < kGemvUnroll; ++u)
                load_x(c + u, xq[u]);
#pragma unroll
            for (int u = 0; u < kGemvUnroll; ++u)
                compute(wl[u], wh[u], xq[u]);
        }
        for (; c < c_end; ++c) {
            uint4 xq[MMA ? NT : 2 * NB];
            const uint4 wl = ld_stream(wp + (size_t)c * 64);
            const uint4 wh = ld_stream(wp + (size_t)c * 64 + 1);
            load_x(c, xq);
            compute(wl, wh, xq);
        }
    }

    pdl_launch_dependents();

    // ---- warp partial -> shared memory: red[warp][row][b]
    if constexpr (MMA) {
#pragma unroll
        for (int nt = 0; nt < NTB; ++nt) {
            red[warp][g][nt * 8 + 2 * t] = acc[nt][0] + acc[NTB + nt][0];
            red[warp][g][nt * 8 + 2 * t + 1] = acc[nt][1] + acc[NTB + nt][1];
            red[warp][g + 8][nt * 8 + 2 * t] = acc[nt][2] + acc[NTB + nt][2];
            red[warp][g + 8][nt * 8 + 2 * t + 1] = acc[nt][3] + acc[NTB + nt][3];
        }
    } else {
#pragma unroll
        for (int i = 0; i < 2 * NB; ++i) {
            float v = acc[i][0];
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            v += __shfl_xor_sync(0xffffffffu, v, 2);
            if (t == 0)
                red[warp][g + 8 * (i & 1)][i >> 1] = v;
        }
    }
    __syncthreads();

    // ---- sum over the warps that split k (fixed order) -> cta_part[rbl][row][b]
    for (int i = threadIdx.x; i < rbs_per_cta * 16 * NB; i += blockDim.x) {
        const int b = i % NB, row = (i / NB) % 16, rl = i / (16 * NB);
        float v = 0.f;
        for (int k = 0; k < p.warps_k; ++k)
            v += red[rl * p.warps_k + k][row][b];
        cta_part[rl][row][b] = v;
    }

    if (p.splits > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();
        if (s == 0) {
            for (int i = threadIdx.x; i < rbs_per_cta * 8 * NB; i += blockDim.x) {
                const int b = i % NB, r = (i / NB) % 8, rl = i / (8 * NB);
                const int rbg = blockIdx.x * rbs_per_cta + rl;
                if (rbg >= p.row_blocks || b >= p.B)
                    continue;
                float v0 = 0.f, v1 = 0.f;
                for (int q = 0; q < p.splits; ++q) {
                    const float *remote = cluster.map_shared_rank(&cta_part[0][0][0], q);
                    v0 += remote[(rl * 16 + r) * NB + b];
                    v1 += remote[(rl * 16 + r + 8) * NB + b];
                }
                apply_epilogue(p.epi, false, p.N, p.b0 + b, rbg * 8 + r, v0, v1);
            }
        }
        cluster.sync();   // peers' shared memory must outlive rank 0's reads
    } else {
        __syncthreads();
        for (int i = threadIdx.x; i < rbs_per_cta * 8 * NB; i += blockDim.x) {
            const int b = i % NB, r = (i / NB) % 8, rl = i / (8 * NB);
            const int rbg = blockIdx.x * rbs_per_cta + rl;
            if (rbg >= p.row_blocks || b >= p.B)
                continue;
            apply_epilogue(p.epi, false, p.N, p.b0 + b, rbg * 8 + r, cta_part[rl][r][b], cta_part[rl][r + 8][b]);
        }
    }
}

template <int NB, bool MMA>
static cudaError_t launch_variant(const GemvParams &p, cudaStream_t s)
{
    const int rbs_per_cta = kGemvWarps / p.warps_k;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((p.row_blocks + rbs_per_cta - 1) / rbs_per_cta, p.splits, 1);
    cfg.blockDim = dim3(kGemvWarps * 32);
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    int n = pdl_attr(at);
    if (p.splits > 1) {
        at[n].id = cudaLaunchAttributeClusterDimension;
        at[n].val.clusterDim.x = 1;
        at[n].val.clusterDim.y = p.splits;
        at[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = at;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, k_gemv_splitk<NB, MMA>, p);
}

static int pow2_floor(int v)
{
    int r = 1;
    while (r * 2 <= v)
        r *= 2;
    return r;
}

cudaError_t launch_gemv(const GemvArgs &a, int sm_count, cudaStream_t s)
{
    if (a.B < 1 || a.B > 16 || a.N % 16 || a.K % 32)
        return cudaErrorInvalidValue;
    GemvParams p;
    p.w = reinterpret_cast<const uint4 *>(a.w);
    p.x = reinterpret_cast<const uint4 *>(a.x);
    p.x_plane = a.x_plane / 8;
    p.B = a.B; p.N = a.N; p.K = a.K; p.b0 = a.b0;
    p.row_blocks = a.N / 16;
    p.kchunks = a.K / 32;
    p.epi = a.epi;

    // Split k so that about 16 warps per SM each own a few tiles.  The choice depends
    // only on the shapes and the SM count, never on the prefetch setting.
    const long long tiles = (long long)p.row_blocks * p.kchunks;
    const long long target_warps = (long long)sm_count * 16;
    long long per_warp = tiles / target_warps;
    if (per_warp < 2) per_warp = 2;
    if (per_warp > 16) per_warp = 16;
    int ks = (int)(p.kchunks / per_warp);
    if (ks < 1) ks = 1;
    ks = pow2_floor(ks);
    if (ks > 64) ks = 64;
    p.warps_k = ks < kGemvWarps ? ks : kGemvWarps;
    p.splits = ks / p.warps_k;
    if (p.splits < 1) p.splits = 1;

    if (a.B == 1) return launch_variant<1, false>(p, s);
    if (a.B == 2) return launch_variant<2, false>(p, s);
    if (a.B <= 4) return launch_variant<4, false>(p, s);
    if (a.B <= 8) return launch_variant<8, true>(p, s);
    return launch_variant<16, true>(p, s);
}

}  // namespace prsv
