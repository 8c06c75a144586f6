// Gather of a step's input buffers from pinned host memory into the layer's staging area in device
// memory, for the host-buffer entry point.  It runs on a stream of its own, so the transfer of one
// call's inputs over PCIe overlaps the kernels of the call before it; the kernels of the step then
// read device memory.  One launch replaces 2P + 1 separate copy calls (whose submission cost alone
// would exceed a small layer's run time).  Every thread keeps eight 16-byte reads in flight: a read
// over PCIe takes microseconds, the link is only busy with tens of thousands of them outstanding.
#include "common.cuh"
#include "kernels.h"

namespace prsv {

struct StageParams {
    const uint4 *src[2 * kMaxParts + 1];
    uint4 *dst[2 * kMaxParts + 1];
    int n;                // buffers
    uint32_t chunks;      // 16-byte pieces per buffer
    const int *ctx_src;   // optional: sequence lengths
    int *ctx_dst;
    int n_ctx;
};

constexpr int kStageThreads = 256;
constexpr int kStageBurst = 8;

__global__ void __launch_bounds__(kStageThreads) k_stage_inputs(const __grid_constant__ StageParams p)
{
    const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x, n_thr = gridDim.x * blockDim.x;
    if (p.ctx_src)
        for (int i = (int)tid; i < p.n_ctx; i += (int)n_thr)
            p.ctx_dst[i] = p.ctx_src[i];
    const uint64_t total = (uint64_t)p.n * p.chunks;
    for (uint64_t i0 = tid; i0 < total; i0 += (uint64_t)n_thr * kStageBurst) {
        uint4 v[kStageBurst];
#pragma unroll
        for (int u = 0; u < kStageBurst; ++u) {
            const uint64_t i = i0 + (uint64_t)u * n_thr;
            if (i < total)
                v[u] = ld_stream(p.src[i / p.chunks] + i % p.chunks);
        }
#pragma unroll
        for (int u = 0; u < kStageBurst; ++u) {
            const uint64_t i = i0 + (uint64_t)u * n_thr;
            if (i < total)
                p.dst[i / p.chunks][i % p.chunks] = v[u];
        }
    }
}

cudaError_t launch_stage_inputs(const void *const *src, void *const *dst, int n, size_t bytes_each, const int *ctx_src,
                                int *ctx_dst, int n_ctx, cudaStream_t s)
{
    if (n < 0 || n > 2 * kMaxParts + 1 || bytes_each % 16)
        return cudaErrorInvalidValue;
    StageParams p = {};
    for (int i = 0; i < n; ++i) {
        p.src[i] = reinterpret_cast<const uint4 *>(src[i]);
        p.dst[i] = reinterpret_cast<uint4 *>(dst[i]);
    }
    p.n = n;
    p.chunks = (uint32_t)(bytes_each / 16);
    p.ctx_src = ctx_src;
    p.ctx_dst = ctx_dst;
    p.n_ctx = n_ctx;
    const uint64_t total = (uint64_t)n * p.chunks;
    int ctas = (int)((total + (uint64_t)kStageThreads * kStageBurst - 1) / ((uint64_t)kStageThreads * kStageBurst));
    // At most 8 CTAs: 8 x 256 threads x 8 reads of 16 bytes = 256 KB in flight keep the link busy (~45 GB/s
    // x a few microseconds of latency), and every further CTA takes a slot - and registers - from the main
    // stream's kernels, whose early-launched CTAs fill the SMs (measured: 4 / 8 / 16 / 32 / 128 CTAs).
    ctas = ctas < 1 ? 1 : (ctas > 8 ? 8 : ctas);
    k_stage_inputs<<<ctas, kStageThreads, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace prsv
