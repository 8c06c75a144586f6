// Read-bandwidth microbenchmark: the denominator for "fraction of what a pure read stream
// reaches on this GPU".  A buffer larger than L2 measures HBM; a buffer well inside L2, read
// repeatedly, measures L2.  The caller owns the buffer; nothing is allocated here.
#include "../../include/preserve.h"
#include "common.cuh"

namespace prsv {

__global__ void __launch_bounds__(512) k_stream_read(const uint4 *p, size_t n_vec, unsigned *sink)
{
    // grid-stride, 8 independent 128-bit loads in flight per thread
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned fold = 0;
    for (; i + 7 * stride < n_vec; i += 8 * stride) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
            v[u] = ld_stream(p + i + u * stride);
#pragma unroll
        for (int u = 0; u < 8; ++u)
            fold ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    for (; i < n_vec; i += stride) {
        const uint4 v = ld_stream(p + i);
        fold ^= v.x ^ v.y ^ v.z ^ v.w;
    }
    if (fold == 0x5eed1234u && sink)      // practically never: keeps the loads alive
        *sink = fold;
}

// ---- single-launch streaming: the whole measurement is ONE kernel that walks the buffer `passes`
// times, so launch ramp and tail are paid once and an L2-resident buffer is really read from L2.
// Every CTA owns a contiguous slice of the buffer (all CTAs together cover it once per pass).
// path 0: 128-bit read-only loads, 8 in flight per thread;
// path 1: bulk async copies (cp.async.bulk, the path the GEMV and attention kernels use) of
//         `chunk` bytes into a shared-memory ring, `stages` copies in flight per CTA.
struct StreamParams {
    const uint8_t *buf;
    size_t slice;        // bytes per CTA (multiple of `chunk`)
    int passes;
    uint32_t chunk;
    int stages;
    int producers;       // path 1 / 2: issuing threads per CTA, each with its own ring and sub-slice
    int same_warp;       // path 2: the issuing threads are lanes of one warp instead of lane 0 of several warps
    int *status;         // status block (bounded waits report here)
    unsigned *sink;
};

__global__ void __launch_bounds__(256) k_stream_ld(const __grid_constant__ StreamParams p)
{
    const uint4 *base = reinterpret_cast<const uint4 *>(p.buf + (size_t)blockIdx.x * p.slice);
    const size_t n_vec = p.slice / 16;
    unsigned fold = 0;
    for (int pass = 0; pass < p.passes; ++pass) {
        size_t i = threadIdx.x;
        for (; i + 7 * blockDim.x < n_vec; i += 8 * blockDim.x) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
                v[u] = ld_stream(base + i + u * blockDim.x);
#pragma unroll
            for (int u = 0; u < 8; ++u)
                fold ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
        }
        for (; i < n_vec; i += blockDim.x) {
            const uint4 v = ld_stream(base + i);
            fold ^= v.x ^ v.y ^ v.z ^ v.w;
        }
    }
    if (fold == 0x5eed1234u && p.sink)
        *p.sink = fold;
}

constexpr int kStreamMaxStages = 12;
constexpr int kStreamMaxProducers = 8;
__global__ void __launch_bounds__(32 * kStreamMaxProducers) k_stream_bulk(const __grid_constant__ StreamParams p)
{
    extern __shared__ uint8_t stream_smem_raw[];
    uint8_t *ring0 = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(stream_smem_raw) + 127) & ~uintptr_t(127));
    __shared__ uint64_t bars[kStreamMaxProducers][kStreamMaxStages];
    // issuing threads: lane 0 of `producers` warps, or (same_warp) lanes 0.. of warp 0
    if (p.same_warp ? (int)threadIdx.x >= p.producers : (threadIdx.x & 31) != 0)
        return;
    const int w = p.same_warp ? (int)threadIdx.x : (int)(threadIdx.x >> 5);
    uint8_t *ring = ring0 + (size_t)w * p.stages * p.chunk;
    for (int i = 0; i < p.stages; ++i)
        mbar_init(&bars[w][i], 1);
    mbar_fence_init();
    const size_t sub = p.slice / p.producers;           // bytes per producer (multiple of chunk)
    const uint8_t *base = p.buf + (size_t)blockIdx.x * p.slice + (size_t)w * sub;
    const size_t per_pass = sub / p.chunk;
    const size_t total = per_pass * (size_t)p.passes;
    // keep `stages` copies in flight: wait for the oldest, issue the next into its slot
    for (size_t i = 0; i < total + p.stages; ++i) {
        const int st = (int)(i % p.stages);
        if (i >= (size_t)p.stages) {
            const uint32_t ph = (uint32_t)((i / p.stages - 1) & 1);
            if (!mbar_wait(&bars[w][st], ph, p.status, ST_TIMEOUT_FULL))
                return;                                 // (copies in flight land in this CTA's memory at most)
        }
        if (i < total) {
            mbar_expect_tx(&bars[w][st], p.chunk);
            bulk_load(ring + (size_t)st * p.chunk, base + (i % per_pass) * p.chunk, p.chunk, &bars[w][st]);
        }
    }
}

// path 3: the tcgen05 GEMM's weight loads - 2-D tiled TMA copies (128-byte swizzle) of boxes of 64 columns x
// `rows` rows out of a [n_rows, 8192] bf16 matrix (row stride 16 KiB): CTA c walks the 128 column blocks of
// row tile c mod n_tiles, `passes` times; producer w of the CTA takes the column blocks w, w + producers, ...
struct StreamTmaParams {
    CUtensorMap map;
    int n_tiles, box_rows, passes, stages, producers;
    uint32_t chunk;
    int *status;
};
constexpr int kStreamK = 8192;
__global__ void __launch_bounds__(32 * kStreamMaxProducers) k_stream_tma(const __grid_constant__ StreamTmaParams p)
{
    extern __shared__ uint8_t stream_smem_raw[];
    uint8_t *ring0 = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(stream_smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t bars[kStreamMaxProducers][kStreamMaxStages];
    if ((threadIdx.x & 31) != 0)
        return;
    const int w = threadIdx.x >> 5;
    uint8_t *ring = ring0 + (size_t)w * p.stages * p.chunk;
    for (int i = 0; i < p.stages; ++i)
        mbar_init(&bars[w][i], 1);
    mbar_fence_init();
    const int row0 = (int)(blockIdx.x % p.n_tiles) * p.box_rows;
    const int kblocks = kStreamK / 64;
    const int mine = (kblocks - w + p.producers - 1) / p.producers;      // column blocks of this producer per pass
    const size_t total = (size_t)mine * p.passes;
    for (size_t i = 0; i < total + p.stages; ++i) {
        const int st = (int)(i % p.stages);
        if (i >= (size_t)p.stages) {
            const uint32_t ph = (uint32_t)((i / p.stages - 1) & 1);
            if (!mbar_wait(&bars[w][st], ph, p.status, ST_TIMEOUT_FULL))
                return;
        }
        if (i < total) {
            const int kb = w + (int)(i % mine) * p.producers;
            mbar_expect_tx(&bars[w][st], p.chunk);
            tma_load_2d(ring + (size_t)st * p.chunk, &p.map, kb * 64, row0, &bars[w][st]);
        }
    }
}

}  // namespace prsv

extern "C" int preserve_measure_stream_tma(const void *device_buffer, size_t bytes, int32_t passes, int32_t ctas,
                                           int32_t stages, int32_t box_rows, int32_t producers, int32_t *status_block,
                                           void *cuda_stream, float *gbs_out)
{
    using namespace prsv;
    if (!device_buffer || !gbs_out || !status_block || passes < 1 || passes > 100000 || ctas < 1 || ctas > 4096 ||
        (reinterpret_cast<uintptr_t>(device_buffer) & 127) || stages < 1 || stages > kStreamMaxStages ||
        producers < 1 || producers > kStreamMaxProducers || box_rows < 8 || box_rows > 256 || box_rows % 8 ||
        (size_t)stages * box_rows * 128 * producers > 200 * 1024)
        return PRESERVE_EINVAL;
    const size_t n_rows = bytes / ((size_t)kStreamK * 2);
    StreamTmaParams p = {};
    p.n_tiles = (int)(n_rows / box_rows);
    if (p.n_tiles < 1)
        return PRESERVE_EINVAL;
    if (!encode_bf16_map_2d(&p.map, device_buffer, kStreamK, n_rows, 64, (uint32_t)box_rows))
        return PRESERVE_EARCH;
    p.box_rows = box_rows;
    p.stages = stages;
    p.producers = producers;
    p.chunk = (uint32_t)box_rows * 128u;
    p.status = status_block;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t smem = (size_t)stages * p.chunk * producers + 1024;
    static PerDeviceSize lim;
    if (ensure_dynamic_smem(k_stream_tma, lim, smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    StreamTmaParams q = p;
    q.passes = 1;
    k_stream_tma<<<ctas, 32 * producers, smem, s>>>(q);
    cudaEventRecord(e0, s);
    p.passes = passes;
    k_stream_tma<<<ctas, 32 * producers, smem, s>>>(p);
    cudaEventRecord(e1, s);
    cudaError_t err = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (err == cudaSuccess)
        err = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (err != cudaSuccess || ms <= 0.f) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    *gbs_out = (float)((double)box_rows * kStreamK * 2.0 * ctas * passes / (ms * 1e-3) / 1e9);
    return PRESERVE_OK;
}

extern "C" int preserve_measure_stream(const void *device_buffer, size_t bytes, int32_t passes, int32_t path,
                                       int32_t ctas, int32_t stages, uint32_t chunk_bytes, int32_t producers,
                                       int32_t *status_block, void *cuda_stream, float *gbs_out)
{
    using namespace prsv;
    if (!device_buffer || !gbs_out || !status_block || passes < 1 || passes > 100000 || ctas < 1 || ctas > 4096 ||
        (path < 0 || path > 2) || (reinterpret_cast<uintptr_t>(device_buffer) & 127))
        return PRESERVE_EINVAL;
    if (path >= 1 && (stages < 1 || stages > kStreamMaxStages || chunk_bytes < 1024 || chunk_bytes % 1024 ||
                      producers < 1 || producers > kStreamMaxProducers ||
                      (size_t)stages * chunk_bytes * producers > 200 * 1024))
        return PRESERVE_EINVAL;
    const uint32_t chunk = path >= 1 ? chunk_bytes : 4096u;
    const size_t unit = (size_t)chunk * (path >= 1 ? producers : 1);
    StreamParams p = {};
    p.buf = static_cast<const uint8_t *>(device_buffer);
    p.producers = path >= 1 ? producers : 1;
    p.same_warp = path == 2;
    p.slice = bytes / (size_t)ctas / unit * unit;
    if (p.slice == 0)
        return PRESERVE_EINVAL;
    p.passes = passes;
    p.chunk = chunk;
    p.stages = stages;
    p.status = status_block;
    p.sink = nullptr;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t smem = path >= 1 ? (size_t)stages * chunk * producers + 128 : 0;
    if (path >= 1) {
        static PerDeviceSize lim;
        if (ensure_dynamic_smem(k_stream_bulk, lim, smem) != cudaSuccess) {
            (void)cudaGetLastError();
            return PRESERVE_ECUDA;
        }
    }
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    auto launch = [&](int n_pass) {
        StreamParams q = p;
        q.passes = n_pass;
        if (path == 0)
            k_stream_ld<<<ctas, 256, 0, s>>>(q);
        else
            k_stream_bulk<<<ctas, 32 * producers, smem, s>>>(q);
    };
    launch(1);                      // warm-up: brings a small buffer into L2, pages in the code
    cudaEventRecord(e0, s);
    launch(passes);
    cudaEventRecord(e1, s);
    cudaError_t err = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (err == cudaSuccess)
        err = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (err != cudaSuccess || ms <= 0.f) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    *gbs_out = (float)((double)p.slice * ctas * passes / (ms * 1e-3) / 1e9);
    return PRESERVE_OK;
}

extern "C" int preserve_measure_read_bandwidth(const void *device_buffer, size_t bytes, int32_t reps,
                                               void *cuda_stream, float *gbs_out)
{
    using namespace prsv;
    if (!device_buffer || !gbs_out || bytes < (1u << 20) || reps < 1 || reps > 1000 ||
        (reinterpret_cast<uintptr_t>(device_buffer) & 15))
        return PRESERVE_EINVAL;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
        (void)cudaGetLastError();
        return PRESERVE_EARCH;
    }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    const size_t n_vec = bytes / 16;
    const uint4 *p = static_cast<const uint4 *>(device_buffer);
    k_stream_read<<<sms * 4, 512, 0, s>>>(p, n_vec, nullptr);      // warm-up (and fills L2 for small buffers)
    cudaEventRecord(e0, s);
    for (int r = 0; r < reps; ++r)
        k_stream_read<<<sms * 4, 512, 0, s>>>(p, n_vec, nullptr);
    cudaEventRecord(e1, s);
    cudaError_t err = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (err == cudaSuccess)
        err = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (err != cudaSuccess || ms <= 0.f) {
        (void)cudaGetLastError();
        return PRESERVE_ECUDA;
    }
    *gbs_out = (float)((double)n_vec * 16.0 * reps / (ms * 1e-3) / 1e9);
    return PRESERVE_OK;
}
