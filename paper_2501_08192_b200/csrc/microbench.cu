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

}  // namespace prsv

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
