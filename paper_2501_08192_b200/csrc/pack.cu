// Weight packing, run once at layer creation.  Sources are the caller's
// [in, out] row-major matrices; destinations are laid out so that the GEMM
// kernels stream them in address order with perfectly coalesced loads.
//
// GEMV path ("fragment-major"): the matrix is cut into tiles of 16 output rows
// x 32 k; tile (rb, kc) occupies 1 KiB at ((rb * K/32) + kc) * 1024.  Inside a
// tile lane L = 4g + t owns 32 contiguous bytes: 16 B of row g (k = 8t..8t+7)
// then 16 B of row g + 8 (same k), which is exactly the A-operand fragment of two
// m16n8k16 MMAs (up to a permutation of k shared with the activations).
//
// Tensor path: plain [N, K] K-major rows (the tcgen05 A operand, fetched by TMA
// with a 128-byte swizzle).
#include <cuda_fp16.h>

#include "epilogue.cuh"

namespace prsv {

struct PackParams {
    const bf16 *src[3];
    int cols[3];
    int n_srcs;
    int N, K, kind;
    int to_fp16;      // store the weights as fp16 (tensor path, matrices whose activations are one fp16 plane)
    bf16 *dst;
};

template <bool TENSOR>
__global__ void k_pack(const __grid_constant__ PackParams p)
{
    // one thread per (k, packed row); packed rows fastest so source reads coalesce
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t total = (size_t)p.N * p.K;
    if (idx >= total)
        return;
    const int row = (int)(idx % p.N);
    const int k = (int)(idx / p.N);
    int src, col;
    packed_row_source(p.kind, TENSOR, row, p.cols, src, col);
    const bf16 v = p.src[src][(size_t)k * p.cols[src] + col];
    size_t o;
    if (TENSOR) {
        o = (size_t)row * p.K + k;
    } else {
        const int rb = row >> 4, r = row & 15, g = r & 7, hi = r >> 3;
        const int kc = k >> 5, t = (k & 31) >> 3, e = k & 7;
        o = ((size_t)rb * (p.K >> 5) + kc) * 512 + (size_t)(g * 4 + t) * 16 + hi * 8 + e;
    }
    if (p.to_fp16) {
        // Both operands of a tcgen05 kind::f16 MMA must have the same 16-bit format, so a matrix that is
        // multiplied with fp16 activations is stored as fp16: exact for every bf16 weight of magnitude
        // 2^-17 .. 65504 (fp16 has the longer mantissa); smaller ones round to a multiple of 2^-24 (error
        // <= 2^-25, far below one bf16 ulp of any output), larger ones saturate
        const float f = fminf(fmaxf(__bfloat162float(v), -65504.f), 65504.f);
        reinterpret_cast<__half *>(p.dst)[o] = __float2half_rn(f);
    } else {
        p.dst[o] = v;
    }
}

static cudaError_t launch_pack(bool tensor, const void *const *srcs, const int *src_cols, int n_srcs, int K,
                               int kind, void *dst, int to_fp16, cudaStream_t s)
{
    PackParams p = {};
    int N = 0;
    for (int i = 0; i < n_srcs; ++i) {
        p.src[i] = reinterpret_cast<const bf16 *>(srcs[i]);
        p.cols[i] = src_cols[i];
        N += src_cols[i];
    }
    p.n_srcs = n_srcs;
    p.N = N;
    p.K = K;
    p.kind = kind;
    p.to_fp16 = to_fp16;
    p.dst = reinterpret_cast<bf16 *>(dst);
    const size_t total = (size_t)N * K;
    const int threads = 256;
    const unsigned blocks = (unsigned)((total + threads - 1) / threads);
    if (tensor)
        k_pack<true><<<blocks, threads, 0, s>>>(p);
    else
        k_pack<false><<<blocks, threads, 0, s>>>(p);
    return cudaGetLastError();
}

// ---- int8 weights (GEMV path: fragment-major tiles; tensor path: [N, K] K-major rows of codes)
struct PackW8Params {
    const bf16 *src[3];
    int cols[3];
    int N, K, kind;
    int tensor;       // tensor-path row order and layout: 128-row tiles per block (1 or 2), 0 = GEMV path
    int8_t *codes;
    float *scales;
};

// scale of every packed row: max |w| over the row's source column, divided by 127 (fp32)
__global__ void k_w8_scales(const __grid_constant__ PackW8Params p)
{
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= p.N)
        return;
    int src, col;
    packed_row_source(p.kind, p.tensor != 0, row, p.cols, src, col);
    float mx = 0.f;
    for (int k = 0; k < p.K; ++k)
        mx = fmaxf(mx, fabsf(__bfloat162float(p.src[src][(size_t)k * p.cols[src] + col])));
    p.scales[row] = __fdiv_rn(mx, 127.0f);
}

__global__ void k_pack_w8(const __grid_constant__ PackW8Params p)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t total = (size_t)p.N * p.K;
    if (idx >= total)
        return;
    const int row = (int)(idx % p.N);
    const int k = (int)(idx / p.N);
    int src, col;
    packed_row_source(p.kind, p.tensor != 0, row, p.cols, src, col);
    const float v = __bfloat162float(p.src[src][(size_t)k * p.cols[src] + col]);
    const float sc = p.scales[row];
    // the code is decided in fp32: one correctly rounded division, round to nearest even, clamp
    float r = sc > 0.f ? rintf(__fdiv_rn(v, sc)) : 0.f;
    r = fminf(fmaxf(r, -127.f), 127.f);
    size_t o;
    if (p.tensor) {
        // the tensor path keeps the codes biased by 128 (unsigned bytes): its widening stage then needs
        // no sign handling
        const int block_rows = p.tensor * 128;
        const size_t block = (size_t)(row / block_rows) * (p.K >> 7) + (k >> 7);
        // (the eight 16-byte groups of a row's 128 k are stored in the order q ^ (row % 8): the widening
        // warps read one group per lane, 32 consecutive rows at a time, without bank conflicts)
        const int rr = row % block_rows, kk = k & 127;
        const int grp = (kk >> 4) ^ (rr & 7);
        p.codes[(block * block_rows + rr) * 128 + grp * 16 + (kk & 15)] = (int8_t)(uint8_t)((int)r + 128);
        return;
    } else {
        const int rb = row >> 4, rr = row & 15, g = rr & 7, hi = rr >> 3;
        const int kc = k >> 6, t = (k & 63) >> 4, e = k & 15;
        o = ((size_t)rb * (p.K >> 6) + kc) * 1024 + (size_t)(g * 4 + t) * 32 + hi * 16 + e;
    }
    p.codes[o] = (int8_t)(int)r;
}

static cudaError_t launch_pack_w8(int tensor, const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind,
                                  void *dst_codes, float *dst_scales, cudaStream_t s)
{
    if (K % 64)
        return cudaErrorInvalidValue;
    PackW8Params p = {};
    int N = 0;
    for (int i = 0; i < n_srcs; ++i) {
        p.src[i] = reinterpret_cast<const bf16 *>(srcs[i]);
        p.cols[i] = src_cols[i];
        N += src_cols[i];
    }
    p.N = N; p.K = K; p.kind = kind;
    p.tensor = tensor;
    p.codes = reinterpret_cast<int8_t *>(dst_codes);
    p.scales = dst_scales;
    k_w8_scales<<<(N + 127) / 128, 128, 0, s>>>(p);
    const size_t total = (size_t)N * K;
    k_pack_w8<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_pack_gemv_w8(const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind,
                                void *dst_codes, float *dst_scales, cudaStream_t s)
{
    return launch_pack_w8(0, srcs, src_cols, n_srcs, K, kind, dst_codes, dst_scales, s);
}
cudaError_t launch_pack_rows_w8(const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind,
                                void *dst_codes, float *dst_scales, int tiles, cudaStream_t s)
{
    if ((tiles != 1 && tiles != 2) || K % 128)
        return cudaErrorInvalidValue;
    return launch_pack_w8(tiles, srcs, src_cols, n_srcs, K, kind, dst_codes, dst_scales, s);
}

cudaError_t launch_pack_gemv(const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind, void *dst,
                             int to_fp16, cudaStream_t s)
{
    (void)to_fp16;      // the GEMV path keeps bf16 weights and hi + lo bf16 activations
    return launch_pack(false, srcs, src_cols, n_srcs, K, kind, dst, 0, s);
}
cudaError_t launch_pack_rows(const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind, void *dst,
                             int to_fp16, cudaStream_t s)
{
    return launch_pack(true, srcs, src_cols, n_srcs, K, kind, dst, to_fp16, s);
}

}  // namespace prsv
