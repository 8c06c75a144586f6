// Pieces shared by the split-KV decode-attention kernels (bf16 cache and int8 cache): the tiling
// constants, the work-item table every CTA builds from the sequence lengths, and the named barrier
// of the consumer warps.
#pragma once
#include "common.cuh"

namespace prsv {

constexpr int kTileKeys = 64;
constexpr int kConsumerWarps = 4;
constexpr int kAttnThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxStreams = 2048;                      // (sequence, kv head) pairs per launch

__device__ __forceinline__ void consumer_barrier()
{
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
}

__device__ __forceinline__ int tiles_of(int ctx) { return (ctx + 1 + kTileKeys - 1) / kTileKeys; }

// First item index of every stream, computed identically by every CTA: the lengths are
// fetched by all threads at once (one memory round trip), then warp 0 scans them.
template <typename Params>
__device__ __forceinline__ void build_item_table(const Params &p, int *item_base)
{
    const int streams = p.B * p.nkv;
    for (int i = threadIdx.x; i < streams; i += blockDim.x) {
        const int nt = tiles_of(p.ctx_len[i / p.nkv]);
        item_base[i + 1] = (nt + p.tiles_per_item - 1) / p.tiles_per_item;
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        int carry = 0;
        for (int base = 0; base < streams; base += 32) {
            const int i = base + threadIdx.x;
            int v = i < streams ? item_base[i + 1] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, v, o);
                if ((int)threadIdx.x >= o)
                    v += n;
            }
            if (i < streams)
                item_base[i + 1] = carry + v;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
        if (threadIdx.x == 0)
            item_base[0] = 0;
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

}  // namespace prsv
