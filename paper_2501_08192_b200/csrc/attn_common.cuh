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

// Work split.  The 64-key tiles of all (sequence, kv head) streams, in cache order, form one line
// of T tiles; CTA c of g takes the tiles [floor(c T / g), floor((c + 1) T / g)), so every CTA
// streams the same number of tiles up to one, whatever the mix of sequence lengths.  Where a CTA's
// range crosses from one stream into the next it is cut there: each piece (a "segment") yields one
// partial result.  Segment ids are c + stream index: along the line either c or the stream index
// grows from one segment to the next, so the ids are distinct, they are contiguous within a
// stream, and none exceeds g + streams - 2, independent of the sequence lengths.
//
// tile_base[i] = first tile of stream i on that line (tile_base[streams] = T), computed identically
// by every CTA: the lengths are fetched by all threads at once (one memory round trip), then warp 0
// scans them.
template <typename Params>
__device__ __forceinline__ void build_tile_table(const Params &p, int *tile_base)
{
    const int streams = p.B * p.nkv;
    for (int i = threadIdx.x; i < streams; i += blockDim.x)
        tile_base[i + 1] = tiles_of(p.ctx_len[i / p.nkv]);
    __syncthreads();
    if (threadIdx.x < 32) {
        int carry = 0;
        for (int base = 0; base < streams; base += 32) {
            const int i = base + threadIdx.x;
            int v = i < streams ? tile_base[i + 1] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, v, o);
                if ((int)threadIdx.x >= o)
                    v += n;
            }
            if (i < streams)
                tile_base[i + 1] = carry + v;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
        if (threadIdx.x == 0)
            tile_base[0] = 0;
    }
}

__device__ __forceinline__ int find_stream(const int *tile_base, int streams, int tile)
{
    int lo = 0, hi = streams;     // tile_base[lo] <= tile < tile_base[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (tile_base[mid] <= tile) lo = mid; else hi = mid;
    }
    return lo;
}

// First tile of CTA c's range, and the CTA whose range holds tile x (T > 0).
__host__ __device__ __forceinline__ int cta_first_tile(int c, int g, int T)
{
    return (int)((long long)c * T / g);
}
__host__ __device__ __forceinline__ int cta_of_tile(int x, int g, int T)
{
    return (int)((((long long)x + 1) * g - 1) / T);
}

// One piece of a CTA's tile range inside one stream.
struct Segment {
    int sidx;       // stream = sequence * nkv + kv head
    int t0, t1;     // tiles [t0, t1) of that stream
    int id;         // index of the partial result
    int pieces;     // segments the whole stream is cut into (1: this one is the whole stream)
};
// The segment of CTA `cta` that starts at line position x (< hi); advances x to the segment's end.
__device__ __forceinline__ Segment next_segment(const int *tile_base, int streams, int g, int cta, int hi, int &x)
{
    Segment sg;
    sg.sidx = find_stream(tile_base, streams, x);
    const int first = tile_base[sg.sidx], end = tile_base[sg.sidx + 1];
    sg.t0 = x - first;
    sg.t1 = min(end, hi) - first;
    sg.id = cta + sg.sidx;
    const int T = tile_base[streams];
    sg.pieces = cta_of_tile(end - 1, g, T) - cta_of_tile(first, g, T) + 1;
    x = first + sg.t1;
    return sg;
}

}  // namespace prsv
