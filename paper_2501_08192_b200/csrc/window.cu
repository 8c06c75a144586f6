// Communication-window stand-in: what the allreduce plus its epilogue would
// deliver on a tensor-parallel system (Section 2, "Multi-device inference";
// Section 3, "Vanilla execution"): h = residual + sum of the P partial-sum
// buffers, then x = RMSNorm(h) * gain.  One cluster of up to 8 CTAs per token
// row, each CTA a slice of the row with one thread per 8 elements: the P + 1
// 128-bit loads of a thread are all in flight together, and a row's bytes are
// requested by many warps on several SMs (the same bytes requested by the few
// warps of one SM take several times longer).  The slices' sums of squares meet
// by one-sided stores into each peer's shared memory and are added in rank order.  fp32
// accumulation in the fixed order residual, part 0..P-1 (part 0 may be fp32: this
// shard's own result, or the previous layer's in a chain).
// Loads of buffers that are inputs of the step are issued before the
// programmatic-dependent-launch wait; only what an earlier kernel of the step
// produces (this shard's own partial sum, the fp32 residual) is read after it.
// The kernel stays narrow (at most 8 B small CTAs): during a real allreduce the
// SMs idle, which is what leaves HBM bandwidth to the prefetch stream.
#include <cooperative_groups.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "kernels.h"

namespace cg = cooperative_groups;

namespace prsv {

constexpr int kWinMaxChunks = 2;   // 8-element chunks per thread
constexpr int kWinMaxCluster = 8;  // CTAs per row

struct WindowParams {
    const uint4 *parts[kMaxParts];
    int n_parts;
    const void *resid;
    const uint4 *gain;
    float eps;
    float *h_f32;
    uint4 *h_bf16;
    uint4 *x_bf16;       // hi plane; the lo plane follows at x_plane uint4s
    size_t x_plane;
    int H;
    int cluster;         // CTAs per row
    int resid_f32, part0_f32;   // the residual / partial 0 are fp32 (handed over by an earlier kernel of the step)
    long long *trace;
    int delay_ns;
    int *status;
    int x_fp16;          // 0: x as bf16 hi + lo planes; 1: one fp16 plane; 2: fp16 hi + lo planes (x = hi + lo, 22 bits)
    int no_hint;         // LEAN: do not even hint the inputs into L2 before the wait (another kernel of the call still writes them)
    int inject;          // test hook: rank 1 of every row withholds its hand-over to rank 0
    // real communication window (COMM instantiation only)
    int comm_rank, comm_window;
    const uint32_t *comm_flags_local;
    uint32_t *comm_flags_peer[kMaxParts];
    uint32_t *comm_epoch;
    unsigned *comm_done;
};

// Loads and stores of the arrival protocol between GPUs (system scope).
__device__ __forceinline__ uint32_t ld_acquire_sys(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_sys(uint32_t *p, uint32_t v)
{
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// 128-bit load that is performed at the memory it names every time (a peer's buffer changes from
// step to step and must never be served from a stale line of this GPU's caches).
__device__ __forceinline__ uint4 ld_volatile_v4(const void *p)
{
    uint4 r;
    asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p)
                 : "memory");
    return r;
}

// (One instantiation for all four input forms: the two windows of a layer then run the same
// instructions, which the second finds in the instruction caches.)
// LEAN, for big batches (hundreds of CTAs): one chunk per thread and the step's input buffers are only
// hinted into L2 before the wait and loaded after it, so that a CTA holds few registers while it
// waits - the grid then fits beside the early-launched GEMM CTAs in one wave instead of several.
// COMM: the real communication window - the partial-sum buffers are the ranks' exchange buffers
// (one-shot all-reduce: every rank reads every rank's buffer through peer-mapped pointers with plain
// 128-bit loads and adds them in rank order, so all ranks obtain the same bits).  Arrival protocol,
// all in this kernel: after the dependency wait (own buffer complete) CTA 0 stores this window's
// epoch number into every peer's flag block (release, system scope); every CTA then polls its own
// GPU's flag block until all peers' entries have reached the epoch (acquire, system scope; bounded -
// a peer that never arrives makes the wait give up with a status code, the kernel still returns).
// The epoch is a device counter that the last CTA of the launch advances, so a replayed graph
// needs no new arguments.  Buffers are reused window after window: a rank overwrites its window-A
// buffer only after it has passed window B of the same layer, by which time every peer has
// announced its window-B buffer and therefore finished reading window A.
template <bool LEAN, bool COMM = false>
__global__ void __launch_bounds__(512) k_window_reduce_rmsnorm(const __grid_constant__ WindowParams p)
{
    constexpr int kWinMaxChunks = LEAN ? 1 : prsv::kWinMaxChunks;
    const bool RESID_F32 = p.resid_f32 != 0, PART0_F32 = p.part0_f32 != 0;
    const int row = blockIdx.x / p.cluster, rank = blockIdx.x % p.cluster;
    const int chunks = (p.H >> 3) / p.cluster;   // uint4 chunks of this CTA's slice of the row
    const size_t row_off = (size_t)row * (p.H >> 3) + (size_t)rank * chunks;
    const int gain_off = rank * chunks;
    float v[kWinMaxChunks][8];
    uint4 gn[kWinMaxChunks];
    float ss = 0.f;

    // the gain does not depend on the previous kernel: fetch it before waiting
#pragma unroll
    for (int c = 0; c < kWinMaxChunks; ++c) {
        const int ch = threadIdx.x + c * blockDim.x;
        gn[c] = ch < chunks ? ld_cached(p.gain + gain_off + ch) : make_uint4(0, 0, 0, 0);
    }

    trace_start(p.trace);
    pdl_launch_dependents();   // the next kernel may start fetching its weights now

    // The slices' sums of squares are handed over one-sidedly: every CTA of the row stores its sum
    // into each peer's recv[] slot, signalling the peer's barrier.  The barriers must exist before
    // anybody sends: one cluster barrier here, long before the data it guards.
    __shared__ uint64_t recv_bar;
    __shared__ float recv[kWinMaxCluster];
    if (p.cluster > 1) {
        if (threadIdx.x == 0) {
            mbar_init(&recv_bar, 1);
            mbar_fence_init();
            mbar_expect_tx(&recv_bar, (uint32_t)(p.cluster - 1) * 4u);
        }
    }

    // Buffers that are inputs of the step (the peers' partial sums, and the residual / partial 0
    // unless they are handed over in fp32 by an earlier kernel of the step) do not depend on the
    // previous kernel either: their loads - the only ones that go to HBM - are issued before the
    // wait, up to 8 partial buffers per chunk.
    uint4 pre[kWinMaxChunks][8], pre_res[kWinMaxChunks];
    auto load_inputs = [&]() {
#pragma unroll
        for (int c = 0; c < kWinMaxChunks; ++c) {
            const int ch = threadIdx.x + c * blockDim.x;
            if (ch < chunks) {
                if (!RESID_F32)
                    pre_res[c] = ld_stream(reinterpret_cast<const uint4 *>(p.resid) + row_off + ch);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (j < p.n_parts && !(PART0_F32 && j == 0))
                        pre[c][j] = COMM ? ld_volatile_v4(p.parts[j] + row_off + ch) : ld_stream(p.parts[j] + row_off + ch);
            }
        }
    };
    if constexpr (LEAN && !COMM) {
        // one hint per 128-byte line (8 threads share a line)
        if (!p.no_hint && (threadIdx.x & 7) == 0 && (int)threadIdx.x < chunks) {
            if (!RESID_F32)
                line_prefetch_l2(reinterpret_cast<const uint4 *>(p.resid) + row_off + threadIdx.x);
            for (int j = 0; j < p.n_parts; ++j)
                if (!(PART0_F32 && j == 0))
                    line_prefetch_l2(p.parts[j] + row_off + threadIdx.x);
        }
    } else if constexpr (!LEAN) {
        load_inputs();
    }

    if (p.cluster > 1)
        cg::this_cluster().sync();      // (the loads above are in flight meanwhile)

    pdl_wait();                // this shard's own partial sum comes from the preceding kernel in the stream
    trace_waited(p.trace);
    const long long t_begin = p.delay_ns ? gtime() : 0;   // the modelled collective starts when its inputs exist
    if constexpr (COMM) {
        __shared__ uint32_t epoch_s;
        if (threadIdx.x == 0)
            epoch_s = *reinterpret_cast<volatile uint32_t *>(p.comm_epoch) + 1u;
        __syncthreads();
        const uint32_t epoch = epoch_s;
        const int t = threadIdx.x;
        if (t < p.n_parts && t != p.comm_rank) {
            if (blockIdx.x == 0) {
                __threadfence_system();          // own buffer (written by the kernel before) before the flag
                st_release_sys(p.comm_flags_peer[t] + p.comm_window * kMaxParts + p.comm_rank, epoch);
            }
            const uint32_t *flag = p.comm_flags_local + p.comm_window * kMaxParts + t;
            const long long t0 = clock64();
            long long limit = kFastWaitCycles;
            bool arrived = false, asked = false;
            for (;;) {
                if ((int32_t)(ld_acquire_sys(flag) - epoch) >= 0) { arrived = true; break; }
                if (clock64() - t0 >= limit) {
                    if (asked)
                        break;
                    limit = *reinterpret_cast<volatile long long *>(p.status + kStatusLimitWord);
                    if (limit <= 0 || limit > kMaxWaitCycles)
                        limit = kMaxWaitCycles;
                    asked = true;
                }
            }
            if (!arrived)
                atomicCAS(p.status, ST_OK, ST_TIMEOUT_PEER);
        }
        __syncthreads();
    }
    if constexpr (LEAN)
        load_inputs();

#pragma unroll
    for (int c = 0; c < kWinMaxChunks; ++c) {
        const int ch = threadIdx.x + c * blockDim.x;
        if (ch < chunks) {
            if (RESID_F32) {
                const float4 *r = reinterpret_cast<const float4 *>(p.resid) + (row_off + ch) * 2;
                float4 a = r[0], b = r[1];
                v[c][0] = a.x; v[c][1] = a.y; v[c][2] = a.z; v[c][3] = a.w;
                v[c][4] = b.x; v[c][5] = b.y; v[c][6] = b.z; v[c][7] = b.w;
            } else {
                const uint4 r = pre_res[c];
                v[c][0] = bf_lo(r.x); v[c][1] = bf_hi(r.x); v[c][2] = bf_lo(r.y); v[c][3] = bf_hi(r.y);
                v[c][4] = bf_lo(r.z); v[c][5] = bf_hi(r.z); v[c][6] = bf_lo(r.w); v[c][7] = bf_hi(r.w);
            }
            if (PART0_F32) {     // partial 0 handed over in fp32 (own result / previous layer of a chain)
                const float4 *r = reinterpret_cast<const float4 *>(p.parts[0]) + (row_off + ch) * 2;
                float4 a = r[0], b = r[1];
                v[c][0] += a.x; v[c][1] += a.y; v[c][2] += a.z; v[c][3] += a.w;
                v[c][4] += b.x; v[c][5] += b.y; v[c][6] += b.z; v[c][7] += b.w;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (j < p.n_parts && !(PART0_F32 && j == 0)) {
                    const uint4 r = pre[c][j];
                    v[c][0] += bf_lo(r.x); v[c][1] += bf_hi(r.x); v[c][2] += bf_lo(r.y); v[c][3] += bf_hi(r.y);
                    v[c][4] += bf_lo(r.z); v[c][5] += bf_hi(r.z); v[c][6] += bf_lo(r.w); v[c][7] += bf_hi(r.w);
                }
            // (more than 8 partial buffers: the rest in bursts of 8)
            for (int q0 = 8; q0 < p.n_parts; q0 += 8) {
                uint4 r[8];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (q0 + j < p.n_parts)
                        r[j] = ld_stream(p.parts[q0 + j] + row_off + ch);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (q0 + j < p.n_parts) {
                        v[c][0] += bf_lo(r[j].x); v[c][1] += bf_hi(r[j].x); v[c][2] += bf_lo(r[j].y); v[c][3] += bf_hi(r[j].y);
                        v[c][4] += bf_lo(r[j].z); v[c][5] += bf_hi(r[j].z); v[c][6] += bf_lo(r[j].w); v[c][7] += bf_hi(r[j].w);
                    }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i)
                ss += v[c][i] * v[c][i];
        }
    }

    // block reduction of the sum of squares (fixed tree: bit-stable run to run)
    __shared__ float warp_sums[32];
    __shared__ float total;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0)
        warp_sums[warp] = ss;
    __syncthreads();
    if (warp == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        float t = lane < nw ? warp_sums[lane] : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
            t += __shfl_xor_sync(0xffffffffu, t, o);      // every lane holds the CTA's sum
        if (lane == 0)
            total = t;
        if (p.cluster > 1 && lane < p.cluster) {
            if (lane == rank)
                recv[rank] = t;
            else if (!(p.inject == INJECT_WINDOW_HANDOVER && rank == 1 && lane == 0))
                st_async_f32(cluster_map(&recv[rank], lane), t, cluster_map(&recv_bar, lane));
        }
    }
    __syncthreads();
    float row_total = total;
    bool recv_short = false;     // the wait for the other CTAs' sums ran out
    if (p.cluster > 1) {
        // sum of the slices in rank order (the same order in every CTA of the row)
        row_total = 0.f;
        recv_short = !mbar_wait(&recv_bar, 0, p.status, ST_TIMEOUT_FULL);
        if (!recv_short)
            for (int q = 0; q < p.cluster; ++q)
                row_total += recv[q];
    }
    const float inv = rsqrtf(row_total / (float)p.H + p.eps);

    // modelled network time of the allreduce this kernel stands in for: hold the result back until
    // delay_ns after its inputs were complete (bounded by the delay itself)
    if (p.delay_ns) {
        while (gtime() - t_begin < (long long)p.delay_ns) {
            __nanosleep(200);
        }
    }

#pragma unroll
    for (int c = 0; c < kWinMaxChunks; ++c) {
        const int ch = threadIdx.x + c * blockDim.x;
        if (ch < chunks) {
            if (p.h_f32) {
                float4 *o = reinterpret_cast<float4 *>(p.h_f32) + (row_off + ch) * 2;
                o[0] = make_float4(v[c][0], v[c][1], v[c][2], v[c][3]);
                o[1] = make_float4(v[c][4], v[c][5], v[c][6], v[c][7]);
            }
            if (p.h_bf16) {
                uint4 o;
                o.x = pack_bf16(v[c][0], v[c][1]); o.y = pack_bf16(v[c][2], v[c][3]);
                o.z = pack_bf16(v[c][4], v[c][5]); o.w = pack_bf16(v[c][6], v[c][7]);
                p.h_bf16[row_off + ch] = o;
            }
            // x is kept as a pair of bf16 planes, x = hi + lo, so the GEMM that consumes it
            // sees ~16 mantissa bits although its operands are bf16
            const uint4 g = gn[c];
            float xv[8];
            xv[0] = v[c][0] * inv * bf_lo(g.x); xv[1] = v[c][1] * inv * bf_hi(g.x);
            xv[2] = v[c][2] * inv * bf_lo(g.y); xv[3] = v[c][3] * inv * bf_hi(g.y);
            xv[4] = v[c][4] * inv * bf_lo(g.z); xv[5] = v[c][5] * inv * bf_hi(g.z);
            xv[6] = v[c][6] * inv * bf_lo(g.w); xv[7] = v[c][7] * inv * bf_hi(g.w);
            if (p.x_fp16 == 2) {
                // hi = fp16(x), lo = fp16(x - hi): the operand format of the tensor path's QKV projection
                uint4 hi, lo;
                uint32_t *hw = &hi.x, *lw = &lo.x;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float a0 = fminf(fmaxf(xv[2 * i], -65504.f), 65504.f);
                    const float a1 = fminf(fmaxf(xv[2 * i + 1], -65504.f), 65504.f);
                    const __half2 h2 = __floats2half2_rn(a0, a1);
                    const float2 hf = __half22float2(h2);
                    const __half2 l2 = __floats2half2_rn(a0 - hf.x, a1 - hf.y);
                    hw[i] = *reinterpret_cast<const uint32_t *>(&h2);
                    lw[i] = *reinterpret_cast<const uint32_t *>(&l2);
                }
                p.x_bf16[row_off + ch] = hi;
                p.x_bf16[p.x_plane + row_off + ch] = lo;
            } else if (p.x_fp16) {
                // normalised activations are bounded (|x| <= sqrt(H) * |gain|): one fp16 plane carries 11
                // significant bits; clamped to the fp16 range so that an absurd gain cannot make an infinity
                uint4 o;
                uint32_t *ow = &o.x;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const __half2 h2 = __floats2half2_rn(fminf(fmaxf(xv[2 * i], -65504.f), 65504.f),
                                                         fminf(fmaxf(xv[2 * i + 1], -65504.f), 65504.f));
                    ow[i] = *reinterpret_cast<const uint32_t *>(&h2);
                }
                p.x_bf16[row_off + ch] = o;
            } else {
                uint4 hi, lo;
                split_bf16x2(xv[0], xv[1], hi.x, lo.x);
                split_bf16x2(xv[2], xv[3], hi.y, lo.y);
                split_bf16x2(xv[4], xv[5], hi.z, lo.z);
                split_bf16x2(xv[6], xv[7], hi.w, lo.w);
                p.x_bf16[row_off + ch] = hi;
                p.x_bf16[p.x_plane + row_off + ch] = lo;
            }
        }
    }
    if constexpr (COMM) {
        // the last CTA of the launch to get here advances this window's epoch
        __syncthreads();
        if (threadIdx.x == 0) {
            const unsigned ticket = atomicAdd(p.comm_done, 1u);
            if (ticket == gridDim.x - 1) {
                *p.comm_done = 0u;
                __threadfence();
                atomicAdd(p.comm_epoch, 1u);
            }
        }
    }
    if (p.cluster > 1) {
        // This CTA gave up waiting for a peer's sum: the peer may still store it into this CTA's shared
        // memory, and a store into a CTA that has exited is a fault.  Stay until every peer has left or
        // reached this point too (its stores were issued before), then give the stores in flight a
        // bounded time to land.  (The barrier counts only threads that have not exited; a CTA whose wait
        // succeeded has received everything and simply leaves.)
        if (__syncthreads_or(recv_short ? 1 : 0)) {
            cluster_arrive_relaxed();
            cluster_wait();
            if (threadIdx.x == 0)
                mbar_wait(&recv_bar, 0, p.status, ST_TIMEOUT_FULL);
            __syncthreads();
        }
    }
    trace_end(p.trace);
}

cudaError_t launch_window(const WindowArgs &a, cudaStream_t s)
{
    WindowParams p;
    for (int i = 0; i < kMaxParts; ++i)
        p.parts[i] = i < a.n_parts ? reinterpret_cast<const uint4 *>(a.parts[i]) : nullptr;
    p.n_parts = a.n_parts;
    p.resid = a.resid;
    p.gain = reinterpret_cast<const uint4 *>(a.gain);
    p.eps = a.eps;
    p.h_f32 = a.h_f32;
    p.h_bf16 = reinterpret_cast<uint4 *>(a.h_bf16);
    p.x_bf16 = reinterpret_cast<uint4 *>(a.x_bf16);
    p.x_plane = a.x_plane_elems / 8;
    p.H = a.H;
    p.trace = a.trace;
    p.delay_ns = a.delay_ns;
    p.status = a.status;
    // CTAs per row: as many (a power of two, at most 8) as leave every CTA at least 128 threads of
    // one 8-element chunk each
    int cl = 1;
    while (cl < kWinMaxCluster && (a.H / 8) % (cl * 2) == 0 && (a.H / 8) / (cl * 2) >= 128)
        cl *= 2;
    p.cluster = cl;
    const int chunks = a.H / 8 / cl;
    // LEAN (inputs read after the wait) for big batches, and whenever an input buffer may still be
    // written by an earlier kernel of the same call
    const bool comm = a.comm_rank >= 0;
    const bool lean = (a.B * cl > 256 || a.inputs_after_wait || comm) && chunks <= 512;
    if ((a.inputs_after_wait || comm) && !lean)
        return cudaErrorInvalidValue;
    if (comm && (a.n_parts > 8 || a.part0_is_f32 || a.comm_rank >= a.n_parts))
        return cudaErrorInvalidValue;
    p.no_hint = a.inputs_after_wait;
    p.x_fp16 = a.x_fp16;
    p.inject = a.inject;
    p.comm_rank = a.comm_rank;
    p.comm_window = a.comm_window;
    p.comm_flags_local = a.comm_flags_local;
    for (int i = 0; i < kMaxParts; ++i)
        p.comm_flags_peer[i] = a.comm_flags_peer[i];
    p.comm_epoch = a.comm_epoch;
    p.comm_done = a.comm_done;
    int threads = (chunks + kWinMaxChunks - 1) / kWinMaxChunks;
    if (chunks <= 512)
        threads = chunks;
    threads = ((threads + 31) / 32) * 32;
    if (threads > 512 || threads * kWinMaxChunks < chunks)
        return cudaErrorInvalidValue;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.B * cl);
    cfg.blockDim = dim3(threads);
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    cfg.attrs = at;
    int n_attr = pdl_attr(at, a.pdl);
    if (cl > 1) {
        at[n_attr].id = cudaLaunchAttributeClusterDimension;
        at[n_attr].val.clusterDim.x = cl;
        at[n_attr].val.clusterDim.y = 1;
        at[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    cfg.numAttrs = n_attr;
    p.resid_f32 = a.resid_is_f32;
    p.part0_f32 = a.part0_is_f32;
    if (comm)
        return cudaLaunchKernelEx(&cfg, k_window_reduce_rmsnorm<true, true>, p);
    return lean ? cudaLaunchKernelEx(&cfg, k_window_reduce_rmsnorm<true, false>, p)
                : cudaLaunchKernelEx(&cfg, k_window_reduce_rmsnorm<false, false>, p);
}

}  // namespace prsv
