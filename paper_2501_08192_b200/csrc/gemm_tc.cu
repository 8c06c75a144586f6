// Skinny GEMM on the 5th-generation tensor cores for decode batches >= 16:
//     y[b, n] = sum_k x[b, k] * W[n, k]
// computed "swapped": the weight tile is the M = 128 operand, the batch (padded
// to a multiple of 16; present twice - the hi and the lo bf16 plane of the
// activations, x = hi + lo - or once, as one fp16 plane) is the N operand, so one tcgen05.mma per 16 k covers a
// 128 x 16-k slab of weights for every batch row at once and the CUDA cores stay
// out of the weight stream entirely.
//
// Per CTA: one 128-row tile of the packed weights (two for wide batches, sharing one activation
// tile) x one slice of k.
//   warp 0 (+ lane 0 of the first one or two epilogue warps): TMA producers - W tile (128 or 256 rows
//               x 64, 128B swizzle) and x tile (2 NB x 64) into a multi-stage shared-memory ring,
//               mbarrier full/empty.  One thread can start a bulk copy only every ~0.4 us whatever
//               its size (measured: a single issuing thread moves 43 GB/s in 16 KiB copies, 131 GB/s
//               in 64 KiB copies, and threads of different warps add up), so one producer alone caps
//               a CTA near 50-70 GB/s - below an SM's share of HBM; the ring's stage uses are
//               therefore dealt round-robin to several issuing threads
//   warp 1    : allocates TMEM, issues tcgen05.mma (kind::f16, bf16 in, fp32
//               accumulate in TMEM), tcgen05.commit frees ring slots
//   warps 2.. : epilogue (8 or 16 warps) - tcgen05.ld the accumulator (lane = output row; the warps of
//               a TMEM lane group share the column chunks), split-K reduction across the cluster as a
//               one-sided reduce-scatter in rank order (every rank finishes NB / splits columns:
//               st.async pieces for narrow batches, bulk shared-memory copies for wide ones; reads
//               through distributed shared memory only where the receive area does not fit), fused
//               epilogue (epilogue.cuh)
// The kernel is instantiated per (epilogue kind, hand-over form): the tail of one instantiation is
// a few KB of instructions, which matters for a kernel that runs for microseconds.
// int8 weights (W8 instantiations): the ring carries the codes of 128 k per stage; the epilogue warps
// that issue no copies widen them (exactly) to the activations' 16-bit format and store them into
// tensor memory (tcgen05.st), where the MMA takes them as its A operand - shared memory stays all
// ring, and nothing widened ever passes through it.  See the converter block below.
// Every mbarrier wait is bounded; a wait that gives up records a status code,
// poisons the rest of the CTA's work, and the CTA still reaches every barrier
// and frees its TMEM.
#include <cooperative_groups.h>
#include <cstdlib>
#include <type_traits>

#include "epilogue.cuh"

namespace cg = cooperative_groups;

namespace prsv {

constexpr int kTcMaxStages = 12;
constexpr int kTcMaxW8Slots = 4;          // int8 weights: widened operand tiles in tensor memory
constexpr int kTcMaxEpiWarps = 16;        // 2-4 per TMEM lane group: the epilogue is a chain of short dependent
                                          // operations per output, so its speed is set by how many warps run it
constexpr int kTcMaxProducers = 3;        // issuing threads of the TMA ring: warp 0, and lane 0 of the first epilogue warps
                                          // (which have nothing else to do until the accumulator is complete)
constexpr int kTcMaxThreads = (2 + kTcMaxEpiWarps) * 32;
constexpr int kTcBlockK = 64;
constexpr int kTcTileM = 128;
constexpr int kATileBytes = kTcTileM * kTcBlockK * 2;   // 16 KiB

struct GemmTcParams {
    CUtensorMap w_map;
    CUtensorMap x_map;
    int B, NB, N, K;
    int mt;             // 128-row weight tiles per CTA (1 or 2): two tiles share one activation tile
    int kblocks;        // K / 64 (int8 weights: K / 128 - a stage carries 128 k)
    int splits;         // cluster size along k
    int stages;
    int push;           // split-K reduction by one-sided hand-over: 1 = st.async, 2 = bulk copies (0: every rank reads all ranks)
    int recv_off;       // push: offset of the receive area behind the ring
    int tmem_cols;
    uint32_t idesc;
    EpilogueArgs epi;
    int *status;
    long long *trace;
    int inject;         // test hook: the producer of CTA (0, 0) never fetches its first weight tile
    int planes;         // activation planes in the B operand: 2 = hi + lo, 1 = a single fp16 plane
    int f16;            // both operands are fp16 (else bf16)
    int epi_warps;      // 8 or 16
    int producers;      // 1..kTcMaxProducers threads that issue the ring's TMA loads (stage uses dealt round-robin)
    int w8;             // the weight tiles arrive as int8 codes and are widened into tensor memory (the MMA's A operand)
    int w8_early;       // w8: the first ring fill's activation tiles complete their own barrier (codes widened before the wait)
    int w8_slots;       // 2..kTcMaxW8Slots widened tiles in tensor memory (mt * 32 columns each) behind the accumulators
    const float *wscale;  // w8: one fp32 scale per packed weight row
    const uint8_t *w8_codes;  // w8: the codes, one contiguous block of mt * 128 rows x 64 bytes per (tile, k-block)
};

// int8 -> 16-bit widening of two weight codes, exact.  The packed matrix holds every code biased by
// 128 (an unsigned byte), so no sign handling is left for the kernel.  SEL places the bytes: 0x4140 =
// bytes (0, 1) of the word, 0x4342 = bytes (2, 3).
// fp16: the byte lands in the mantissa of 1024.0, i.e. the number 1152 + code; subtract 1152.
// bf16 (7 mantissa bits): the low seven bits land in the mantissa of 128.0, i.e. 128 + (byte & 127);
// subtract 128 when the byte's top bit is set (code >= 0), 256 when it is not.
template <uint32_t SEL, bool F16>
__device__ __forceinline__ uint32_t widen_u8x2(uint32_t biased)
{
    uint32_t r;
    if constexpr (F16) {
        r = __byte_perm(biased, 0x64646464u, SEL);
        const uint32_t off = 0x64806480u;      // (1152.0, 1152.0)
        asm("sub.f16x2 %0, %0, %1;" : "+r"(r) : "r"(off));
    } else {
        const uint32_t w = __byte_perm(biased, 0x43434343u, SEL);
        const uint32_t minuend = w & 0xff7fff7fu, subtrahend = (w & 0x00800080u) ^ 0x43804380u;
        asm("sub.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(minuend), "r"(subtrahend));
    }
    return r;
}
// One widening pass of a converter thread over a tile: `n` tasks of 16 codes (one 16-byte load, two
// 16-byte stores); consecutive tasks of a thread are `src_step` / `dst_step` bytes apart.
// 16 codes (one 16-byte word group) widened to eight 32-bit registers: k elements 2c (low half) and
// 2c + 1 (high half) in register c - the packing of a 16-bit A operand in tensor memory.
template <bool F16>
__device__ __forceinline__ void widen16(uint4 w, uint32_t (&r)[8])
{
    r[0] = widen_u8x2<0x4140, F16>(w.x); r[1] = widen_u8x2<0x4342, F16>(w.x);
    r[2] = widen_u8x2<0x4140, F16>(w.y); r[3] = widen_u8x2<0x4342, F16>(w.y);
    r[4] = widen_u8x2<0x4140, F16>(w.z); r[5] = widen_u8x2<0x4342, F16>(w.z);
    r[6] = widen_u8x2<0x4140, F16>(w.w); r[7] = widen_u8x2<0x4342, F16>(w.w);
}
// registers -> 8 consecutive TMEM columns of this thread's lane (asynchronous; tc_st_wait completes it)
__device__ __forceinline__ void tc_st8(uint32_t taddr, const uint32_t (&r)[8])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]),
                 "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tc_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr)
{
    // K-major operand, 128-byte swizzle: 8-row atoms of 1024 B (stride-byte-offset 1024),
    // descriptor version 1, layout type 2 (SWIZZLE_128B)
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
                 "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
                 : "memory");
}
// the same with the A operand in tensor memory (row m of A in lane m, two 16-bit k elements per column)
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
                 "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
                 : "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// TMEM -> registers, 16 consecutive columns of this thread's lane.  The load is asynchronous: the
// registers are valid after tc_ld_wait, which names them so that no use can move above it.
__device__ __forceinline__ void tc_ld16_issue(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
                   "=r"(r[15])
                 : "r"(taddr));
}
__device__ __forceinline__ void tc_ld_wait4(uint32_t (&a)[16], uint32_t (&b)[16], uint32_t (&c)[16], uint32_t (&d)[16])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                   "+r"(a[8]), "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15]),
                   "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7]),
                   "+r"(b[8]), "+r"(b[9]), "+r"(b[10]), "+r"(b[11]), "+r"(b[12]), "+r"(b[13]), "+r"(b[14]), "+r"(b[15]),
                   "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3]), "+r"(c[4]), "+r"(c[5]), "+r"(c[6]), "+r"(c[7]),
                   "+r"(c[8]), "+r"(c[9]), "+r"(c[10]), "+r"(c[11]), "+r"(c[12]), "+r"(c[13]), "+r"(c[14]), "+r"(c[15]),
                   "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]), "+r"(d[4]), "+r"(d[5]), "+r"(d[6]), "+r"(d[7]),
                   "+r"(d[8]), "+r"(d[9]), "+r"(d[10]), "+r"(d[11]), "+r"(d[12]), "+r"(d[13]), "+r"(d[14]), "+r"(d[15])
                 :
                 : "memory");
}
__device__ __forceinline__ void tc_ld_wait(uint32_t (&a)[16], uint32_t (&b)[16])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]),
                   "+r"(a[8]), "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15]),
                   "+r"(b[0]), "+r"(b[1]), "+r"(b[2]), "+r"(b[3]), "+r"(b[4]), "+r"(b[5]), "+r"(b[6]), "+r"(b[7]),
                   "+r"(b[8]), "+r"(b[9]), "+r"(b[10]), "+r"(b[11]), "+r"(b[12]), "+r"(b[13]), "+r"(b[14]), "+r"(b[15])
                 :
                 : "memory");
}

// KIND: the epilogue; PUSH: the split-K hand-over (0 pull, 1 st.async, 2 bulk copies) - template
// arguments, so that each instantiation carries a single tail and its instructions stay close together.
template <int KIND, int PUSH, bool W8 = false, bool EARLY = false>
__global__ void __launch_bounds__(kTcMaxThreads, 1) k_gemm_tcgen05(const __grid_constant__ GemmTcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t full[kTcMaxStages], empty[kTcMaxStages], accum_bar, push_bar;
    __shared__ uint64_t conv[kTcMaxW8Slots], slot_free[kTcMaxW8Slots];   // int8 weights: a widened tile is complete / has been consumed
    // int8 weights: the activation tiles of the ring's FIRST fill complete a barrier of their own, so that
    // those codes - which land while the kernel in front is still running - are widened before the
    // activations exist (later uses of a stage complete one barrier with both, as without int8)
    __shared__ uint64_t fullb[(W8 && EARLY) ? kTcMaxStages : 1];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile int poisoned;
    __shared__ EpilogueTables tabs;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x;
    const int s = blockIdx.y;
    // k per stage: 64, or 128 with int8 weights (a weight tile is 16 KiB either way) - what the MMA thread and
    // the tensor pipe's front end spend per stage does not depend on what the stage carries, and an int8
    // stage of 64 k carries half the bytes
    constexpr int kBlk = W8 ? 2 * kTcBlockK : kTcBlockK;
    // int8 weights, narrow batches: the codes of the ring's first fill are widened before the activations exist
    constexpr bool kEarly = W8 && EARLY;
    const int a_bytes = p.mt * kATileBytes;
    const int b_bytes = p.planes * p.NB * kBlk * 2;
    const int stage_bytes = a_bytes + b_bytes;
    const int acc_cols = p.planes * p.NB;      // TMEM columns of one weight tile's accumulator
    const int kb0 = (int)((long long)p.kblocks * s / p.splits);
    const int kb1 = (int)((long long)p.kblocks * (s + 1) / p.splits);

    // MMA-issuing threads (see run_mma): two for the int8 kernels with two weight tiles and sixteen epilogue warps
    // (the last of them is then not needed as a converter)
    const int n_issuers = (W8 && p.mt == 2 && p.epi_warps == 16 && p.producers == 3) ? 2 : 1;
    trace_start(p.trace);
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int i = 0; i < p.stages; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], n_issuers);
        }
        mbar_init(&accum_bar, n_issuers);
        if (kEarly) {
            for (int i = 0; i < p.stages; ++i)
                mbar_init(&fullb[i], 1);
        }
        if (W8) {
            // the epilogue warps that issue no TMA loads widen the tiles: one arrival per warp and tile
            for (int j = 0; j < p.w8_slots; ++j) {
                mbar_init(&conv[j], 4);        // one converter warp per TMEM lane quadrant
                mbar_init(&slot_free[j], n_issuers);
            }
        }
        if (PUSH && p.splits > 1) {
            // this rank will receive NB / splits columns of every other rank's partial tile
            mbar_init(&push_bar, 1);
        }
        mbar_fence_init();
        poisoned = 0;
        if (PUSH && p.splits > 1)
            mbar_expect_tx(&push_bar, (uint32_t)(p.splits - 1) * p.mt * kTcTileM * (p.NB / p.splits) * 4u);
        // The ring's first fill, weights only, right here: they never depend on earlier kernels, and a CTA
        // that becomes resident late - after the kernel in front has ended - should have its first bytes
        // under way before anything else of the prologue (tensor-memory allocation, tables, barriers
        // across the CTA and the cluster: 1.5-2 us measured from a CTA's start to its dependency wait).
        {
            const uint64_t pol = policy_evict_first();   // every weight byte is read once per step
            const int n_kb = kb1 - kb0;
            const int pre = n_kb < p.stages ? n_kb : p.stages;
            for (int i = 0; i < pre; ++i) {
                mbar_expect_tx(&full[i], kEarly ? a_bytes : stage_bytes);
                if (p.inject == INJECT_TC_RING && i == 0 && tile == 0 && s == 0)
                    continue;
                if constexpr (W8)
                    bulk_load_hint(smem + (size_t)i * stage_bytes, p.w8_codes + ((size_t)tile * p.kblocks + kb0 + i) * a_bytes,
                                   a_bytes, &full[i], pol);
                else
                    tma_load_2d_hint(smem + (size_t)i * stage_bytes, &p.w_map, (kb0 + i) * kTcBlockK,
                                     tile * p.mt * kTcTileM, &full[i], pol);
            }
        }
        tma_prefetch_desc(&p.x_map);
    }
    load_epilogue_tables(p.epi, tabs, 0, p.B);   // inputs of the step: safe before the wait
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)),
                     "r"((uint32_t)p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    // Every rank's barrier must exist before anybody sends to it: arrive here, wait just before the first
    // send (the tail), so that the cluster barrier's latency is not part of the prologue.
    if (PUSH && p.splits > 1)
        cluster_arrive_relaxed();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    const bool is_epi = warp >= 2;
    // ------------------------------------------------------------ TMA producers
    // Weights never depend on earlier kernels, the activations do: fill the whole ring with
    // weight tiles first (they stream in while the previous kernel finishes), then wait for the
    // previous kernel and add the activation tiles.  Producer j of NP owns the stage uses
    // it = j, j + NP, ...  (one thread each: lane 0 of warp 0, and of epilogue warps 2, 3).
    auto run_producer = [&](int prod) {
        const uint64_t pol = policy_evict_first();   // every weight byte is read once per step
        const int NP = p.producers;
        const int n_kb = kb1 - kb0;
        const int pre = n_kb < p.stages ? n_kb : p.stages;
        // (the ring's first fill of weight tiles was issued by thread 0 at the top of the kernel)
        pdl_wait();
        if (prod == 0)
            trace_waited(p.trace);
        auto load_b = [&](int st_, int kb_, bool first_fill) {
            uint8_t *b_dst = smem + (size_t)st_ * stage_bytes + a_bytes;
            if constexpr (W8) {    // two 64-k boxes
                uint64_t *bar = (kEarly && first_fill) ? &fullb[st_] : &full[st_];
                if (kEarly && first_fill)
                    mbar_expect_tx(bar, b_bytes);
                tma_load_2d(b_dst, &p.x_map, kb_ * kBlk, 0, bar);
                tma_load_2d(b_dst + b_bytes / 2, &p.x_map, kb_ * kBlk + kTcBlockK, 0, bar);
            } else {
                tma_load_2d(b_dst, &p.x_map, kb_ * kBlk, 0, &full[st_]);
            }
        };
        for (int i = prod; i < pre; i += NP)
            load_b(i, kb0 + i, kEarly);
        int it = prod;
        while (it < pre)
            it += NP;
        // (stage and phase of use `it` are kept incrementally: no division on this thread's path)
        int st = it % p.stages;
        uint32_t ph = (uint32_t)(it / p.stages) & 1;
        for (; it < n_kb; it += NP) {
            const int kb = kb0 + it;
            if (!mbar_wait(&empty[st], ph ^ 1, p.status, ST_TIMEOUT_EMPTY)) { poisoned = 1; break; }
            uint8_t *a_dst = smem + (size_t)st * stage_bytes;
            mbar_expect_tx(&full[st], stage_bytes);
            if constexpr (W8)
                bulk_load_hint(a_dst, p.w8_codes + ((size_t)tile * p.kblocks + kb) * a_bytes, a_bytes, &full[st], pol);
            else
                tma_load_2d_hint(a_dst, &p.w_map, kb * kTcBlockK, tile * p.mt * kTcTileM, &full[st], pol);
            load_b(st, kb, false);
            st += NP;
            while (st >= p.stages) {
                st -= p.stages;
                ph ^= 1;
            }
        }
    };
    // ------------------------------------------------------------ MMA issuers
    // One thread issues the MMAs of weight tiles [m_lo, m_hi).  The int8 kernels with two weight tiles
    // per CTA use two such threads (warp 1 and the last epilogue warp, lane 0 each), one per tile: the
    // tiles have separate accumulators, so their MMAs are independent, and what one thread spends per
    // stage (issuing eight MMAs at the pace the tensor pipe takes them, two commits, the next wait) is
    // longer than an int8 stage may take.  A stage and a widened slot are free once both have committed.
    auto run_mma = [&](int m_lo, int m_hi) {
        bool ok = true;
        int st = 0, j = 0;               // ring stage and (int8 weights) widened slot of this use, with their phases
        uint32_t ph = 0, phj = 0;
        for (int kb = kb0; kb < kb1; ++kb) {
            // (int8 weights: the widened tile of this use completes after the stage has landed)
            if (!(W8 ? mbar_wait(&conv[j], phj, p.status, ST_TIMEOUT_FULL)
                       : mbar_wait(&full[st], ph, p.status, ST_TIMEOUT_FULL))) { poisoned = 1; ok = false; break; }
            if constexpr (kEarly) {      // ... and, in the ring's first fill, the stage's activation tiles
                if (kb - kb0 < p.stages && !mbar_wait(&fullb[st], 0, p.status, ST_TIMEOUT_FULL)) { poisoned = 1; ok = false; break; }
            }
            tc_fence_after();
            const uint32_t st_addr = smem_u32(smem + (size_t)st * stage_bytes);
            const uint64_t bdesc = make_smem_desc(st_addr + a_bytes);
            for (int m = m_lo; m < m_hi; ++m) {
                // each 128-row weight tile has its own accumulator (2 * NB TMEM columns)
                if constexpr (W8) {
                    // widened tile of this use: 64 columns per weight tile (128 k), 8 per MMA; the activations
                    // are two 64-k boxes
                    const uint32_t a_tmem = tmem_base + p.mt * acc_cols + (j * p.mt + m) * 64;
                    const uint64_t bdesc2 = make_smem_desc(st_addr + a_bytes + b_bytes / 2);
#pragma unroll
                    for (int k = 0; k < kBlk / 16; ++k)
                        tc_mma_ts(tmem_base + m * acc_cols, a_tmem + 8 * k, (k < 4 ? bdesc : bdesc2) + 2 * (k & 3), p.idesc,
                                  (kb > kb0 || k > 0) ? 1u : 0u);
                } else {
                    const uint64_t adesc = make_smem_desc(st_addr + m * kATileBytes);
#pragma unroll
                    for (int k = 0; k < kTcBlockK / 16; ++k)
                        tc_mma(tmem_base + m * acc_cols, adesc + 2 * k, bdesc + 2 * k, p.idesc,
                               (kb > kb0 || k > 0) ? 1u : 0u);
                }
            }
            tc_commit(&empty[st]);      // slot is free once these MMAs have read it
            if (W8) {
                tc_commit(&slot_free[j]);
                if (++j == p.w8_slots) { j = 0; phj ^= 1; }
            }
            if (++st == p.stages) { st = 0; ph ^= 1; }
        }
        if (ok)
            tc_commit(&accum_bar);      // this issuer's accumulators are complete
    };
    if (warp == 0) {
        if (lane == 0)
            run_producer(0);
    } else if (warp == 1) {
        if (lane == 0)
            run_mma(0, n_issuers == 2 ? 1 : p.mt);
    }
    __syncwarp();

    // ---------------------------------------------------------------- epilogue
    // Accumulator column b holds the hi-plane product of batch row b, column NB + b the
    // lo-plane product; their sum is the result.  Handled 16 batch rows at a time.
    const int lane_grp = warp & 3;          // TMEM lanes this warp may read: 32 * (warp % 4)
    const int row = lane_grp * 32 + lane;   // row of the tile
    const int nchunks = p.NB / 16;
    const int sub = is_epi ? (warp - 2) >> 2 : 0;        // which of the lane group's warps this is
    // int8 weights: every accumulator row (= packed weight row) is multiplied by its scale as it leaves
    // TMEM.  The scales are weights - fetched here, ahead of the stream, not behind the last MMA where
    // their memory round trip would sit on the kernel's tail.
    float wsc[2] = {1.f, 1.f};
    if (W8 && is_epi) {
        wsc[0] = p.wscale[(size_t)(tile * p.mt) * kTcTileM + row];
        if (p.mt == 2)
            wsc[1] = p.wscale[(size_t)(tile * p.mt + 1) * kTcTileM + row];
    }
    const int kSubs = ((int)blockDim.x / 32 - 2) / 4;    // warps per lane group
    const int par = lane & 1;
    // Rotary factors of this thread's first two finish iterations of a one-sided split-K reduction
    // (the iteration order is fixed: column pairs sub, sub + kSubs, ... of this rank's columns):
    // computed here, while the weights stream, instead of in the tail.
    float2 trig[2] = {make_float2(1.f, 0.f), make_float2(1.f, 0.f)};
    if (is_epi && KIND == EPI_QKV && p.splits > 1 && PUSH == 2) {
        // (bulk form: a warp's first item is column warp - 2 of this rank's mt * cols (m, column)
        // items, a lane's two pairs are rows 4 * lane .. 4 * lane + 3)
        const int cols = p.NB / p.splits;
        int m = 0, cl = warp - 2;
        while (cl >= cols) { cl -= cols; ++m; }
        const int b = s * cols + cl;
        if (m < p.mt && b < p.B) {
            trig[0] = rope_trig(p.epi, tabs, tabs.pos[b], tile * p.mt + m, 2 * lane);
            trig[1] = rope_trig(p.epi, tabs, tabs.pos[b], tile * p.mt + m, 2 * lane + 1);
        }
    } else if (is_epi && KIND == EPI_QKV && p.splits > 1 && PUSH == 1) {
        const int cols = p.NB / p.splits, hp = cols / 2;
        int m = 0, c2 = sub;
        while (c2 >= hp) { c2 -= hp; ++m; }
#pragma unroll
        for (int k = 0; k < 2; ++k)
            if (m < p.mt) {
                const int b = s * cols + 2 * c2 + par;
                if (b < p.B)
                    trig[k] = rope_trig(p.epi, tabs, tabs.pos[b], tile * p.mt + m, row >> 1);
                c2 += kSubs;
                while (c2 >= hp) { c2 -= hp; ++m; }
            }
    }
    // one finished pair of iteration k (k < 2 uses the factors above)
    auto finish_pair = [&](int k, int m, int b, float v0, float v1) {
        const int pair = ((tile * p.mt + m) * kTcTileM + row) >> 1;
        if constexpr (KIND == EPI_QKV) {
            const int pos = tabs.pos[b], hd = pair >> 6, i = pair & 63;
            const float2 cs = k == 0 ? trig[0] : (k == 1 ? trig[1] : rope_trig(p.epi, tabs, pos, hd, i));
            epilogue_qkv(p.epi, pos, b, hd, i, v0, v1, cs);
        } else {
            apply_epilogue_t<KIND>(p.epi, tabs, b, true, p.N, b, pair, v0, v1);
        }
    };
    // the first epilogue warps lend their lane 0 to the ring (the warp reconverges behind the block)
    if (is_epi && warp - 1 < p.producers) {
        if (lane == 0)
            run_producer(warp - 1);
        __syncwarp();
    }
    else if (is_epi && W8 && n_issuers == 2 && warp == 1 + p.epi_warps) {
        if (lane == 0)
            run_mma(1, 2);
        __syncwarp();
    }
    else if (is_epi && W8) {
        // ---------------------------------------------------- int8 weights: widen every tile
        // Tile use `itc` is widened from its ring stage into tensor-memory slot itc % slots, where the
        // MMA takes it as its A operand: row r of a weight tile in TMEM lane r, 64 columns per 128 k.
        // A warp reaches the 32 lanes of its quadrant (warp % 4) only, so the converter warps of a
        // quadrant share that quadrant's tasks: task (m, q) = rows 32 * quadrant .. + 31 of weight
        // tile m, k = 16 q .. 16 q + 15 - per lane one 16-byte load (the packed block keeps the four
        // 16-byte groups of a row in an order that makes these loads conflict-free) and one store of
        // 8 columns.  The slot is written again only after the MMAs of use itc - slots have read it.
        // The converter warps form groups of four, one warp per quadrant; group g widens the tile uses
        // g, g + G, ... on its own, so successive stages are widened concurrently (a single group
        // needs longer for one stage than the stage may take).
        const int quad = warp & 3;
        int iq = 0, n_min = 1 << 30;     // this warp's index among its quadrant's converter warps; the groups
        for (int q2 = 0; q2 < 4; ++q2) {
            int n = 0;
            for (int w2 = p.producers + 1; w2 < 2 + p.epi_warps - (n_issuers == 2 ? 1 : 0); ++w2)
                if ((w2 & 3) == q2) {
                    if (q2 == quad && w2 < warp)
                        ++iq;
                    ++n;
                }
            n_min = n < n_min ? n : n_min;
        }
        const int G = n_min;
        const bool f16 = p.f16 != 0;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(p.mt * acc_cols);
        const uint32_t src_lane = (uint32_t)row * 128;
        const uint32_t swz = (uint32_t)(row & 7);
        int st = 0, j = 0;
        uint32_t ph = 0, phj = 0;
        bool reuse = false;          // the slot has been used before: wait until the MMAs of that use are done
        int turn = 0;                // use index modulo G
        for (int kb = kb0; kb < kb1 && iq < G; ++kb) {
            if (turn == iq) {
                int ok = 1;
                if (lane == 0) {
                    ok = mbar_wait(&full[st], ph, p.status, ST_TIMEOUT_FULL) ? 1 : 0;
                    if (ok && reuse)
                        ok = mbar_wait(&slot_free[j], phj ^ 1, p.status, ST_TIMEOUT_EMPTY) ? 1 : 0;
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { poisoned = 1; break; }
                tc_fence_after();
                const uint8_t *a8 = smem + (size_t)st * stage_bytes + src_lane;
                const uint32_t slot_addr = lane_addr + (uint32_t)(j * p.mt * 64);
                for (int mh = 0; mh < 2 * p.mt; ++mh) {      // (weight tile, half of its 128 k): four 16-byte groups
                    const int m = mh >> 1, q0 = (mh & 1) * 4;
                    uint4 w[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        w[q] = *reinterpret_cast<const uint4 *>(a8 + m * (kTcTileM * 128) + (((q0 + q) ^ swz) << 4));
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t r[8];
                        if (f16)
                            widen16<true>(w[q], r);
                        else
                            widen16<false>(w[q], r);
                        tc_st8(slot_addr + (uint32_t)(m * 64 + (q0 + q) * 8), r);
                    }
                }
                tc_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0)
                    mbar_arrive(&conv[j]);
            }
            if (++turn == G) turn = 0;
            if (++j == p.w8_slots) { j = 0; phj ^= 1; reuse = true; }
            if (++st == p.stages) { st = 0; ph ^= 1; }
        }
        __syncwarp();
    }
    bool have = false;
    if (is_epi) {
        have = mbar_wait(&accum_bar, 0, p.status, ST_TIMEOUT_MMA);
        if (!have)
            poisoned = 1;
        tc_fence_after();
        trace_streamed(p.trace, threadIdx.x == 64);
    }
    const uint32_t t_lane = tmem_base + ((uint32_t)(lane_grp * 32) << 16);
    float *red = reinterpret_cast<float *>(smem);      // [mt][NB][128] fp32, reuses the ring

    auto wscale_of = [&](int m) -> float {
        if constexpr (W8)
            return m ? wsc[1] : wsc[0];
        else
            return 1.f;
    };
    // hi- and lo-plane columns are fetched together, one wait for both
    auto load_chunk = [&](int m, int c, float (&v)[16]) {
        if (have) {
            uint32_t hi[16], lo[16];
            tc_ld16_issue(t_lane + m * acc_cols + c * 16, hi);
            if (p.planes == 2) {
                tc_ld16_issue(t_lane + m * acc_cols + p.NB + c * 16, lo);
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    lo[i] = 0u;
            }
            tc_ld_wait(hi, lo);
#pragma unroll
            for (int i = 0; i < 16; ++i)
                v[i] = (__uint_as_float(hi[i]) + __uint_as_float(lo[i])) * wscale_of(m);
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i)
                v[i] = 0.f;
        }
    };

    if (PUSH == 2 && p.splits > 1) {
        // Split-K across the cluster for wide batches, one-sided reduce-scatter by bulk copies: every
        // rank lays its partial tiles out in its own (idle) ring as [m][column][row], then one bulk
        // copy per (owner, m) moves the owner's columns - a contiguous slice - into the owner's receive
        // area [source slot][m][column][row], signalling the owner's barrier with the bytes.  The owner
        // waits for its area, sums the sources in rank order (its own share straight from its ring)
        // and applies the epilogue.  The cluster barrier that keeps the senders' shared memory alive
        // until the copies have landed is split: arrive once this rank's area is complete, wait at
        // the very end, so its latency hides behind the epilogue.
        cg::cluster_group cluster = cg::this_cluster();
        const int cols = p.NB / p.splits;
        float *recv = reinterpret_cast<float *>(smem + p.recv_off);
        cluster_wait();       // (the arrival at the top of the kernel: every rank's receive barrier exists)
        if (is_epi) {
            // two chunks (four TMEM loads) in flight per wait
            const uint32_t red_row = smem_u32(red) + (uint32_t)row * 4u;
            for (int j = sub; j < p.mt * nchunks; j += 2 * kSubs) {
                const int j1 = j + kSubs;
                const bool two = j1 < p.mt * nchunks;
                const int m0 = j / nchunks, c0 = j % nchunks;
                const int m1 = two ? j1 / nchunks : m0, c1 = two ? j1 % nchunks : c0;
                uint32_t h0[16], l0[16], h1[16], l1[16];
                if (have) {
                    tc_ld16_issue(t_lane + m0 * acc_cols + c0 * 16, h0);
                    tc_ld16_issue(t_lane + m1 * acc_cols + c1 * 16, h1);
                    if (p.planes == 2) {
                        tc_ld16_issue(t_lane + m0 * acc_cols + p.NB + c0 * 16, l0);
                        tc_ld16_issue(t_lane + m1 * acc_cols + p.NB + c1 * 16, l1);
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            l0[i] = l1[i] = 0u;
                    }
                    tc_ld_wait4(h0, l0, h1, l1);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        h0[i] = l0[i] = h1[i] = l1[i] = 0u;
                }
                const uint32_t a0 = red_row + (uint32_t)((m0 * p.NB + c0 * 16) * kTcTileM) * 4u;
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    sts_f32(a0 + i * (kTcTileM * 4), (__uint_as_float(h0[i]) + __uint_as_float(l0[i])) * wscale_of(m0));
                if (two) {
                    const uint32_t a1 = red_row + (uint32_t)((m1 * p.NB + c1 * 16) * kTcTileM) * 4u;
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        sts_f32(a1 + i * (kTcTileM * 4), (__uint_as_float(h1[i]) + __uint_as_float(l1[i])) * wscale_of(m1));
                }
            }
            fence_proxy_async_smem();
            asm volatile("bar.sync 1, %0;" ::"r"(kSubs * 128) : "memory");
            // copy e is issued by lane e / n_warps of epilogue warp e % n_warps: spread over the warps,
            // the (splits - 1) * mt copies go out side by side
            const int n_ewarps = kSubs * 4;
            const int e = lane < 8 ? (warp - 2) + lane * n_ewarps : 1 << 30;
            if (e < (p.splits - 1) * p.mt) {
                const int slot_q = e / p.mt, m = e % p.mt;
                const int q = slot_q < s ? slot_q : slot_q + 1;      // owner
                const int my_slot = s < q ? s : s - 1;               // where the owner keeps this rank's share
                bulk_copy_to_cluster(cluster_map(recv + ((size_t)(my_slot * p.mt + m) * cols) * kTcTileM, q),
                                     smem_u32(red + ((size_t)m * p.NB + q * cols) * kTcTileM),
                                     (uint32_t)cols * kTcTileM * 4u, cluster_map(&push_bar, q));
            }
            if (!mbar_wait(&push_bar, 0, p.status, ST_TIMEOUT_MMA))
                poisoned = 1;
        }
        cluster_arrive_relaxed();
        if (is_epi) {
            // finish this rank's columns: one (m, column) item per warp and iteration, a lane takes
            // rows 4 * lane .. 4 * lane + 3 - two complete output pairs - with one 16-byte load per rank
            const int n_ew = kSubs * 4;
            const uint32_t red_a = smem_u32(red) + (uint32_t)(s * cols * kTcTileM) * 4u + lane * 16u;
            const uint32_t recv_a = smem_u32(recv) + lane * 16u;
            const bool bad = poisoned;
            auto finish = [&](auto sp_tag) {
                constexpr int SP = decltype(sp_tag)::value;
                // per source rank: address of (m = 0, column 0, this lane's rows) and the stride between m
                uint32_t base[SP], mstr[SP];
#pragma unroll
                for (int q = 0; q < SP; ++q) {
                    base[q] = q == s ? red_a : recv_a + (uint32_t)((q < s ? q : q - 1) * p.mt * cols) * (kTcTileM * 4u);
                    mstr[q] = (uint32_t)(q == s ? p.NB : cols) * (kTcTileM * 4u);
                }
                int m = 0, cl = warp - 2;
                while (cl >= cols) { cl -= cols; ++m; }
                for (int k = 0; m < p.mt; ++k) {
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int q = 0; q < SP; ++q) {         // rank order
                        const float4 t4 = lds_f32x4(base[q] + m * mstr[q] + (uint32_t)cl * (kTcTileM * 4u));
                        acc.x += t4.x; acc.y += t4.y; acc.z += t4.z; acc.w += t4.w;
                    }
                    const int b = s * cols + cl;
                    if (b < p.B && !bad)
                        apply_epilogue_quad_t<KIND>(p.epi, tabs, p.N, b, (tile * p.mt + m) * (kTcTileM / 2) + 2 * lane, acc, k == 0,
                                            trig[0], trig[1]);
                    cl += n_ew;
                    while (cl >= cols) { cl -= cols; ++m; }
                }
            };
            if (p.splits == 2)
                finish(std::integral_constant<int, 2>());
            else if (p.splits == 4)
                finish(std::integral_constant<int, 4>());
            else if (p.splits == 8)
                finish(std::integral_constant<int, 8>());
            else
                finish(std::integral_constant<int, 16>());
        }
        cluster_wait();
        // (failure path: every peer has issued its copies by now; let those in flight land before the exit,
        // and give this CTA's own copies - whose source is its shared memory, and whose receivers may have
        // arrived at the barrier without them - 20 us to leave it)
        if (poisoned && threadIdx.x == 0) {
            mbar_wait(&push_bar, 0, p.status, ST_TIMEOUT_MMA);
            const long long t_lin = gtime();
            while (gtime() - t_lin < 20000)
                __nanosleep(1000);
        }
    } else if (PUSH == 1 && p.splits > 1) {
        // Split-K across the cluster, one-sided reduce-scatter: rank q finishes columns [q * cols,
        // (q + 1) * cols).  Every rank stores those columns of its partial tile into rank q's receive
        // area [source rank][m][row][cols] (st.async, signalling q's barrier with the bytes; its own
        // share with plain stores), then waits until its own area is complete and sums the sources in
        // rank order.  No cluster barrier and no remote loads on the critical path.
        const int cols = p.NB / p.splits;
        const uint32_t recv_a = smem_u32(smem + p.recv_off);
        const uint32_t src_stride = (uint32_t)p.mt * kTcTileM * cols * 4u;          // bytes per source rank
        cluster_wait();       // (the arrival at the top of the kernel: every rank's receive barrier exists)
        if (is_epi) {
            for (int j = sub; j < p.mt * nchunks; j += kSubs) {
                const int m = j / nchunks, c = j % nchunks;
                float v[16];
                load_chunk(m, c, v);
                const uint32_t off = recv_a + s * src_stride + (uint32_t)((m * kTcTileM + row) * cols) * 4u;   // my slot, my row
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    const int col = c * 16 + i, q = col / cols, cl = col % cols;
                    if (cols % 4 == 0) {
                        if (i % 4 == 0) {
                            const float4 val = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                            if (q == s)
                                sts_f32x4(off + cl * 4, val);
                            else
                                st_async_v4(cluster_map_addr(off + cl * 4, q), val, cluster_map(&push_bar, q));
                        }
                    } else {
                        const float2 val = make_float2(v[i], v[i + 1]);
                        if (q == s)
                            sts_f32x2(off + cl * 4, val);
                        else
                            st_async_v2(cluster_map_addr(off + cl * 4, q), val, cluster_map(&push_bar, q));
                    }
                }
            }
            asm volatile("bar.sync 1, %0;" ::"r"(kSubs * 128) : "memory");    // own share stored by all epilogue warps
            if (!mbar_wait(&push_bar, 0, p.status, ST_TIMEOUT_MMA))
                poisoned = 1;
            const bool bad = poisoned;
            const uint32_t row_a = recv_a + (uint32_t)(row * cols) * 4u;
            const uint32_t mstr = (uint32_t)(kTcTileM * cols) * 4u;
            auto finish = [&](auto sp_tag) {
                constexpr int SP = decltype(sp_tag)::value;
                const int hp = cols / 2;                   // column pairs per m
                int m = 0, c2 = sub;
                while (c2 >= hp) { c2 -= hp; ++m; }
                for (int k = 0; m < p.mt; ++k) {
                    const uint32_t a = row_a + m * mstr + c2 * 8u;
                    float mine[2] = {0.f, 0.f};
#pragma unroll
                    for (int q = 0; q < SP; ++q) {         // rank order
                        const float2 t2 = lds_f32x2(a + q * src_stride);
                        mine[0] += t2.x;
                        mine[1] += t2.y;
                    }
                    const float got = __shfl_xor_sync(0xffffffffu, par ? mine[0] : mine[1], 1);
                    const int b = s * cols + 2 * c2 + par;
                    if (b < p.B && !bad)
                        finish_pair(k, m, b, par ? got : mine[0], par ? mine[1] : got);
                    c2 += kSubs;
                    while (c2 >= hp) { c2 -= hp; ++m; }
                }
            };
            if (p.splits == 2)
                finish(std::integral_constant<int, 2>());
            else if (p.splits == 4)
                finish(std::integral_constant<int, 4>());
            else
                finish(std::integral_constant<int, 8>());
        }
    } else if (PUSH == 0 && p.splits > 1) {
        // Split-K across the cluster, reduce-scatter style: every rank publishes its partial tiles in
        // its own shared memory, then finishes NB / splits of the batch columns - reading that slice
        // from all ranks in rank order - so the reduction and the epilogue work are spread over the
        // whole cluster.
        cg::cluster_group cluster = cg::this_cluster();
        if (is_epi) {
            for (int j = sub; j < p.mt * nchunks; j += kSubs) {      // the lane group's warps share the chunks
                const int m = j / nchunks, c = j % nchunks;
                float v[16];
                load_chunk(m, c, v);
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    red[((size_t)m * p.NB + c * 16 + i) * kTcTileM + row] = v[i];
            }
        }
        cluster.sync();
        if (is_epi) {
            const float *remote[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
                remote[q] = cluster.map_shared_rank(red, q < p.splits ? q : 0) + row;
            const int cols = p.NB / p.splits;             // columns finished by this rank (>= 2, even)
            const int n_pairs = p.mt * cols / 2;
            // The remote loads of a block of column pairs (16 values per rank slot in flight) are
            // issued before the first pair of the block is finished: distributed shared memory has a
            // latency of ~800 cycles, so a thread that fetched pair by pair would spend that long on
            // each of its mt * cols / 2 pairs.
            auto run = [&](auto sp_tag) {
                constexpr int SP = decltype(sp_tag)::value;
                constexpr int D = 16 / SP;                 // pairs per block
                // (this warp's pairs: sub, sub + kSubs, ...)
                for (int it0 = sub; it0 < n_pairs; it0 += D * kSubs) {
                    float buf[D][2][SP];
#pragma unroll
                    for (int d = 0; d < D; ++d) {
                        const int it = it0 + d * kSubs;
                        if (it < n_pairs) {
                            const int m = it / (cols / 2), b0 = s * cols + 2 * (it % (cols / 2));
#pragma unroll
                            for (int q = 0; q < SP; ++q) {
                                buf[d][0][q] = remote[q][((size_t)m * p.NB + b0 + 0) * kTcTileM];
                                buf[d][1][q] = remote[q][((size_t)m * p.NB + b0 + 1) * kTcTileM];
                            }
                        }
                    }
#pragma unroll
                    for (int d = 0; d < D; ++d) {
                        const int it = it0 + d * kSubs;
                        if (it < n_pairs) {
                            const int m = it / (cols / 2), b0 = s * cols + 2 * (it % (cols / 2));
                            const int pair = ((tile * p.mt + m) * kTcTileM + row) >> 1;
                            float mine[2] = {0.f, 0.f};
#pragma unroll
                            for (int q = 0; q < SP; ++q) {       // rank order
                                mine[0] += buf[d][0][q];
                                mine[1] += buf[d][1][q];
                            }
                            // rows 2r and 2r + 1 (adjacent lanes) form the output pair: the even lane finishes
                            // column b0, the odd lane column b0 + 1, each with one value from its neighbour -
                            // one exchange and one epilogue call for the whole warp
                            const float recv = __shfl_xor_sync(0xffffffffu, par ? mine[0] : mine[1], 1);
                            const int b = b0 + par;
                            if (b < p.B && !poisoned)
                                apply_epilogue_t<KIND>(p.epi, tabs, b, true, p.N, b, pair, par ? recv : mine[0], par ? mine[1] : recv);
                        }
                    }
                }
            };
            if (p.splits == 2)
                run(std::integral_constant<int, 2>());
            else if (p.splits == 4)
                run(std::integral_constant<int, 4>());
            else
                run(std::integral_constant<int, 8>());
        }
        cluster.sync();        // peers' shared memory must outlive the reads
    } else if (is_epi) {
        for (int j = sub; j < p.mt * nchunks; j += kSubs) {
            const int m = j / nchunks, c = j % nchunks;
            const int pair = ((tile * p.mt + m) * kTcTileM + row) >> 1;
            float v[16];
            load_chunk(m, c, v);
#pragma unroll
            for (int i = 0; i < 16; i += 2) {
                // (as above: the even lane of a row pair finishes column i, the odd lane column i + 1)
                const float recv = __shfl_xor_sync(0xffffffffu, par ? v[i] : v[i + 1], 1);
                const int b = c * 16 + i + par;
                if (b < p.B && !poisoned)
                    apply_epilogue_t<KIND>(p.epi, tabs, b, true, p.N, b, pair, par ? recv : v[i], par ? v[i + 1] : recv);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PUSH == 1 && p.splits > 1 && poisoned) {
        // A wait of this CTA ran out, so it may be about to leave before every peer has stored its share
        // into this CTA's receive area - and a store into the shared memory of a CTA that has exited is
        // a fault.  Stay until every peer has either left (its stores were issued before that) or
        // reached this point too, then give the stores in flight a bounded time to land.  (A CTA whose
        // waits all succeeded has received everything and may simply leave: the barrier counts only
        // threads that have not exited.)
        cluster_arrive_relaxed();
        cluster_wait();
        if (threadIdx.x == 0)
            mbar_wait(&push_bar, 0, p.status, ST_TIMEOUT_MMA);
        __syncthreads();
    }
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols)
                     : "memory");
    }
    trace_end(p.trace);
}

template <int KIND, int PUSH, bool W8 = false, bool EARLY = false>
static cudaError_t launch_instance(cudaLaunchConfig_t &cfg, const GemmTcParams &p, size_t smem)
{
    static PerDeviceSize smem_limit, np_set;      // per instantiation and device
    cudaError_t e = ensure_dynamic_smem(k_gemm_tcgen05<KIND, PUSH, W8, EARLY>, smem_limit, smem);
    if (e != cudaSuccess)
        return e;
    if (p.splits > 8) {
        const int dev = current_device_index();
        if (dev < 0)
            return cudaErrorInvalidDevice;
        if (!np_set.v[dev]) {
            e = cudaFuncSetAttribute(k_gemm_tcgen05<KIND, PUSH, W8, EARLY>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
            if (e != cudaSuccess)
                return e;
            np_set.v[dev] = 1;
        }
    }
    return cudaLaunchKernelEx(&cfg, k_gemm_tcgen05<KIND, PUSH, W8, EARLY>, p);
}

// int8 weights: 128-row weight tiles per CTA (1 or 2).  The two widened tiles behind the ring cost
// mt * 32 KiB; one weight tile per CTA when that is what lets two CTAs share an SM (the second streams
// while the first is in its epilogue).  The packed codes are laid out for this number (pack.cu).
int gemm_tc_w8_tiles(int NB, int N, int x_fp16)
{
    // Narrow batches: one tile, so that two CTAs can share an SM's tensor memory (and the grid has
    // twice the CTAs to fill the SMs with).  Wide batches: two tiles (one activation tile serves both)
    // whenever the matrix has an even number of them and tensor memory (512 columns) holds two
    // accumulators plus at least two widened tiles of 2 * 64 columns (128 k).
    if (NB <= 32)
        return 1;
    const int acc = (x_fp16 ? 1 : 2) * NB;
    return (N % (2 * kTcTileM) == 0 && 2 * acc + 2 * 2 * 64 <= 512) ? 2 : 1;
}

cudaError_t launch_gemm_tc(const GemmTcArgs &a, int sm_count, cudaStream_t s)
{
    if (a.NB < 16 || a.NB > 128 || a.NB % 16 || a.N % kTcTileM || a.K % (a.w8 ? 2 * kTcBlockK : kTcBlockK) || a.B > a.NB)
        return cudaErrorInvalidValue;
    GemmTcParams p;
    p.w_map = a.w_map;
    p.x_map = a.x_map;
    p.B = a.B; p.NB = a.NB; p.N = a.N; p.K = a.K;
    p.kblocks = a.K / (a.w8 ? 2 * kTcBlockK : kTcBlockK);
    p.epi = a.epi;
    p.status = a.status;
    p.trace = a.trace;
    p.inject = a.inject;
    const int planes = a.x_fp16 == 1 ? 1 : 2;
    p.planes = planes;
    p.f16 = a.x_fp16 ? 1 : 0;
    // Two 128-row weight tiles per CTA share one activation tile when the activation tile (planes * NB
    // rows) weighs about as much as a weight tile: halves the L2->SM traffic of the activations, which
    // every CTA re-reads.  With a single fp16 plane of 64 rows it does not: one tile per CTA then gives
    // twice the CTAs (two per SM) and measured 1-1.5 us less on the O and down projections of config 4.
    const int mt = a.w8 ? gemm_tc_w8_tiles(a.NB, a.N, a.x_fp16 == 1)
                        : ((planes * a.NB >= 96 && a.N % (2 * kTcTileM) == 0 && a.w_map256) ? 2 : 1);
    if (a.w8 && (!a.w8_codes || !a.scales))
        return cudaErrorInvalidValue;
    p.w8_codes = static_cast<const uint8_t *>(a.w8_codes);
    p.mt = mt;
    if (mt == 2 && !a.w8)
        p.w_map = *a.w_map256;
    const int tiles = a.N / (kTcTileM * mt);
    // int8 weights: a stage holds the codes (half a 16-bit tile) and the activations; the widened tiles
    // live in tensor memory behind the accumulators (as many as fit, at most four), so the whole of
    // shared memory is ring: a deep ring is what keeps enough int8 bytes in flight.  One CTA per SM
    // (tensor memory is per SM).
    const int stage_bytes = mt * kATileBytes + planes * a.NB * (a.w8 ? 2 * kTcBlockK : kTcBlockK) * 2;
    // Two CTAs per SM when each needs at most half of tensor memory (accumulators + at least two widened
    // tiles in 256 columns) and half of shared memory still holds three stages; else one.
    int w8_slots = 0;
    bool w8_two = false;
    if (a.w8) {
        const int acc = mt * planes * a.NB;
        w8_two = acc + 2 * mt * 64 <= 256 && (100 * 1024) / stage_bytes >= 3;
        w8_slots = ((w8_two ? 256 : 512) - acc) / (mt * 64);
        w8_slots = w8_slots > kTcMaxW8Slots ? kTcMaxW8Slots : w8_slots;
        if (w8_slots < 2)
            return cudaErrorInvalidValue;
    }
    p.w8_slots = w8_slots;
    // (measured: pays for narrow batches - two CTAs per SM, few stages per CTA - and costs ~1 % on wide ones)
    p.w8_early = a.w8 && w8_two;
    const int a16_bytes = 0;
    p.w8 = a.w8;
    p.wscale = a.scales;
    // Ring depth, CTAs per SM and cluster splits.  Two CTAs per SM (rings <= 100 KiB) whenever that
    // leaves >= 4 stages: measured better than one CTA with a ring twice as deep, because the second
    // CTA streams while the first is in its epilogue.  The grid (tiles x splits) must fit the
    // co-resident slots (a second wave doubles the kernel); splits are a power of two <= 8 that leave
    // every rank >= 2 k-blocks.
    int stages = (200 * 1024 - a16_bytes) / stage_bytes, per_sm = 1;
    if (a.w8 ? w8_two : (100 * 1024 - a16_bytes) / stage_bytes >= 4) {
        stages = (100 * 1024 - a16_bytes) / stage_bytes;
        per_sm = 2;
    }
    if (stages > kTcMaxStages) stages = kTcMaxStages;
    if (stages < 2)
        return cudaErrorInvalidValue;
    const int slots = sm_count * per_sm;
    int splits = 1;
    while (splits < 8 && tiles * splits * 2 <= slots && p.kblocks / (splits * 2) >= 2) splits *= 2;
    // Sixteen ranks (a cluster size the device has to be asked for) when even eight leave half of the
    // SMs without a CTA; only with the bulk hand-over, whose owners may hold a single column.
    const size_t need16 = (size_t)mt * a.NB * kTcTileM * 4 / 16 * 15;
    const bool sixteen = splits == 8 && tiles * 16 <= slots && tiles * 8 * 5 <= sm_count * 3 && p.kblocks / 16 >= 2 &&
                         a.NB % 16 == 0 &&
                         (size_t)3 * stage_bytes + a16_bytes + need16 + 1024 <= (size_t)(per_sm == 2 ? 108 : 225) * 1024;
    if (sixteen)
        splits = 16;
    p.stages = stages;
    p.splits = splits;
    int cols = 32;
    while (cols < mt * planes * a.NB + w8_slots * mt * 64) cols *= 2;
    p.tmem_cols = cols;
    // instruction descriptor: fp32 accumulate; A (weights) and B (activations) in the same 16-bit format -
    // both bf16 (B = hi + lo planes) or both fp16 (B = one plane); N = columns of the B tile, M = 128
    const uint32_t fmt = a.x_fp16 ? 0u : 1u;
    p.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)((planes * a.NB) >> 3) << 17) |
              ((uint32_t)(kTcTileM >> 4) << 24);

    // one-sided split-K reduction when the receive area (one partial tile per CTA) is small - every
    // thread then hands over one or two 16-byte pieces per owner; wide batches keep the pull form,
    // whose remote accesses are full 128-byte rows - and fits behind the ring
    const size_t recv_bytes = (size_t)mt * a.NB * kTcTileM * 4;
    const size_t smem_cap = (per_sm == 2 ? 108 : 225) * 1024;
    p.push = 0;
    if (splits > 1 && splits <= 8 && recv_bytes <= 16 * 1024) {
        int st = stages;
        while (st > 3 && (size_t)st * stage_bytes + a16_bytes + recv_bytes + 1024 > smem_cap) --st;
        if ((size_t)st * stage_bytes + a16_bytes + recv_bytes + 1024 <= smem_cap) {
            stages = st;
            p.stages = st;
            p.push = 1;
        }
    }
    // wide batches: the same by bulk copies (receive area: the other ranks' shares of this rank's columns)
    size_t recv_alloc = p.push ? recv_bytes : 0;
    if (splits > 1 && !p.push) {
        const size_t need = recv_bytes / splits * (splits - 1);
        int st = stages;
        while (st > 3 && (size_t)st * stage_bytes + a16_bytes + need + 1024 > smem_cap) --st;
        if ((size_t)st * stage_bytes + a16_bytes + need + 1024 <= smem_cap) {
            stages = st;
            p.stages = st;
            p.push = 2;
            recv_alloc = need;
        }
    }
    p.recv_off = stages * stage_bytes + a16_bytes;
    size_t smem = (size_t)stages * stage_bytes + a16_bytes + recv_alloc + 1024;
    const size_t red_bytes = (size_t)mt * a.NB * kTcTileM * 4 + 1024;
    if (smem < red_bytes) smem = red_bytes;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(tiles, splits, 1);
    // epilogue warps: 16 when the CTA has the SM to itself and enough column pairs per thread to share,
    // else 8 (two CTAs per SM must share the registers)
    const int epi_warps = (per_sm == 1 && mt * (a.NB / splits) / 2 >= 8) ? 16 : 8;
    p.epi_warps = epi_warps;
    p.producers = stages < kTcMaxProducers ? stages : kTcMaxProducers;
    if (a.w8 && (!a.scales || epi_warps - (p.producers - 1) < 1))
        return cudaErrorInvalidValue;
    cfg.blockDim = dim3((2 + epi_warps) * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    int n = pdl_attr(at, a.pdl);
    if (splits > 1) {
        at[n].id = cudaLaunchAttributeClusterDimension;
        at[n].val.clusterDim.x = 1;
        at[n].val.clusterDim.y = splits;
        at[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = at;
    cfg.numAttrs = n;
    const int push = splits > 1 ? p.push : 0;
#define PRSV_TC_CASE(KIND, PUSH)                                   \
    if (a.epi.kind == (KIND) && push == (PUSH))                    \
        return a.w8 ? (p.w8_early ? launch_instance<KIND, PUSH, true, true>(cfg, p, smem) : launch_instance<KIND, PUSH, true, false>(cfg, p, smem)) \
                    : launch_instance<KIND, PUSH, false>(cfg, p, smem);
    PRSV_TC_CASE(EPI_PLAIN, 0) PRSV_TC_CASE(EPI_PLAIN, 1) PRSV_TC_CASE(EPI_PLAIN, 2)
    PRSV_TC_CASE(EPI_QKV, 0) PRSV_TC_CASE(EPI_QKV, 1) PRSV_TC_CASE(EPI_QKV, 2)
    PRSV_TC_CASE(EPI_SWIGLU, 0) PRSV_TC_CASE(EPI_SWIGLU, 1) PRSV_TC_CASE(EPI_SWIGLU, 2)
#undef PRSV_TC_CASE
    return cudaErrorInvalidValue;
}

}  // namespace prsv
