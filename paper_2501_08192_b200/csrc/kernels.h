// Internal launch interface between the layer runtime (api.cu) and the kernels.
// Every launcher is asynchronous on the given stream and returns the launch's
// cudaError_t.  No launcher allocates.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

namespace prsv {

// Programmatic dependent launch: when `pdl` is non-zero the kernel is launched with the
// programmatic-serialization attribute, so its prologue (index setup, first weight
// loads) may overlap the previous kernel's tail.  Each kernel executes
// griddepcontrol.wait before it touches anything another kernel wrote.  The switch is
// a launch argument (every launcher's args carry it): no process-wide state.
inline int pdl_attr(cudaLaunchAttribute *at, int pdl)
{
    if (!pdl)
        return 0;
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    return 1;
}

// cudaFuncSetAttribute applies to the current device only, so "already set" is kept per
// device (indexed by cudaGetDevice), never per process.  Setting an attribute twice is
// harmless, so two threads that race here both succeed.
constexpr int kMaxDevices = 64;
struct PerDeviceSize {
    size_t v[kMaxDevices] = {};
};
inline int current_device_index()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return -1;
    return dev;
}
// Raise kernel `fn`'s dynamic shared-memory limit to at least `bytes` on the current device.
template <typename Fn>
inline cudaError_t ensure_dynamic_smem(Fn fn, PerDeviceSize &state, size_t bytes)
{
    const int dev = current_device_index();
    if (dev < 0)
        return cudaErrorInvalidDevice;
    if (bytes <= state.v[dev])
        return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess)
        state.v[dev] = bytes;
    return e;
}

// Test hooks (preserve_debug_set): make ONE producer of a kernel withhold ONE issue, so that the
// consumer's bounded wait runs out and the give-up path runs.  Nothing faults or hangs: the wait
// expires after the handle's wait limit and the kernel returns with a status code.
enum Inject : int { INJECT_NONE = 0, INJECT_WINDOW_HANDOVER = 1, INJECT_GEMV_RING = 2, INJECT_TC_RING = 3,
                    INJECT_ATTN_RING = 4 };

// Device status block of a layer (ints): [0] status word (first writer wins), [2..3] the handle's
// limit on any mbarrier wait in SM cycles (64-bit, 0 = the default below), [8] sink of the
// prefetch kernel's load variant, [16..27] the prefetch kernels' own evaluation of the plan
// (uint64 [2][3], written by CTA 0 of each prefetch launch).
enum : int { ST_OK = 0, ST_TIMEOUT_FULL = 1, ST_TIMEOUT_EMPTY = 2, ST_TIMEOUT_MMA = 3, ST_TIMEOUT_TMEM = 4,
             ST_ITEMS_OVERFLOW = 5, ST_TIMEOUT_PEER = 6 };
constexpr int kStatusLimitWord = 2, kStatusSinkWord = 8, kStatusPlanWord = 16;

constexpr int kMaxParts = 16;   // most partial-sum buffers in one window
constexpr int kHeadDim = 128;

// ---- communication-window stand-in: h = resid + sum_p part_p ; x = RMSNorm(h) * gain
struct WindowArgs {
    const void *parts[kMaxParts];  // bf16 [B,H] each (parts[0] fp32 when part0_is_f32)
    int n_parts;
    int part0_is_f32;
    const void *resid;             // bf16 [B,H] or fp32 [B,H]
    int resid_is_f32;
    const void *gain;              // bf16 [H]
    float eps;
    float *h_f32;                  // optional fp32 [B,H]
    void *h_bf16;                  // optional bf16 [B,H]
    void *x_bf16;                  // bf16 [2][rows][H]: hi plane then lo plane (x = hi + lo); with x_fp16: fp16 [rows][H]
    int x_fp16;
    size_t x_plane_elems;          // elements between the planes
    int B, H;
    long long *trace;              // optional timeline slot (kTraceSlots values), see common.cuh
    int delay_ns;                  // modelled communication latency added to the window (0 = none)
    int *status;                   // device status block (bounded waits report here)
    int pdl;                       // launch with the programmatic-serialization attribute
    int inputs_after_wait;         // the step's input buffers may still be written by an earlier kernel of the
                                   // same call: read them only after the dependency wait
    int inject;                    // test hook (Inject)
    // Real communication window (one process per GPU): parts[] are the ranks' exchange buffers in rank
    // order (peer-mapped pointers, this rank's own included), all bf16.  After the dependency wait
    // the kernel tells every peer that this rank's buffer is complete, waits (bounded) until every
    // peer has said the same, and only then reads.  comm_rank < 0: no communication.
    int comm_rank;
    int comm_window;                       // 0 / 1: which of the layer's two windows (selects the flag row)
    const uint32_t *comm_flags_local;      // this rank's flag block: uint32 [2][kMaxParts]
    uint32_t *comm_flags_peer[16];         // every rank's flag block, by rank
    uint32_t *comm_epoch;                  // this rank's count of completed windows of this kind (device)
    unsigned *comm_done;                   // CTA ticket of the launch (device)
};
cudaError_t launch_window(const WindowArgs &a, cudaStream_t s);

// ---- skinny GEMM epilogues (shared by the GEMV and the tcgen05 paths)
enum Epilogue : int { EPI_PLAIN = 0, EPI_QKV = 1, EPI_SWIGLU = 2 };
struct EpilogueArgs {
    int kind;
    void *out;            // PLAIN: bf16 [B,N]; SWIGLU: split bf16 [2][rows][N/2]
    size_t out_plane;     // SWIGLU: elements between the hi and lo planes of out
    int out_fp16;         // SWIGLU: out is ONE fp16 plane [rows][N/2] (clamped to +-65504) instead of split bf16
    void *out2;           // PLAIN: optional second copy of the output (bf16 [B,N])
    float *out_f32;       // PLAIN: optional unrounded copy (fp32 [B,N])
    // QKV: rows are heads [q | k | v] x head_dim; rotary embedding on q and k, k/v appended
    void *q_out;          // split bf16 [2][rows][nq,d]
    size_t q_plane;       // elements between the hi and lo planes of q_out
    void *k_cache;        // bf16 [*,nkv,cap,d]
    void *v_cache;
    const int *ctx_len;   // device [B]
    int nq, nkv, cap;
    const double *inv_freq;  // device [d/2]: theta^(-2i/d); NULL disables the rotary embedding
    float *kv_new;        // int8 cache: the new k and v go here as fp32 ([2][max_batch*nkv][d], planes kv_new_plane
    size_t kv_new_plane;  // elements apart) instead of into k_cache / v_cache; NULL: bf16 cache
};

// Packing kinds: how logical output features map to packed rows.
//   GEMV path  : 16-row blocks; row r<8 and row r+8 of a block form an epilogue pair.
//   tensor path: rows 2m and 2m+1 form a pair.
// PLAIN has no pairing (identity order).  The packers and the epilogues agree through
// packed_row_to_feature() in pack.cu / epilogue.cuh.
cudaError_t launch_pack_gemv(const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind,
                             void *dst, int to_fp16, cudaStream_t s);
cudaError_t launch_pack_rows(const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind,
                             void *dst, int to_fp16, cudaStream_t s);
// int8 weights for the GEMV path: symmetric per-output-channel quantisation (scale = max |w| / 127 of the
// output feature's column, code = round-to-nearest-even(w / scale), both in fp32), codes in fragment-major
// 1 KiB tiles of 16 rows x 64 k, scales [N] in packed row order.
cudaError_t launch_pack_gemv_w8(const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind,
                                void *dst_codes, float *dst_scales, cudaStream_t s);
// the same codes and scales for the tensor path, rows in the tensor path's order: the codes, biased by 128
// (unsigned bytes), in contiguous blocks of (tiles * 128 rows) x 128 k, block (row tile, k block) at
// ((row tile) * K / 128 + k block) * tiles * 16384 - a CTA's stream of k blocks is one contiguous run; inside a
// row the eight 16-byte groups are permuted by the row index (pack.cu)
cudaError_t launch_pack_rows_w8(const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind,
                                void *dst_codes, float *dst_scales, int tiles, cudaStream_t s);

// ---- split-K GEMV (batch < 16): y[b,n] = sum_k x[b,k] W[n,k]; W in fragment-major tiles
struct GemvArgs {
    const void *w;        // packed weights (N*K bf16)
    const void *x;        // split bf16 [2][rows][K]
    size_t x_plane;       // elements between the hi and lo planes
    int B, N, K;          // B <= 16 batch rows starting at b0
    int b0;
    EpilogueArgs epi;
    int *status;
    long long *trace;
    const void *next_w;   // optional: weights of the kernel that follows, prefetched to L2 once this one has streamed its own
    size_t next_bytes;
    int pdl;
    int inject;
    int w8;               // the weights are int8 codes (1 KiB tiles of 16 rows x 64 k) with one fp32 scale per packed row
    const float *scales;  // w8: [N] in packed row order
};
cudaError_t launch_gemv(const GemvArgs &a, int sm_count, cudaStream_t s);

// ---- tcgen05 skinny GEMM (batch >= 16): W [N,K] K-major through TMA
struct GemmTcArgs {
    CUtensorMap w_map;    // dims (K, N), box (64, 128), 128B swizzle
    const CUtensorMap *w_map256;  // optional: same tensor with box (64, 256), for two weight tiles per CTA
    CUtensorMap x_map;    // dims (K, 2*NB): hi rows then lo rows; box (64, 2*NB), 128B swizzle - or, with x_fp16,
                          // dims (K, NB): one fp16 plane, box (64, NB)
    int x_fp16;           // 0: two bf16 planes; 2: two fp16 planes (hi rows then lo rows); 1: the activations are one fp16 plane (inputs that come out of an RMSNorm: bounded,
                          // 11 significant bits suffice) instead of bf16 hi + lo planes
    int B, NB, N, K;      // NB = batch rows per plane (multiple of 16)
    EpilogueArgs epi;
    int *status;
    long long *trace;
    int pdl;
    int inject;
    // int8 weights: the codes come from w8_codes by plain bulk copies (w_map / w_map256 are unused); the
    // kernel widens every tile to the activations' 16-bit format into tensor memory (the MMA's A operand)
    // and multiplies every accumulator row by its scale
    int w8;
    const float *scales;  // w8: [N] in packed row order
    const void *w8_codes; // w8: the packed codes (launch_pack_rows_w8 with gemm_tc_w8_tiles() rows per block)
};
// int8 weights: 128-row weight tiles per CTA for a matrix of N rows and a padded batch of NB (the packed
// layout depends on it)
int gemm_tc_w8_tiles(int NB, int N, int x_fp16);
cudaError_t launch_gemm_tc(const GemmTcArgs &a, int sm_count, cudaStream_t s);

// ---- split-KV decode attention + merge
struct AttnArgs {
    CUtensorMap k_map;    // dims (d, max_batch*nkv*cap), box (64, 64), 128B swizzle
    CUtensorMap v_map;
    const void *q;        // split bf16 [2][rows][nq,d]
    size_t q_plane;
    const int *ctx_len;   // device [B]; keys attended = ctx_len[b] + 1
    int B, nq, nkv, cap;
    int grid;             // persistent CTAs
    int tiles_per_item;   // 64-key tiles per work item
    int max_items;        // capacity of the partial buffers
    float *part_o;        // fp32 [max_items, G, d]: one partial per work item
    float *part_ml;       // fp32 [max_items, G, 2]
    int max_items_per_stream;   // work items of the longest sequence (sizes the merge CTAs)
    void *o_out;          // split bf16 [2][rows][nq,d]
    size_t o_plane;
    int o_fp16;           // o_out is ONE fp16 plane [rows][nq,d] instead
    int *status;
    cudaEvent_t mid_event; // optional: recorded between the split-KV kernel and the merge kernel
    int phases;            // bit 0: split-KV kernel, bit 1: merge kernel (0 = both)
    long long *trace;      // optional: two consecutive timeline slots (split-KV, merge)
    int pdl;
    int inject;
    // int8 cache (kv8 != 0): k_map / v_map are uint8 maps with dims (d, max_batch*nkv*cap), box (128, 64);
    // one fp32 scale per cached vector in k_scale / v_scale [max_batch*nkv][scale_cap] (scale_cap a
    // multiple of 64); the step's new key and value arrive as fp32 vectors in kv_new ([2][max_batch*nkv][d],
    // written by the QKV projection) and the kernel stores their codes and scales into the cache.
    int kv8;
    float *k_scale, *v_scale;
    void *k_codes, *v_codes;
    int scale_cap;
    const float *kv_new;
    size_t kv_new_plane;
};
cudaError_t launch_attention(const AttnArgs &a, cudaStream_t s);
// the int8-cache split-KV kernel alone (attn_kv8.cu); launch_attention adds the merge kernel
cudaError_t launch_attention_kv8_kernel(const AttnArgs &a, const cudaLaunchConfig_t &base_cfg);
int attention_kv8_stages();
// Grid size (persistent CTAs) and tiles per work item for the given sequence lengths (host array);
// depends only on the lengths and the SM count.
// `stages` = tiles the kernel's ring holds (3 for the bf16 cache, attention_kv8_stages() for int8);
// `item_cost` = what starting an item, combining and writing its partial costs, in tile times (an int8
// tile streams in half the time, so the same fixed work weighs twice as much).
void plan_attention(const int32_t *ctx_len_host, int batch, int nkv, int sm_count, int *grid, int *tiles_per_item,
                    int stages = 3, double item_cost = 1.5);
// 2-D uint8 tensor map (rows x cols bytes, cols contiguous), box (box_cols x box_rows), 128-byte swizzle.
bool encode_u8_map_2d(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint32_t box_cols,
                      uint32_t box_rows);

// 2-D bf16 tensor map (rows x cols, cols contiguous), box (box_cols x box_rows), 128-byte swizzle.
bool encode_bf16_map_2d(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint32_t box_cols,
                        uint32_t box_rows);

// ---- L2 prefetch (no arithmetic on the data).  The launch carries one window's node list in
// breadth-first order and the budget; the kernel evaluates Algorithm 1 itself with the live
// sequence lengths, so the arguments do not change from step to step of a decode loop.
constexpr int kPfMaxNodes = 6;
struct PrefetchNode {
    const void *base;     // weights: the contiguous packed matrix; SelfAttention: the K cache
    const void *base2;    // SelfAttention: the V cache
    uint64_t bytes;       // weights: the node's memSize; unused for the SelfAttention node
};
struct PrefetchArgs {
    PrefetchNode node[kPfMaxNodes];
    int n_nodes;
    int kv_node;            // index of the SelfAttention node in node[], or -1
    int kv_count;           // (sequence, kv head) runs
    int kv_ranges_per_seq;  // kv heads per sequence: run i belongs to sequence i / kv_ranges_per_seq
    int kv_token_bytes;     // bytes per cached token per run (head_dim * 2)
    uint64_t kv_stride;     // bytes between consecutive runs
    uint64_t budget;        // Algorithm 1's C for this window
    int plan_mode;          // PRESERVE_PLAN_*
    int mechanism;          // 0 bulk L2 prefetch, 1 per-line hints, 2 plain loads
    uint32_t chunk;         // bytes per prefetch instruction / per thread visit (multiple of 128)
    const int *ctx_len;     // device [sequences]
    int *sink;              // scratch word for the load variant (practically never written)
    unsigned long long *plan_out;   // optional: device uint64[kPfMaxNodes], receives the bytes taken per node
};
// ---- exchange memory of the real communication window (comm.cu)
struct CommView {
    int rank, n_ranks;
    uint8_t *buf[kMaxParts];      // every rank's exchange buffer of one window, by rank (peer-mapped)
    uint32_t *flags[kMaxParts];   // every rank's flag block
    uint32_t *epoch;              // own counters of that window
    unsigned *done;
};
}  // namespace prsv
struct preserve_comm;
namespace prsv {
bool comm_fill(const preserve_comm *c, int window, CommView *v);   // false until every peer is connected
int comm_hidden(const preserve_comm *c);
int comm_max_batch(const preserve_comm *c);

// ---- Algorithm 1 over an explicit operator graph (planner.cu; host only).  Successors in CSR form.
struct PlanHit { int comm, node; uint64_t bytes; };      // prefetch `bytes` of `node` beside communication op `comm`
int plan_graph(int n_nodes, const int32_t *kind, const uint64_t *mem_bytes, const int32_t *succ_off,
               const int32_t *succ, uint64_t budget, int mode, std::vector<PlanHit> &out);

// ---- host-buffer entry point: gather of pinned host buffers (device views) into device memory
cudaError_t launch_stage_inputs(const void *const *src, void *const *dst, int n, size_t bytes_each, const int *ctx_src,
                                int *ctx_dst, int n_ctx, cudaStream_t s);

cudaError_t launch_prefetch(const PrefetchArgs &a, int ctas, cudaStream_t s, const cudaLaunchAttribute *attrs,
                            int n_attrs);

}  // namespace prsv
