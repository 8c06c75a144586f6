// Internal launch interface between the layer runtime (api.cu) and the kernels.
// Every launcher is asynchronous on the given stream and returns the launch's
// cudaError_t.  No launcher allocates.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace prsv {

// Programmatic dependent launch: when non-zero, every kernel of the main stream is
// launched with the programmatic-serialization attribute, so its prologue (index
// setup, first weight loads) may overlap the previous kernel's tail.  Each kernel
// executes griddepcontrol.wait before it touches anything another kernel wrote.
extern int g_pdl;
inline int pdl_attr(cudaLaunchAttribute *at)
{
    if (!g_pdl)
        return 0;
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    return 1;
}

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
    void *x_bf16;                  // bf16 [2][rows][H]: hi plane then lo plane (x = hi + lo)
    size_t x_plane_elems;          // elements between the planes
    int B, H;
    long long *trace;              // optional timeline slot (kTraceSlots values), see common.cuh
    int delay_ns;                  // modelled communication latency added to the window (0 = none)
    int *status;                   // device error word (bounded waits report here)
};
cudaError_t launch_window(const WindowArgs &a, cudaStream_t s);

// ---- skinny GEMM epilogues (shared by the GEMV and the tcgen05 paths)
enum Epilogue : int { EPI_PLAIN = 0, EPI_QKV = 1, EPI_SWIGLU = 2 };
struct EpilogueArgs {
    int kind;
    void *out;            // PLAIN: bf16 [B,N]; SWIGLU: split bf16 [2][rows][N/2]
    size_t out_plane;     // SWIGLU: elements between the hi and lo planes of out
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
};

// Packing kinds: how logical output features map to packed rows.
//   GEMV path  : 16-row blocks; row r<8 and row r+8 of a block form an epilogue pair.
//   tensor path: rows 2m and 2m+1 form a pair.
// PLAIN has no pairing (identity order).  The packers and the epilogues agree through
// packed_row_to_feature() in pack.cu / epilogue.cuh.
cudaError_t launch_pack_gemv(const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind,
                             void *dst, cudaStream_t s);
cudaError_t launch_pack_rows(const void *const *srcs, const int *src_cols, int n_srcs, int K, int kind,
                             void *dst, cudaStream_t s);

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
};
cudaError_t launch_gemv(const GemvArgs &a, int sm_count, cudaStream_t s);

// ---- tcgen05 skinny GEMM (batch >= 16): W [N,K] K-major through TMA
struct GemmTcArgs {
    CUtensorMap w_map;    // dims (K, N), box (64, 128), 128B swizzle
    const CUtensorMap *w_map256;  // optional: same tensor with box (64, 256), for two weight tiles per CTA
    CUtensorMap x_map;    // dims (K, 2*NB): hi rows then lo rows; box (64, 2*NB), 128B swizzle
    int B, NB, N, K;      // NB = batch rows per plane (multiple of 16)
    EpilogueArgs epi;
    int *status;
    long long *trace;
};
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
    int *status;
    cudaEvent_t mid_event; // optional: recorded between the split-KV kernel and the merge kernel
    int phases;            // bit 0: split-KV kernel, bit 1: merge kernel (0 = both)
    long long *trace;      // optional: two consecutive timeline slots (split-KV, merge)
};
cudaError_t launch_attention(const AttnArgs &a, cudaStream_t s);
// Grid size (persistent CTAs) and tiles per work item for the given sequence lengths (host array);
// depends only on the lengths and the SM count.
void plan_attention(const int32_t *ctx_len_host, int batch, int nkv, int sm_count, int *grid, int *tiles_per_item);

// 2-D bf16 tensor map (rows x cols, cols contiguous), box (box_cols x box_rows), 128-byte swizzle.
bool encode_bf16_map_2d(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint32_t box_cols,
                        uint32_t box_rows);

// ---- L2 prefetch (no arithmetic, writes nothing)
struct PrefetchSeg {
    const void *base;     // contiguous range, or the K cache when per_seq_tokens != 0
    const void *base2;    // the V cache when per_seq_tokens != 0
    uint64_t stride;      // KV: bytes between consecutive (sequence, kv head) runs
    uint64_t bytes;       // bytes to prefetch from this segment (the planner's figure)
    int count;            // KV: number of (sequence, kv head) runs
    int per_seq_tokens;   // != 0: KV segment; run i holds ctx_len[i / ranges_per_seq] live tokens
    int ranges_per_seq;   // KV heads per sequence
    int token_bytes;      // bytes per token per run (head_dim * 2)
};
struct PrefetchArgs {
    PrefetchSeg seg[6];
    int n_segs;
    const int *ctx_len;
    int *sink;            // scratch word for the load variant (practically never written)
};
// ---- host-buffer entry point: gather of pinned host buffers (device views) into device memory
cudaError_t launch_stage_inputs(const void *const *src, void *const *dst, int n, size_t bytes_each, const int *ctx_src,
                                int *ctx_dst, int n_ctx, cudaStream_t s);

void set_prefetch_kernel_mode(int mode, uint32_t chunk_bytes);
cudaError_t launch_prefetch(const PrefetchArgs &a, int ctas, cudaStream_t s, const cudaLaunchAttribute *attrs,
                            int n_attrs);

}  // namespace prsv
