// Layer runtime and C ABI: weight arena, workspaces, the prefetch planner
// (Algorithm 1 over the layer's fixed operator list), the two-stream schedule
// (Section 3, "PRESERVE": prefetch operators run in a stream parallel to the main
// stream and are ordered by events) and CUDA-graph replay of whole steps.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/preserve.h"
#include "kernels.h"

using namespace prsv;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 tensor map: `rows` rows of `cols` contiguous elements, box (box_cols x box_rows), 128-byte swizzle.
bool make_map_2d(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint32_t box_cols, uint32_t box_rows)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn)
        return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D uint8 tensor map: `rows` rows of `cols` contiguous bytes, box (box_cols x box_rows), 128-byte swizzle.
bool make_u8_map_2d(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint32_t box_cols, uint32_t box_rows)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn)
        return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A replayable graph and everything its kernel nodes were captured with: a cached graph is
// reused only when the whole signature matches word for word (no bare hash).
struct GraphEntry {
    std::vector<uint64_t> sig;
    cudaGraphExec_t exec;
    uint64_t stamp;
};
constexpr size_t kMaxCachedGraphs = 32;

}  // namespace

namespace prsv {
bool encode_bf16_map_2d(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint32_t box_cols,
                        uint32_t box_rows)
{
    return make_map_2d(m, base, cols, rows, box_cols, box_rows);
}
bool encode_u8_map_2d(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint32_t box_cols,
                      uint32_t box_rows)
{
    return make_u8_map_2d(m, base, cols, rows, box_cols, box_rows);
}
}  // namespace prsv

struct preserve_layer {
    preserve_layer_config_t cfg;
    int dev, sm_count, l2_bytes, max_persist, max_window;
    bool tensor_path;
    int group;

    uint8_t *arena;              // packed weights: Wqkv | Wo | Wgate,up | Wdown, then gains
    size_t arena_bytes;
    size_t off[4];
    uint64_t wbytes[4];
    void *g_attn, *g_mlp;
    double *inv_freq;
    bool w8;                     // int8 weights (GEMV path): arena holds codes, `scales` one fp32 per packed row
    float *scales;
    size_t soff[4];
    bool kv8;                    // int8 KV-cache: codes then scales in each cache buffer (preserve_kv8_layout)
    float *kv_new;               // kv8: the step's new key and value, fp32 [2][max_batch * n_kv][d] (QKV projection ->
                                 // attention, which quantises them into the cache)
    uint64_t kv8_scale_off;      // byte offset of the scales inside a cache buffer
    int kv8_scale_cap;           // scales per (sequence, kv head): capacity rounded up to 64

    float *h_f32;                              // window A sum (residual for window B)
    float *attn_f32, *h2_f32, *mlp_f32;        // unrounded copies: own attention partial (window B input),
                                               // and the two outputs (handed to the next layer of a linked chain)
    void *x, *q, *o, *x2, *a;                  // split bf16 [2][rows][...] (hi + lo)
    int rows;                                  // batch rows per plane (max_batch, padded to 16 on the tensor path)
    float *part_o, *part_ml;
    int max_items;
    int *status;

    // staging for the host-buffer entry point
    uint8_t *stage_in, *stage_out;
    int *ctx_dev;

    // tensor path
    CUtensorMap wmap[4];
    CUtensorMap wmap256[4];      // box of 256 rows (valid when has256[i])
    bool has256[4];
    CUtensorMap xmap[4];         // x, o, x2, a as B operands
    int nb_pad;

    // K/V maps (re-encoded when the cache pointers change)
    const void *k_ptr, *v_ptr;
    CUtensorMap k_map, v_map;

    cudaStream_t side;
    cudaEvent_t ev_a, ev_b, ev_join;
    cudaStream_t xfer;           // host-buffer entry point: the stream the input gather runs on
    cudaEvent_t ev_in_ready, ev_in_free;
    bool in_free_valid;
    bool side_pending;           // prefetch work queued on the side stream and not yet joined
    bool no_early;               // ablation: prefetch into L2 only, no early launch of the consumer kernels
    int window_delay_ns;         // modelled extra duration of each communication window
    int pf_mechanism;            // prefetch kernel: 0 bulk L2 prefetch, 1 per-line hints, 2 plain loads
    uint32_t pf_chunk;           // bytes per prefetch instruction
    int inject;                  // test hook (prsv::Inject): one producer withholds one issue
    preserve_comm *comm;         // real communication window (NULL: the local stand-in)
    const void *ext_attn_sum;    // window B's partial 0 comes from this caller-reduced buffer instead of the own result
    uint64_t n_captures;         // graphs captured so far by calls whose first layer is this handle

    size_t budget;
    int plan_mode;
    uint64_t planned[2][3];
    uint64_t kv_bytes, alg_bytes;
    int last_cuda;
    int prefetch_ctas;

    std::vector<GraphEntry> graphs;
    uint64_t stamp;
    bool budget_is_default;      // preserve_set_prefetch_bytes has not been called: the library picks per path

    // per-kernel timing (preserve_profile_step): events around the main-stream kernels
    long long *trace_buf;        // device [PRESERVE_N_KERNELS][PRESERVE_TRACE_SLOTS] timeline slots, used when tracing
    bool tracing;
    int only;                    // >= 0: enqueue_step launches only this kernel (preserve_run_kernel)
    bool profiling;
    cudaEvent_t prof[PRESERVE_N_KERNELS + 1];
};

namespace {

int cuda_fail(preserve_layer *L, cudaError_t e)
{
    if (L)
        L->last_cuda = (int)e;
    (void)cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? PRESERVE_ENOMEM : PRESERVE_ECUDA;
}

#define CK(L, expr)                                \
    do {                                           \
        cudaError_t e__ = (expr);                  \
        if (e__ != cudaSuccess)                    \
            return cuda_fail((L), e__);            \
    } while (0)

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int validate_config(const preserve_layer_config_t *c)
{
    if (c->head_dim != kHeadDim)
        return PRESERVE_ESHAPE;
    if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads || c->n_q_heads / c->n_kv_heads > 16)
        return PRESERVE_ESHAPE;
    if (c->hidden < 128 || c->hidden % 128 || c->hidden > 16384)
        return PRESERVE_ESHAPE;
    if (c->max_batch < 1 || c->max_batch > 128)
        return PRESERVE_ESHAPE;
    if (c->ffn < 32 || c->ffn % 32 || (c->max_batch >= 16 && c->ffn % 128))
        return PRESERVE_ESHAPE;
    if (c->tp_degree < 1 || c->tp_degree > kMaxParts)
        return PRESERVE_ESHAPE;
    if (c->max_ctx < 0 || (long long)c->max_batch * c->n_kv_heads > 2048)
        return PRESERVE_ESHAPE;
    if ((long long)c->max_batch * c->n_kv_heads * ((long long)c->max_ctx + 1) > 0x7fffffffll)
        return PRESERVE_ESHAPE;
    if (c->flags & PRESERVE_FLAG_INT8_WEIGHTS) {
        // the GEMV path's int8 tiles (1 KiB) cover 64 k
        if (c->ffn % 64)
            return PRESERVE_ESHAPE;
    }
    if (c->flags & PRESERVE_FLAG_INT8_KV) {
        // the int8-cache attention kernel takes groups of at most 8 query heads per KV head
        if (c->n_q_heads / c->n_kv_heads > 8)
            return PRESERVE_ESHAPE;
    }
    return PRESERVE_OK;
}

// Layout of one int8 cache buffer: codes [max_batch, n_kv, cap, d] int8, then (256-byte aligned) one
// fp32 scale per cached vector [max_batch, n_kv, scale_cap], scale_cap = cap rounded up to 64.
void kv8_layout(const preserve_layer_config_t &c, uint64_t *scale_off, int *scale_cap, uint64_t *total)
{
    const uint64_t streams = (uint64_t)c.max_batch * c.n_kv_heads, cap = (uint64_t)c.max_ctx + 1;
    const uint64_t codes = streams * cap * (uint64_t)c.head_dim;
    const uint64_t off = (codes + 255) & ~uint64_t(255);
    const uint64_t scap = (cap + 63) & ~uint64_t(63);
    *scale_off = off;
    *scale_cap = (int)scap;
    *total = off + streams * scap * 4;
}

struct Dims {
    int n[4], k[4];
};
Dims layer_dims(const preserve_layer_config_t &c)
{
    Dims d;
    d.n[0] = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim; d.k[0] = c.hidden;
    d.n[1] = c.hidden;                                      d.k[1] = c.n_q_heads * c.head_dim;
    d.n[2] = 2 * c.ffn;                                     d.k[2] = c.hidden;
    d.n[3] = c.hidden;                                      d.k[3] = c.ffn;
    return d;
}

// bytes of weight matrix i as the kernels stream it: bf16, or int8 codes (their fp32 scales, one per
// output feature, are 4 / K of that and not counted)
uint64_t weight_bytes(const preserve_layer_config_t &c, const Dims &d, int i)
{
    return (uint64_t)d.n[i] * d.k[i] * ((c.flags & PRESERVE_FLAG_INT8_WEIGHTS) ? 1 : 2);
}

uint64_t activation_bytes(const preserve_layer_config_t &c, int B)
{
    const bool kv8 = (c.flags & PRESERVE_FLAG_INT8_KV) != 0;
    const uint64_t BH = (uint64_t)B * c.hidden * 2, Bq = (uint64_t)B * c.n_q_heads * c.head_dim * 2;
    const uint64_t Bkv = (uint64_t)B * c.n_kv_heads * c.head_dim * 2, BF = (uint64_t)B * c.ffn * 2;
    const uint64_t gain = (uint64_t)c.hidden * 2, P = c.tp_degree;
    uint64_t t = 0;
    t += (P + 1) * BH + gain + 2 * BH;   // window A: reads, gain, writes h and x
    t += BH + Bq;                        // QKV: reads x, writes q ...
    if (!kv8)
        t += 2 * Bkv;                    // ... and appends k and v
    else                                 // ... leaves k and v as fp32 (write, read), attention stores codes and scales
        t += 2 * (2 * Bkv + 2 * Bkv) + Bkv + 2 * (uint64_t)B * c.n_kv_heads * 4;
    t += Bq + Bq;                        // attention: reads q, writes o
    t += Bq + BH;                        // O: reads o, writes the attention partial
    t += (P + 1) * BH + gain + 2 * BH;   // window B
    t += BH + BF;                        // gate/up: reads x2, writes a
    t += BF + BH;                        // down: reads a, writes the MLP partial
    return t;
}

void plan_window(const uint64_t *node_bytes, int n, uint64_t budget, int mode, uint64_t *out)
{
    // Algorithm 1 for one communication op whose successors, in breadth-first order, are the
    // given MatMul / SelfAttention nodes followed by the next communication op.
    uint64_t cache_sum = 0;
    for (int i = 0; i < n; ++i)
        out[i] = 0;
    for (int i = 0; i < n; ++i) {
        if (cache_sum + node_bytes[i] < budget) {       // strict: a node that makes cacheSum reach C is not inserted (Algorithm 1)
            cache_sum += node_bytes[i];
            out[i] = node_bytes[i];
        } else {
            if (mode == PRESERVE_PLAN_TRUNCATE) {
                const uint64_t room = budget > cache_sum ? budget - cache_sum : 0;
                uint64_t part = room & ~uint64_t(127);
                if (part > node_bytes[i])
                    part = node_bytes[i];
                out[i] = part;
            }
            break;                                      // end of the walk for this op
        }
    }
}

// ------------------------------------------------------------------ one step
struct StepPtrs {
    int batch;
    const int *ctx_len;
    const int *ctx_len_host;
    const void *parts[kMaxParts];
    const void *peers[kMaxParts];
    const void *residual_in;
    int resid_f32, part0_f32;      // linked chain: residual_in / parts[0] are the previous layer's fp32 copies
    void *k_cache, *v_cache;
    void *residual_out, *mlp_partial_out, *attn_partial_out;
    int late_a, late_b;            // an input of window A / B is an output of an earlier layer of the same call:
                                   // the window reads its inputs only after the dependency wait
    int first_of_call;             // first layer of a call
};

// What the host decides for one step before anything is queued (Algorithm 1 per window over the
// layer's fixed operator list, the attention work split): everything the launches depend on besides
// the pointers.  Nothing here depends on the VALUES of the sequence lengths except through these
// few derived numbers, so a decode loop whose contexts advance keeps replaying one graph.
struct StepPlan {
    uint64_t planned[2][3];
    uint64_t kv_bytes, alg_bytes;
    bool pf_a, pf_b;
    int pdl;
    int attn_grid, attn_tpi, attn_items_per_stream;
};

int check_step(preserve_layer *L, const preserve_step_io_t *io, StepPtrs *sp)
{
    if (!L || !io)
        return PRESERVE_EINVAL;
    const auto &c = L->cfg;
    if (io->batch < 1 || io->batch > c.max_batch)
        return PRESERVE_ESHAPE;
    if (!io->ctx_len || !io->ctx_len_host || !io->partials_in || !io->residual_in || !io->k_cache || !io->v_cache ||
        !io->residual_out || !io->mlp_partial_out)
        return PRESERVE_EINVAL;
    if (c.tp_degree > 1 && !io->attn_peer_partials)
        return PRESERVE_EINVAL;
    sp->batch = io->batch;
    sp->ctx_len = io->ctx_len;
    sp->ctx_len_host = io->ctx_len_host;
    for (int i = 0; i < c.tp_degree; ++i) {
        if (!io->partials_in[i])
            return PRESERVE_EINVAL;
        if (!aligned16(io->partials_in[i]))
            return PRESERVE_EALIGN;
        sp->parts[i] = io->partials_in[i];
    }
    for (int i = 0; i + 1 < c.tp_degree; ++i) {
        if (!io->attn_peer_partials[i])
            return PRESERVE_EINVAL;
        if (!aligned16(io->attn_peer_partials[i]))
            return PRESERVE_EALIGN;
        sp->peers[i] = io->attn_peer_partials[i];
    }
    const void *ptrs[] = {io->residual_in, io->k_cache, io->v_cache, io->residual_out, io->mlp_partial_out,
                          io->attn_partial_out};
    for (const void *p : ptrs)
        if (p && !aligned16(p))
            return PRESERVE_EALIGN;
    if (reinterpret_cast<uintptr_t>(io->ctx_len) & 3)
        return PRESERVE_EALIGN;
    for (int b = 0; b < io->batch; ++b)
        if (io->ctx_len_host[b] < 0 || io->ctx_len_host[b] > c.max_ctx)
            return PRESERVE_ESHAPE;
    sp->residual_in = io->residual_in;
    sp->k_cache = io->k_cache;
    sp->v_cache = io->v_cache;
    sp->residual_out = io->residual_out;
    sp->mlp_partial_out = io->mlp_partial_out;
    sp->attn_partial_out = io->attn_partial_out;
    return PRESERVE_OK;
}

int launch_gemm(preserve_layer *L, int which, const void *x, int B, const EpilogueArgs &epi, int pdl, cudaStream_t s,
                long long *trace)
{
    const Dims d = layer_dims(L->cfg);
    if (L->tensor_path) {
        GemmTcArgs a = {};
        a.w_map = L->wmap[which];
        a.w_map256 = L->has256[which] ? &L->wmap256[which] : nullptr;
        a.x_map = L->xmap[which];
        (void)x;
        a.B = B; a.NB = L->nb_pad; a.N = d.n[which]; a.K = d.k[which];
        a.epi = epi;
        a.status = L->status;
        a.trace = trace;
        a.pdl = pdl;
        a.inject = L->inject == INJECT_TC_RING && which == 0 ? INJECT_TC_RING : INJECT_NONE;
        // The gate/up projection takes its input as one fp16 plane (an RMSNorm output is bounded, and 11
        // significant bits keep the SwiGLU output well inside the tolerance): half the activation
        // traffic and half the MMA work of the largest GEMM.  The QKV projection keeps two planes, hi + lo
        // (fp16 each, its weights stored as fp16 like the others: with int8 weights the codes then take the
        // cheap fp16 widening): rounding of q is amplified by the softmax (measured: one fp16 plane put the
        // 70B-shaped chain's attention partial sums at 1.02 of the bound).
        a.x_fp16 = which >= 1 ? 1 : 2;
        a.w8 = L->w8 ? 1 : 0;
        a.scales = L->w8 ? L->scales + L->soff[which] : nullptr;
        a.w8_codes = L->w8 ? L->arena + L->off[which] : nullptr;
        CK(L, launch_gemm_tc(a, L->sm_count, s));
        return PRESERVE_OK;
    }
    for (int b0 = 0; b0 < B; b0 += 16) {
        GemvArgs a;
        a.w = L->arena + L->off[which];
        a.x = x;
        a.x_plane = (size_t)L->rows * d.k[which];
        a.B = B - b0 < 16 ? B - b0 : 16;
        a.b0 = b0;
        a.N = d.n[which]; a.K = d.k[which];
        a.epi = epi;
        a.status = L->status;
        a.trace = trace;
        a.pdl = pdl;
        a.inject = L->inject == INJECT_GEMV_RING && which == 0 ? INJECT_GEMV_RING : INJECT_NONE;
        a.w8 = L->w8 ? 1 : 0;
        a.scales = L->w8 ? L->scales + L->soff[which] : nullptr;
        a.next_w = nullptr;
        a.next_bytes = 0;
        // Prefetching on: the gate/up projection fills both CTA slots of most SMs, so most CTAs of the
        // down projection start only when it ends and would fetch their first tiles from idle HBM
        // after that; the gate/up CTAs request them into L2 as soon as their own stream is over.
        // (Not when a single kernel is run alone for timing: nothing would consume the bytes.)
        if (which == 2 && L->only == -1 && L->budget > 0 && !L->no_early && L->wbytes[3] <= L->l2_bytes / 4) {
            a.next_w = L->arena + L->off[3];
            a.next_bytes = (size_t)L->wbytes[3];
        }
        CK(L, launch_gemv(a, L->sm_count, s));
    }
    return PRESERVE_OK;
}

// Host planning of one step: Algorithm 1 per window over {Wqkv, KV, Wo} and {Wgate|up, Wdown}, the
// byte accounting, and the split of the attention work.
void plan_step(preserve_layer *L, const StepPtrs &sp, StepPlan *pl)
{
    const auto &c = L->cfg;
    const int B = sp.batch;
    uint64_t sum_ctx = 0, max_tiles_seq = 0;
    for (int b = 0; b < B; ++b) {
        sum_ctx += (uint64_t)sp.ctx_len_host[b];
        const uint64_t nt = (uint64_t)(sp.ctx_len_host[b] + 1 + 63) / 64;
        max_tiles_seq = nt > max_tiles_seq ? nt : max_tiles_seq;
    }
    // K and V bytes of the cached tokens: the SelfAttention node's memSize for Algorithm 1 (an int8
    // cache: the codes; its scales, 4 bytes per 128, are read too but not prefetched)
    pl->kv_bytes = 2 * sum_ctx * c.n_kv_heads * c.head_dim * (L->kv8 ? 1 : 2);
    // The layer's operator chain as Algorithm 1 sees it: window A -> Wqkv -> (rotary, append) ->
    // SelfAttention -> Wo -> window B -> Wgate|up -> (activation) -> Wdown -> next window.
    {
        static const int32_t kind[10] = {PRESERVE_NODE_COMM, PRESERVE_NODE_MATMUL, PRESERVE_NODE_OTHER,
                                         PRESERVE_NODE_ATTENTION, PRESERVE_NODE_MATMUL, PRESERVE_NODE_COMM,
                                         PRESERVE_NODE_MATMUL, PRESERVE_NODE_OTHER, PRESERVE_NODE_MATMUL,
                                         PRESERVE_NODE_COMM};
        static const int32_t succ_off[11] = {0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 9};
        static const int32_t succ[9] = {1, 2, 3, 4, 5, 6, 7, 8, 9};
        const uint64_t mem[10] = {0, L->wbytes[0], 0, pl->kv_bytes, L->wbytes[1], 0, L->wbytes[2], 0, L->wbytes[3], 0};
        static const int slot_of_node[10] = {-1, 0, -1, 1, 2, -1, 0, -1, 1, -1};
        std::vector<PlanHit> hits;
        plan_graph(10, kind, mem, succ_off, succ, L->budget, L->plan_mode, hits);
        memset(pl->planned, 0, sizeof(pl->planned));
        for (const PlanHit &h : hits)
            pl->planned[h.comm == 0 ? 0 : 1][slot_of_node[h.node]] = h.bytes;
    }
    pl->alg_bytes = L->wbytes[0] + L->wbytes[1] + L->wbytes[2] + L->wbytes[3] + pl->kv_bytes + activation_bytes(c, B);
    if (L->kv8)
        pl->alg_bytes += 2 * sum_ctx * c.n_kv_heads * 4;
    // budget 0 = vanilla execution: every kernel starts after its predecessor has completed and
    // nothing is fetched ahead of the dependency
    pl->pdl = (L->budget > 0 && !L->no_early) ? 1 : 0;
    // (only == -1: the whole step; -2 / -3: just the prefetch beside window A / B; k >= 0: just kernel k)
    pl->pf_a = (L->only == -1 || L->only == -2) && pl->planned[0][0] + pl->planned[0][1] + pl->planned[0][2] > 0;
    pl->pf_b = (L->only == -1 || L->only == -3) && pl->planned[1][0] + pl->planned[1][1] > 0;
    plan_attention(sp.ctx_len_host, B, c.n_kv_heads, L->sm_count, &pl->attn_grid, &pl->attn_tpi,
                   L->kv8 ? attention_kv8_stages() : 3, L->kv8 ? 3.0 : 1.5);
    pl->attn_items_per_stream = (int)((max_tiles_seq + pl->attn_tpi - 1) / pl->attn_tpi);
    // (the merge kernel sizes its CTAs from this, between 4 and 32 warps: clamp here so that the
    // number that enters the graph signature changes as rarely as the launch does)
    if (pl->attn_items_per_stream < 4) pl->attn_items_per_stream = 4;
    if (pl->attn_items_per_stream > 32) pl->attn_items_per_stream = 32;
}

// Queue one layer step on `s` (directly, or into an ongoing capture of `s`).
int enqueue_step(preserve_layer *L, const StepPtrs &sp, const StepPlan &pl, bool direct, cudaStream_t s)
{
    const auto &c = L->cfg;
    const int B = sp.batch, H = c.hidden, cap = c.max_ctx + 1;

    L->kv_bytes = pl.kv_bytes;
    L->alg_bytes = pl.alg_bytes;
    for (int w = 0; w < 2; ++w)
        for (int j = 0; j < 3; ++j)
            L->planned[w][j] = pl.planned[w][j];
    const int pdl = pl.pdl;
    const bool pf_a = pl.pf_a, pf_b = pl.pf_b;
#define WANT(k) (L->only == -1 || L->only == (k))
#define TRACE(k) (L->tracing ? L->trace_buf + PRESERVE_TRACE_SLOTS * (k) : nullptr)

    // ---- K/V tensor maps
    if (sp.k_cache != L->k_ptr || sp.v_cache != L->v_ptr) {
        const uint64_t rows = (uint64_t)c.max_batch * c.n_kv_heads * cap;
        const bool ok = L->kv8 ? make_u8_map_2d(&L->k_map, sp.k_cache, kHeadDim, rows, 128, 64) &&
                                     make_u8_map_2d(&L->v_map, sp.v_cache, kHeadDim, rows, 128, 64)
                               : make_map_2d(&L->k_map, sp.k_cache, kHeadDim, rows, 64, 64) &&
                                     make_map_2d(&L->v_map, sp.v_cache, kHeadDim, rows, 64, 64);
        if (!ok)
            return PRESERVE_EARCH;
        L->k_ptr = sp.k_cache;
        L->v_ptr = sp.v_cache;
    }

    int mark = 0;
#define MARK()                                                   \
    do {                                                         \
        if (L->profiling)                                        \
            CK(L, cudaEventRecord(L->prof[mark++], s));          \
    } while (0)

    // Optional: mark the prefetched weight range as persisting in L2 (access-policy window on the
    // prefetch kernel).  Only the weight arena can be covered (one contiguous window per launch).
    cudaLaunchAttribute pf_attr[1];
    auto persist_window = [&](size_t first_off, uint64_t bytes) -> int {
        if (!(c.flags & PRESERVE_FLAG_PERSIST_L2) || bytes == 0 || L->max_window <= 0)
            return 0;
        if (bytes > (uint64_t)L->max_window)
            bytes = (uint64_t)L->max_window;
        pf_attr[0].id = cudaLaunchAttributeAccessPolicyWindow;
        pf_attr[0].val.accessPolicyWindow.base_ptr = L->arena + first_off;
        pf_attr[0].val.accessPolicyWindow.num_bytes = (size_t)bytes;
        pf_attr[0].val.accessPolicyWindow.hitRatio = 1.0f;
        pf_attr[0].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
        pf_attr[0].val.accessPolicyWindow.missProp = cudaAccessPropertyStreaming;
        return 1;
    };
    auto prefetch_base = [&](int window) {
        PrefetchArgs pa = {};
        pa.ctx_len = sp.ctx_len;
        pa.sink = L->status + kStatusSinkWord;
        pa.plan_out = reinterpret_cast<unsigned long long *>(L->status + kStatusPlanWord) + 3 * window;
        pa.budget = L->budget;
        pa.plan_mode = L->plan_mode;
        pa.mechanism = L->pf_mechanism;
        pa.chunk = L->pf_chunk;
        pa.kv_node = -1;
        return pa;
    };

    // ---- window A  ||  prefetch {Wqkv, K/V, Wo}: the kernel walks the three nodes itself
    if (pf_a) {
        CK(L, cudaEventRecord(L->ev_a, s));
        CK(L, cudaStreamWaitEvent(L->side, L->ev_a, 0));
        PrefetchArgs pa = prefetch_base(0);
        pa.n_nodes = 3;
        pa.node[0].base = L->arena + L->off[0];
        pa.node[0].bytes = L->wbytes[0];
        pa.node[1].base = sp.k_cache;
        pa.node[1].base2 = sp.v_cache;
        pa.node[2].base = L->arena + L->off[1];
        pa.node[2].bytes = L->wbytes[1];
        pa.kv_node = 1;
        pa.kv_count = B * c.n_kv_heads;
        pa.kv_ranges_per_seq = c.n_kv_heads;
        pa.kv_token_bytes = kHeadDim * (L->kv8 ? 1 : 2);
        pa.kv_stride = (uint64_t)cap * kHeadDim * (L->kv8 ? 1 : 2);
        // Wqkv and Wo are adjacent in the arena
        const int na = persist_window(L->off[0], L->wbytes[0] + L->wbytes[1]);
        CK(L, launch_prefetch(pa, L->prefetch_ctas, L->side, na ? pf_attr : nullptr, na));
    }
    MARK();   // 0: window A starts
    if (WANT(0)) {
        WindowArgs w = {};
        for (int i = 0; i < c.tp_degree; ++i)
            w.parts[i] = sp.parts[i];
        w.n_parts = c.tp_degree;
        w.resid = sp.residual_in;
        w.resid_is_f32 = sp.resid_f32;
        w.part0_is_f32 = sp.part0_f32;
        w.gain = L->g_attn;
        w.eps = c.rms_eps;
        w.h_f32 = L->h_f32;
        w.h_bf16 = nullptr;
        w.x_bf16 = L->x;
        w.x_fp16 = L->tensor_path ? 2 : 0;
        w.x_plane_elems = (size_t)L->rows * H;
        w.B = B; w.H = H;
        w.trace = TRACE(0);
        w.delay_ns = L->window_delay_ns;
        w.status = L->status;
        // Launched directly, the first kernel of a call must not start before everything queued on
        // the stream earlier has finished: it reads its input buffers ahead of the dependency wait,
        // and an earlier call may still be writing them.  (Inside a graph the launch itself is
        // ordered after the earlier work.)
        w.pdl = pdl && !(direct && sp.first_of_call);
        w.inputs_after_wait = sp.late_a;
        w.inject = L->inject == INJECT_WINDOW_HANDOVER ? INJECT_WINDOW_HANDOVER : INJECT_NONE;
        w.comm_rank = -1;
        if (L->comm) {
            // the real window: the ranks' exchange buffers instead of the step's partial-sum inputs
            CommView cv;
            if (!comm_fill(L->comm, 0, &cv))
                return PRESERVE_EINVAL;
            for (int i = 0; i < cv.n_ranks; ++i) {
                w.parts[i] = cv.buf[i];
                w.comm_flags_peer[i] = cv.flags[i];
            }
            w.part0_is_f32 = 0;
            w.comm_rank = cv.rank;
            w.comm_window = 0;
            w.comm_flags_local = cv.flags[cv.rank];
            w.comm_epoch = cv.epoch;
            w.comm_done = cv.done;
        }
        CK(L, launch_window(w, s));
    }
    // ---- QKV projection + rotary embedding + KV append
    MARK();   // 1
    if (WANT(1)) {
        EpilogueArgs e = {};
        e.kind = EPI_QKV;
        e.q_out = L->q;
        e.q_plane = (size_t)L->rows * c.n_q_heads * kHeadDim;
        e.k_cache = sp.k_cache;
        e.v_cache = sp.v_cache;
        e.ctx_len = sp.ctx_len;
        e.nq = c.n_q_heads; e.nkv = c.n_kv_heads; e.cap = cap;
        e.inv_freq = c.rope_theta > 0.f ? L->inv_freq : nullptr;
        if (L->kv8) {
            e.kv_new = L->kv_new;
            e.kv_new_plane = (size_t)c.max_batch * c.n_kv_heads * kHeadDim;
        }
        int rc = launch_gemm(L, 0, L->x, B, e, pdl, s, TRACE(1));
        if (rc)
            return rc;
    }
    // ---- attention
    MARK();   // 2
    if (WANT(2) || WANT(3)) {
        AttnArgs a = {};
        a.phases = (WANT(2) ? 1 : 0) | (WANT(3) ? 2 : 0);
        a.mid_event = L->profiling ? L->prof[mark++] : nullptr;   // 3: merge starts
        a.k_map = L->k_map;
        a.v_map = L->v_map;
        a.q = L->q;
        a.q_plane = (size_t)L->rows * c.n_q_heads * kHeadDim;
        a.o_plane = a.q_plane;
        a.o_fp16 = L->tensor_path ? 1 : 0;
        a.ctx_len = sp.ctx_len;
        a.B = B; a.nq = c.n_q_heads; a.nkv = c.n_kv_heads; a.cap = cap;
        a.grid = pl.attn_grid;
        a.tiles_per_item = pl.attn_tpi;
        a.max_items_per_stream = pl.attn_items_per_stream;
        a.max_items = L->max_items;
        a.part_o = L->part_o;
        a.part_ml = L->part_ml;
        a.o_out = L->o;
        a.status = L->status;
        a.trace = TRACE(2);
        a.pdl = pdl;
        a.inject = L->inject == INJECT_ATTN_RING ? INJECT_ATTN_RING : INJECT_NONE;
        if (L->kv8) {
            a.kv8 = 1;
            a.k_codes = sp.k_cache;
            a.v_codes = sp.v_cache;
            a.k_scale = reinterpret_cast<float *>(static_cast<uint8_t *>(sp.k_cache) + L->kv8_scale_off);
            a.v_scale = reinterpret_cast<float *>(static_cast<uint8_t *>(sp.v_cache) + L->kv8_scale_off);
            a.scale_cap = L->kv8_scale_cap;
            a.kv_new = L->kv_new;
            a.kv_new_plane = (size_t)c.max_batch * c.n_kv_heads * kHeadDim;
        }
        CK(L, launch_attention(a, s));
    }
    // ---- output projection -> this shard's attention partial sum
    MARK();   // 4
    if (WANT(4)) {
        EpilogueArgs e = {};
        e.kind = EPI_PLAIN;
        e.out = nullptr;
        e.out2 = sp.attn_partial_out;
        e.out_f32 = L->attn_f32;
        if (L->comm) {
            CommView cv;
            if (!comm_fill(L->comm, 1, &cv))
                return PRESERVE_EINVAL;
            e.out = cv.buf[cv.rank];      // this rank's attention partial sums, for every rank's window B
        }
        int rc = launch_gemm(L, 1, L->o, B, e, pdl, s, TRACE(4));
        if (rc)
            return rc;
    }
    // ---- window B  ||  prefetch {Wgate|up, Wdown}
    if (pf_b) {
        CK(L, cudaEventRecord(L->ev_b, s));
        CK(L, cudaStreamWaitEvent(L->side, L->ev_b, 0));
        PrefetchArgs pa = prefetch_base(1);
        pa.n_nodes = 2;
        for (int i = 0; i < 2; ++i) {
            pa.node[i].base = L->arena + L->off[2 + i];
            pa.node[i].bytes = L->wbytes[2 + i];
        }
        const int nb_attr = persist_window(L->off[2], L->wbytes[2] + L->wbytes[3]);
        CK(L, launch_prefetch(pa, L->prefetch_ctas, L->side, nb_attr ? pf_attr : nullptr, nb_attr));
    }
    MARK();   // 5: window B starts
    if (WANT(5)) {
        WindowArgs w = {};
        w.parts[0] = L->attn_f32;
        w.part0_is_f32 = 1;
        for (int i = 0; i + 1 < c.tp_degree; ++i)
            w.parts[i + 1] = sp.peers[i];
        w.n_parts = c.tp_degree;
        w.resid = L->h_f32;
        w.resid_is_f32 = 1;
        w.gain = L->g_mlp;
        w.eps = c.rms_eps;
        w.h_f32 = L->h2_f32;
        w.h_bf16 = sp.residual_out;
        w.x_bf16 = L->x2;
        w.x_fp16 = L->tensor_path ? 1 : 0;
        w.x_plane_elems = (size_t)L->rows * H;
        w.B = B; w.H = H;
        w.trace = TRACE(5);
        w.delay_ns = L->window_delay_ns;
        w.status = L->status;
        w.pdl = pdl;
        w.inputs_after_wait = sp.late_b;
        w.comm_rank = -1;
        if (L->ext_attn_sum) {
            w.parts[0] = L->ext_attn_sum;     // reduced by the caller (e.g. a library all-reduce) beforehand
            w.part0_is_f32 = 0;
        }
        if (L->comm) {
            CommView cv;
            if (!comm_fill(L->comm, 1, &cv))
                return PRESERVE_EINVAL;
            for (int i = 0; i < cv.n_ranks; ++i) {
                w.parts[i] = cv.buf[i];
                w.comm_flags_peer[i] = cv.flags[i];
            }
            w.part0_is_f32 = 0;
            w.comm_rank = cv.rank;
            w.comm_window = 1;
            w.comm_flags_local = cv.flags[cv.rank];
            w.comm_epoch = cv.epoch;
            w.comm_done = cv.done;
        }
        CK(L, launch_window(w, s));
    }
    // ---- gate/up projection + SwiGLU, down projection
    MARK();   // 6
    if (WANT(6)) {
        EpilogueArgs e = {};
        e.kind = EPI_SWIGLU;
        e.out = L->a;
        e.out_plane = (size_t)L->rows * c.ffn;
        e.out_fp16 = L->tensor_path ? 1 : 0;
        int rc = launch_gemm(L, 2, L->x2, B, e, pdl, s, TRACE(6));
        if (rc)
            return rc;
    }
    MARK();   // 7
    if (WANT(7)) {
        EpilogueArgs e = {};
        e.kind = EPI_PLAIN;
        e.out = sp.mlp_partial_out;
        e.out_f32 = L->mlp_f32;
        if (L->comm) {
            CommView cv;
            if (!comm_fill(L->comm, 0, &cv))
                return PRESERVE_EINVAL;
            e.out2 = cv.buf[cv.rank];     // this rank's MLP partial sums, for every rank's next window A
        }
        int rc = launch_gemm(L, 3, L->a, B, e, pdl, s, TRACE(7));
        if (rc)
            return rc;
    }
    MARK();   // 8: end of the last kernel
#undef MARK
#undef WANT
#undef TRACE
    // ---- the side stream is joined once, after the last layer of the call (the prefetch kernels only
    // read, so nothing on the main stream has to wait for them earlier)
    if (pf_a || pf_b)
        L->side_pending = true;       // joined by run_steps after the last layer
    return PRESERVE_OK;
}

int join_side_streams(preserve_layer *const *layers, int n, cudaStream_t s)
{
    for (int i = 0; i < n; ++i) {
        preserve_layer *L = layers[i];
        if (!L->side_pending)
            continue;
        CK(L, cudaEventRecord(L->ev_join, L->side));
        CK(L, cudaStreamWaitEvent(s, L->ev_join, 0));
        L->side_pending = false;
    }
    return PRESERVE_OK;
}

// Everything the captured kernel nodes of one step depend on: the handle, every pointer, the
// settings, and the few numbers the host derives from the sequence lengths (whether each window
// prefetches at all, the attention grid, tiles per work item, merge warps).  The lengths themselves
// are read by the kernels from device memory and are not part of it.
void step_signature(const preserve_layer *L, const StepPtrs &sp, const StepPlan &pl, std::vector<uint64_t> &sig)
{
    auto put = [&](uint64_t v) { sig.push_back(v); };
    auto putp = [&](const void *p) { sig.push_back((uint64_t)reinterpret_cast<uintptr_t>(p)); };
    putp(L);
    put((uint64_t)sp.batch);
    putp(sp.ctx_len);
    for (int i = 0; i < L->cfg.tp_degree; ++i)
        putp(sp.parts[i]);
    for (int i = 0; i + 1 < L->cfg.tp_degree; ++i)
        putp(sp.peers[i]);
    putp(sp.residual_in); putp(sp.k_cache); putp(sp.v_cache);
    putp(sp.residual_out); putp(sp.mlp_partial_out); putp(sp.attn_partial_out);
    put((uint64_t)sp.resid_f32 | (uint64_t)sp.part0_f32 << 1 | (uint64_t)sp.late_a << 2 | (uint64_t)sp.late_b << 3 |
        (uint64_t)(L->tracing ? 1 : 0) << 4 | (uint64_t)pl.pdl << 5 | (uint64_t)(pl.pf_a ? 1 : 0) << 6 |
        (uint64_t)(pl.pf_b ? 1 : 0) << 7 | (uint64_t)L->inject << 8 | (uint64_t)L->pf_mechanism << 16 |
        (uint64_t)L->plan_mode << 24);
    put((uint64_t)L->budget);
    put((uint64_t)L->window_delay_ns | (uint64_t)L->pf_chunk << 32);
    put((uint64_t)L->prefetch_ctas);
    put((uint64_t)pl.attn_grid | (uint64_t)pl.attn_tpi << 32);
    put((uint64_t)pl.attn_items_per_stream);
    putp(L->comm);
    putp(L->ext_attn_sum);
}

// Run `n` steps (already validated) as one replayed graph, or directly.
int run_steps(preserve_layer *const *layers, StepPtrs *sps, int n, cudaStream_t s)
{
    preserve_layer *L0 = layers[0];
    bool direct = (L0->cfg.flags & PRESERVE_FLAG_NO_GRAPH) || s == nullptr || s == cudaStreamLegacy;
    std::vector<StepPlan> plans((size_t)n);
    for (int i = 0; i < n; ++i) {
        sps[i].first_of_call = i == 0;
        plan_step(layers[i], sps[i], &plans[i]);
    }
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (!direct) {
        CK(L0, cudaStreamIsCapturing(s, &cs));
        // the caller is capturing already: just add our nodes to their graph (the capture orders them
        // after the caller's earlier nodes, as a graph launch of our own would)
    }
    if (direct || cs != cudaStreamCaptureStatusNone) {
        for (int i = 0; i < n; ++i) {
            // (first kernel without the early-launch attribute in both cases: nothing orders it
            // after the earlier work on the stream, or the caller's earlier nodes, otherwise)
            int rc = enqueue_step(layers[i], sps[i], plans[i], true, s);
            if (rc)
                return rc;
        }
        return join_side_streams(layers, n, s);
    }
    std::vector<uint64_t> sig;
    sig.reserve((size_t)n * 40 + 2);
    sig.push_back((uint64_t)reinterpret_cast<uintptr_t>(s));
    sig.push_back((uint64_t)n);
    for (int i = 0; i < n; ++i)
        step_signature(layers[i], sps[i], plans[i], sig);
    for (auto &g : L0->graphs)
        if (g.sig == sig) {
            g.stamp = ++L0->stamp;
            for (int i = 0; i < n; ++i) {      // what get_info reports follows the step, replayed or not
                preserve_layer *L = layers[i];
                L->kv_bytes = plans[i].kv_bytes;
                L->alg_bytes = plans[i].alg_bytes;
                memcpy(L->planned, plans[i].planned, sizeof(L->planned));
            }
            CK(L0, cudaGraphLaunch(g.exec, s));
            return PRESERVE_OK;
        }
    // capture
    CK(L0, cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal));
    int rc = PRESERVE_OK;
    for (int i = 0; i < n && rc == PRESERVE_OK; ++i)
        rc = enqueue_step(layers[i], sps[i], plans[i], false, s);
    if (rc == PRESERVE_OK)
        rc = join_side_streams(layers, n, s);
    cudaGraph_t graph = nullptr;
    cudaError_t e = cudaStreamEndCapture(s, &graph);
    if (rc != PRESERVE_OK) {
        if (graph)
            cudaGraphDestroy(graph);
        return rc;
    }
    if (e != cudaSuccess)
        return cuda_fail(L0, e);
    cudaGraphExec_t exec = nullptr;
    e = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess)
        return cuda_fail(L0, e);
    ++L0->n_captures;
    if (L0->graphs.size() >= kMaxCachedGraphs) {
        size_t victim = 0;
        for (size_t i = 1; i < L0->graphs.size(); ++i)
            if (L0->graphs[i].stamp < L0->graphs[victim].stamp)
                victim = i;
        cudaGraphExecDestroy(L0->graphs[victim].exec);
        L0->graphs.erase(L0->graphs.begin() + victim);
    }
    L0->graphs.push_back({std::move(sig), exec, ++L0->stamp});
    CK(L0, cudaGraphLaunch(exec, s));
    return PRESERVE_OK;
}

void drop_graphs(preserve_layer *L)
{
    for (auto &g : L->graphs)
        cudaGraphExecDestroy(g.exec);
    L->graphs.clear();
}

}  // namespace

// ============================================================== C ABI
extern "C" {

const char *preserve_strerror(int code)
{
    switch (code) {
    case PRESERVE_OK: return "ok";
    case PRESERVE_EINVAL: return "invalid argument";
    case PRESERVE_EALIGN: return "device pointer not 16-byte aligned";
    case PRESERVE_ESHAPE: return "unsupported shape";
    case PRESERVE_ENOMEM: return "out of memory";
    case PRESERVE_ECUDA: return "CUDA call failed";
    case PRESERVE_EARCH: return "needs an sm_100 device";
    case PRESERVE_ETIMEOUT: return "a bounded device-side wait gave up";
    case PRESERVE_ETOOBIG: return "problem exceeds the fixed scratch capacity of the allocation-free entry point";
    default: return "unknown error";
    }
}

int preserve_plan_window(const uint64_t *node_bytes, int32_t n_nodes, uint64_t budget, int32_t mode,
                         uint64_t *out_bytes)
{
    if (!node_bytes || !out_bytes || n_nodes < 0)
        return PRESERVE_EINVAL;
    if (mode != PRESERVE_PLAN_WHOLE_NODE && mode != PRESERVE_PLAN_TRUNCATE)
        return PRESERVE_EINVAL;
    plan_window(node_bytes, n_nodes, budget, mode, out_bytes);
    return PRESERVE_OK;
}

uint64_t preserve_algorithmic_bytes(const preserve_layer_config_t *cfg, int32_t batch, uint64_t sum_ctx)
{
    if (!cfg || validate_config(cfg) != PRESERVE_OK || batch < 1)
        return 0;
    const Dims d = layer_dims(*cfg);
    uint64_t w = 0;
    for (int i = 0; i < 4; ++i)
        w += weight_bytes(*cfg, d, i);
    const bool kv8 = (cfg->flags & PRESERVE_FLAG_INT8_KV) != 0;
    const uint64_t kv = kv8 ? 2 * sum_ctx * cfg->n_kv_heads * ((uint64_t)cfg->head_dim + 4)
                            : 2 * sum_ctx * cfg->n_kv_heads * cfg->head_dim * 2;
    return w + kv + activation_bytes(*cfg, batch);
}

int preserve_kv8_layout(const preserve_layer_config_t *cfg, uint64_t *scale_offset_bytes, int32_t *scale_capacity,
                        uint64_t *buffer_bytes)
{
    if (!cfg || !scale_offset_bytes || !scale_capacity || !buffer_bytes)
        return PRESERVE_EINVAL;
    int rc = validate_config(cfg);
    if (rc != PRESERVE_OK)
        return rc;
    int scap = 0;
    kv8_layout(*cfg, scale_offset_bytes, &scap, buffer_bytes);
    *scale_capacity = scap;
    return PRESERVE_OK;
}

void preserve_layer_destroy(preserve_layer_t *L)
{
    if (!L)
        return;
    cudaSetDevice(L->dev);
    if (L->side)
        cudaStreamSynchronize(L->side);
    drop_graphs(L);
    void *ptrs[] = {L->kv_new, L->scales, L->trace_buf, L->attn_f32, L->h2_f32, L->mlp_f32, L->arena, L->inv_freq, L->h_f32, L->x, L->q, L->o, L->x2, L->a,
                    L->part_o, L->part_ml, L->status, L->stage_in, L->stage_out, L->ctx_dev};
    for (void *p : ptrs)
        if (p)
            cudaFree(p);
    for (cudaEvent_t e : L->prof)
        if (e)
            cudaEventDestroy(e);
    if (L->ev_a) cudaEventDestroy(L->ev_a);
    if (L->ev_b) cudaEventDestroy(L->ev_b);
    if (L->ev_join) cudaEventDestroy(L->ev_join);
    if (L->side) cudaStreamDestroy(L->side);
    if (L->xfer) { cudaStreamSynchronize(L->xfer); cudaStreamDestroy(L->xfer); }
    if (L->ev_in_ready) cudaEventDestroy(L->ev_in_ready);
    if (L->ev_in_free) cudaEventDestroy(L->ev_in_free);
    delete L;
}

int preserve_layer_init(const preserve_layer_config_t *cfg, const preserve_layer_weights_t *w,
                        preserve_layer_t **out)
{
    if (out)
        *out = nullptr;
    if (!cfg || !w || !out)
        return PRESERVE_EINVAL;
    int rc = validate_config(cfg);
    if (rc)
        return rc;
    const void *wp[] = {w->w_q, w->w_k, w->w_v, w->w_o, w->w_gate, w->w_up, w->w_down, w->g_attn, w->g_mlp};
    for (const void *p : wp) {
        if (!p)
            return PRESERVE_EINVAL;
        if (!aligned16(p))
            return PRESERVE_EALIGN;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return PRESERVE_EARCH;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess || prop.major != 10) {
        (void)cudaGetLastError();
        return PRESERVE_EARCH;
    }
    if (!get_encode_fn())
        return PRESERVE_EARCH;

    preserve_layer *L = new (std::nothrow) preserve_layer();
    if (!L)
        return PRESERVE_ENOMEM;
    L->cfg = *cfg;
    L->only = -1;
    L->dev = dev;
    L->sm_count = prop.multiProcessorCount;
    L->l2_bytes = prop.l2CacheSize;
    L->max_persist = prop.persistingL2CacheMaxSize;
    L->max_window = prop.accessPolicyMaxWindowSize;
    L->group = cfg->n_q_heads / cfg->n_kv_heads;
    const bool force_gemv = (cfg->flags & PRESERVE_FLAG_FORCE_GEMV) != 0;
    const bool force_tc = (cfg->flags & PRESERVE_FLAG_FORCE_TENSOR) != 0 && cfg->ffn % 128 == 0;
    L->tensor_path = (cfg->max_batch >= 16 && !force_gemv) || force_tc;
    L->no_early = (cfg->flags & PRESERVE_FLAG_NO_EARLY_LAUNCH) != 0;
    L->pf_mechanism = 0;      // measured: bulk L2 prefetch from 128 CTAs disturbs the main stream least
    L->pf_chunk = 4096;
    L->prefetch_ctas = 128;
    L->budget_is_default = true;
    // Measured on all five benchmark configurations with the bare stand-in windows (a few
    // microseconds): early launch alone is the fastest setting; the side-stream L2 kernel costs
    // 1-9 % there and only pays once a window lasts >= ~10 us.  So the default plans nothing for L2.
    L->budget = PRESERVE_BUDGET_EARLY_LAUNCH_ONLY;
    L->plan_mode = PRESERVE_PLAN_TRUNCATE;

#define CKI(expr)                                   \
    do {                                            \
        cudaError_t e__ = (expr);                   \
        if (e__ != cudaSuccess) {                   \
            int r__ = cuda_fail(L, e__);            \
            preserve_layer_destroy(L);              \
            return r__;                             \
        }                                           \
    } while (0)

    const auto &c = L->cfg;
    const Dims d = layer_dims(c);
    const int H = c.hidden, B = c.max_batch;
    size_t off = 0;
    for (int i = 0; i < 4; ++i) {
        L->off[i] = off;
        L->wbytes[i] = weight_bytes(c, d, i);
        off += (size_t)L->wbytes[i];
    }
    const size_t gains_off = off;
    off += (size_t)2 * H * 2;
    L->arena_bytes = off;
    CKI(cudaMalloc(&L->arena, L->arena_bytes));
    L->g_attn = L->arena + gains_off;
    L->g_mlp = L->arena + gains_off + (size_t)H * 2;
    CKI(cudaMemcpy(L->g_attn, w->g_attn, (size_t)H * 2, cudaMemcpyDeviceToDevice));
    CKI(cudaMemcpy(L->g_mlp, w->g_mlp, (size_t)H * 2, cudaMemcpyDeviceToDevice));

    // pack the four weight blocks in consumption order
    {
        const void *s_qkv[3] = {w->w_q, w->w_k, w->w_v};
        const int c_qkv[3] = {c.n_q_heads * c.head_dim, c.n_kv_heads * c.head_dim, c.n_kv_heads * c.head_dim};
        const void *s_o[1] = {w->w_o};
        const int c_o[1] = {H};
        const void *s_gu[2] = {w->w_gate, w->w_up};
        const int c_gu[2] = {c.ffn, c.ffn};
        const void *s_dn[1] = {w->w_down};
        const int c_dn[1] = {H};
        L->w8 = (c.flags & PRESERVE_FLAG_INT8_WEIGHTS) != 0;
        if (L->w8) {
            size_t so = 0;
            for (int i = 0; i < 4; ++i) {
                L->soff[i] = so;
                so += (size_t)d.n[i];
            }
            CKI(cudaMalloc(&L->scales, so * sizeof(float)));
            // (tensor path: blocks of one or two 128-row tiles, as the GEMM will take them per CTA)
            const int nbp = ((c.max_batch + 15) / 16) * 16;
            auto pack8 = [&](const void *const *srcs, const int *cols, int n, int i, int kind) -> cudaError_t {
                return L->tensor_path ? launch_pack_rows_w8(srcs, cols, n, d.k[i], kind, L->arena + L->off[i],
                                                            L->scales + L->soff[i], gemm_tc_w8_tiles(nbp, d.n[i], i >= 1),
                                                            nullptr)
                                      : launch_pack_gemv_w8(srcs, cols, n, d.k[i], kind, L->arena + L->off[i],
                                                            L->scales + L->soff[i], nullptr);
            };
            CKI(pack8(s_qkv, c_qkv, 3, 0, EPI_QKV));
            CKI(pack8(s_o, c_o, 1, 1, EPI_PLAIN));
            CKI(pack8(s_gu, c_gu, 2, 2, EPI_SWIGLU));
            CKI(pack8(s_dn, c_dn, 1, 3, EPI_PLAIN));
        } else {
            auto pack = L->tensor_path ? launch_pack_rows : launch_pack_gemv;
            // (tensor path: Wgate|up meets the fp16 RMSNorm output x2 and is stored as fp16)
            CKI(pack(s_qkv, c_qkv, 3, d.k[0], EPI_QKV, L->arena + L->off[0], L->tensor_path ? 1 : 0, nullptr));
            CKI(pack(s_o, c_o, 1, d.k[1], EPI_PLAIN, L->arena + L->off[1], 1, nullptr));
            CKI(pack(s_gu, c_gu, 2, d.k[2], EPI_SWIGLU, L->arena + L->off[2], 1, nullptr));
            CKI(pack(s_dn, c_dn, 1, d.k[3], EPI_PLAIN, L->arena + L->off[3], 1, nullptr));
        }
    }
    // rotary frequencies theta^(-2i/d)
    {
        double f[kHeadDim / 2];
        for (int i = 0; i < kHeadDim / 2; ++i)
            f[i] = c.rope_theta > 0.f ? std::pow((double)c.rope_theta, -2.0 * i / (double)kHeadDim) : 0.0;
        CKI(cudaMalloc(&L->inv_freq, sizeof(f)));
        CKI(cudaMemcpy(L->inv_freq, f, sizeof(f), cudaMemcpyHostToDevice));
    }
    // workspaces
    L->nb_pad = ((B + 15) / 16) * 16;
    L->rows = L->tensor_path ? L->nb_pad : B;
    const size_t BH = (size_t)B * H;
    const size_t RH = (size_t)L->rows * H, Rq = (size_t)L->rows * c.n_q_heads * c.head_dim;
    const size_t RF = (size_t)L->rows * c.ffn;
    CKI(cudaMalloc(&L->h_f32, BH * 4));
    CKI(cudaMalloc(&L->attn_f32, BH * 4));
    CKI(cudaMalloc(&L->h2_f32, BH * 4));
    CKI(cudaMalloc(&L->mlp_f32, BH * 4));
    CKI(cudaMalloc(&L->x, 2 * RH * 2));
    CKI(cudaMalloc(&L->q, 2 * Rq * 2));
    CKI(cudaMalloc(&L->o, 2 * Rq * 2));
    CKI(cudaMalloc(&L->x2, 2 * RH * 2));
    CKI(cudaMalloc(&L->a, 2 * RF * 2));
    CKI(cudaMemset(L->x, 0, 2 * RH * 2));
    CKI(cudaMemset(L->q, 0, 2 * Rq * 2));
    CKI(cudaMemset(L->o, 0, 2 * Rq * 2));
    CKI(cudaMemset(L->x2, 0, 2 * RH * 2));
    CKI(cudaMemset(L->a, 0, 2 * RF * 2));
    // work items of the attention kernel: at most 2 CTAs per SM x 4 items each, plus one short
    // item per (sequence, kv head) from rounding up
    L->max_items = L->sm_count * 8 + B * c.n_kv_heads + 8;
    CKI(cudaMalloc(&L->part_o, (size_t)L->max_items * L->group * kHeadDim * 4));
    CKI(cudaMalloc(&L->part_ml, (size_t)L->max_items * L->group * 2 * 4));
    L->kv8 = (c.flags & PRESERVE_FLAG_INT8_KV) != 0;
    if (L->kv8) {
        uint64_t total = 0;
        kv8_layout(c, &L->kv8_scale_off, &L->kv8_scale_cap, &total);
        CKI(cudaMalloc(&L->kv_new, (size_t)2 * B * c.n_kv_heads * kHeadDim * sizeof(float)));
        CKI(cudaMemset(L->kv_new, 0, (size_t)2 * B * c.n_kv_heads * kHeadDim * sizeof(float)));
    }
    CKI(cudaMalloc(&L->status, 256));
    CKI(cudaMemset(L->status, 0, 256));
    const size_t n_in = (size_t)(2 * c.tp_degree) * BH * 2;
    CKI(cudaMalloc(&L->stage_in, n_in));
    CKI(cudaMalloc(&L->stage_out, 2 * BH * 2));
    CKI(cudaMalloc(&L->ctx_dev, (size_t)B * 4));
    CKI(cudaMalloc(&L->trace_buf, sizeof(long long) * PRESERVE_TRACE_SLOTS * PRESERVE_N_KERNELS));

    if (L->tensor_path) {
        // activations as the B operand: [2 * nb_pad, K] = hi rows then lo rows, one box covers both
        const void *xb[4] = {L->x, L->o, L->x2, L->a};
        for (int i = 0; i < 4; ++i) {
            // x (two fp16 planes: hi rows, lo rows) feeds the QKV projection; o, x2 and a are one fp16 plane each
            const uint32_t brows = (uint32_t)(i >= 1 ? L->nb_pad : 2 * L->nb_pad);
            // (int8 weights are fetched by plain bulk copies: no map over them)
            const bool wok = L->w8 || make_map_2d(&L->wmap[i], L->arena + L->off[i], d.k[i], d.n[i], 64, 128);
            if (!wok || !make_map_2d(&L->xmap[i], xb[i], d.k[i], brows, 64, brows)) {
                preserve_layer_destroy(L);
                return PRESERVE_EARCH;
            }
            L->has256[i] = !L->w8 && d.n[i] % 256 == 0 &&
                           make_map_2d(&L->wmap256[i], L->arena + L->off[i], d.k[i], d.n[i], 64, 256);
        }
    }
    if ((c.flags & PRESERVE_FLAG_PERSIST_L2) && L->max_persist > 0) {
        // a context-wide limit of this process: reserve up to 3/4 of what the device allows
        CKI(cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, (size_t)L->max_persist / 4 * 3));
    }
    CKI(cudaStreamCreateWithFlags(&L->side, cudaStreamNonBlocking));
    CKI(cudaEventCreateWithFlags(&L->ev_a, cudaEventDisableTiming));
    CKI(cudaEventCreateWithFlags(&L->ev_b, cudaEventDisableTiming));
    CKI(cudaEventCreateWithFlags(&L->ev_join, cudaEventDisableTiming));
    {
        // highest priority: its few CTAs take the first slots that free up beside the main stream's kernels
        int prio_lo = 0, prio_hi = 0;
        CKI(cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi));
        CKI(cudaStreamCreateWithPriority(&L->xfer, cudaStreamNonBlocking, prio_hi));
    }
    CKI(cudaEventCreateWithFlags(&L->ev_in_ready, cudaEventDisableTiming));
    CKI(cudaEventCreateWithFlags(&L->ev_in_free, cudaEventDisableTiming));
    L->in_free_valid = false;
    for (int i = 0; i <= PRESERVE_N_KERNELS; ++i)
        CKI(cudaEventCreate(&L->prof[i]));
    CKI(cudaDeviceSynchronize());
#undef CKI
    *out = L;
    return PRESERVE_OK;
}

int preserve_set_prefetch_bytes(preserve_layer_t *L, size_t bytes_per_window)
{
    if (!L)
        return PRESERVE_EINVAL;
    L->budget = bytes_per_window;
    L->budget_is_default = false;
    return PRESERVE_OK;
}

int preserve_set_prefetch_mechanism(preserve_layer_t *L, int32_t mechanism, uint32_t chunk_bytes, int32_t ctas)
{
    if (!L || mechanism < 0 || mechanism > 2 || chunk_bytes < 128 || chunk_bytes % 128 || chunk_bytes > (1u << 20) ||
        ctas < 1 || ctas > 1024)
        return PRESERVE_EINVAL;
    L->pf_mechanism = mechanism;
    L->pf_chunk = chunk_bytes;
    L->prefetch_ctas = ctas;
    return PRESERVE_OK;
}

int preserve_debug_set(preserve_layer_t *L, int32_t what, int64_t value)
{
    if (!L)
        return PRESERVE_EINVAL;
    if (what == PRESERVE_DEBUG_WITHHOLD) {
        if (value < 0 || value > INJECT_ATTN_RING)
            return PRESERVE_EINVAL;
        L->inject = (int)value;
        return PRESERVE_OK;
    }
    if (what == PRESERVE_DEBUG_WAIT_LIMIT_CYCLES) {
        if (value < 0)
            return PRESERVE_EINVAL;
        CK(L, cudaSetDevice(L->dev));
        CK(L, cudaDeviceSynchronize());
        long long lim = value;
        CK(L, cudaMemcpy(L->status + kStatusLimitWord, &lim, sizeof(lim), cudaMemcpyHostToDevice));
        return PRESERVE_OK;
    }
    return PRESERVE_EINVAL;
}

int preserve_clear_status(preserve_layer_t *L)
{
    if (!L)
        return PRESERVE_EINVAL;
    CK(L, cudaSetDevice(L->dev));
    CK(L, cudaDeviceSynchronize());
    CK(L, cudaMemset(L->status, 0, sizeof(int)));
    return PRESERVE_OK;
}

int preserve_layer_set_comm(preserve_layer_t *L, preserve_comm_t *comm)
{
    if (!L)
        return PRESERVE_EINVAL;
    if (comm) {
        CommView cv;
        if (!comm_fill(comm, 0, &cv))
            return PRESERVE_EINVAL;                 // not every peer connected
        if (cv.n_ranks != L->cfg.tp_degree || comm_hidden(comm) != L->cfg.hidden ||
            comm_max_batch(comm) < L->cfg.max_batch)
            return PRESERVE_ESHAPE;
        if (L->ext_attn_sum)
            return PRESERVE_EINVAL;
    }
    L->comm = comm;
    return PRESERVE_OK;
}

int preserve_layer_set_external_attention_sum(preserve_layer_t *L, const void *reduced_attn_partial)
{
    if (!L || (reduced_attn_partial && L->comm))
        return PRESERVE_EINVAL;
    if (reduced_attn_partial && !aligned16(reduced_attn_partial))
        return PRESERVE_EALIGN;
    L->ext_attn_sum = reduced_attn_partial;
    return PRESERVE_OK;
}

int64_t preserve_graph_captures(const preserve_layer_t *L) { return L ? (int64_t)L->n_captures : -1; }

int preserve_set_window_delay_ns(preserve_layer_t *L, int32_t ns)
{
    if (!L || ns < 0 || ns > 1000000)
        return PRESERVE_EINVAL;
    L->window_delay_ns = ns;
    return PRESERVE_OK;
}

int preserve_set_plan_mode(preserve_layer_t *L, int mode)
{
    if (!L || (mode != PRESERVE_PLAN_WHOLE_NODE && mode != PRESERVE_PLAN_TRUNCATE))
        return PRESERVE_EINVAL;
    L->plan_mode = mode;
    return PRESERVE_OK;
}

int preserve_decode_step(preserve_layer_t *L, const preserve_step_io_t *io, void *cuda_stream)
{
    StepPtrs sp = {};
    int rc = check_step(L, io, &sp);
    if (rc)
        return rc;
    preserve_layer *layers[1] = {L};
    return run_steps(layers, &sp, 1, static_cast<cudaStream_t>(cuda_stream));
}

namespace {
bool ranges_overlap(const void *a, size_t na, const void *b, size_t nb)
{
    if (!a || !b)
        return false;
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + nb && y < x + na;
}
}  // namespace

int preserve_decode_chain(preserve_layer_t *const *layers, int32_t n, const preserve_step_io_t *ios, int32_t link,
                          void *cuda_stream)
{
    if (!layers || !ios || n < 1 || n > 256)
        return PRESERVE_EINVAL;
    std::vector<StepPtrs> sps((size_t)n);
    for (int i = 0; i < n; ++i) {
        int rc = check_step(layers[i], &ios[i], &sps[i]);
        if (rc)
            return rc;
        if (sps[i].batch != sps[0].batch)
            return PRESERVE_ESHAPE;
        if (link && i > 0) {
            if (layers[i]->cfg.hidden != layers[0]->cfg.hidden)
                return PRESERVE_ESHAPE;
            // hand the previous layer's results over unrounded (fp32); its bf16 outputs are written too
            sps[i].parts[0] = layers[i - 1]->mlp_f32;
            sps[i].part0_f32 = 1;
            sps[i].residual_in = layers[i - 1]->h2_f32;
            sps[i].resid_f32 = 1;
        }
    }
    // The window kernels request the step's input buffers before they wait for the kernel in front
    // of them.  Inside one call that is only safe for buffers no earlier layer of the call writes:
    // where an input of layer i overlaps an output of a layer before it (layers wired output to
    // input without `link`), that window reads its inputs after the wait instead.
    for (int i = 1; i < n; ++i) {
        const size_t nb = (size_t)sps[i].batch * layers[i]->cfg.hidden * 2;
        const int P = layers[i]->cfg.tp_degree;
        for (int j = 0; j < i; ++j) {
            const size_t mb = (size_t)sps[j].batch * layers[j]->cfg.hidden * 2;
            const void *outs[3] = {sps[j].residual_out, sps[j].mlp_partial_out, sps[j].attn_partial_out};
            for (const void *o : outs) {
                if (!sps[i].resid_f32 && ranges_overlap(sps[i].residual_in, nb, o, mb))
                    sps[i].late_a = 1;
                for (int q = 0; q < P; ++q)
                    if (!(q == 0 && sps[i].part0_f32) && ranges_overlap(sps[i].parts[q], nb, o, mb))
                        sps[i].late_a = 1;
                for (int q = 0; q + 1 < P; ++q)
                    if (ranges_overlap(sps[i].peers[q], nb, o, mb))
                        sps[i].late_b = 1;
            }
        }
    }
    return run_steps(layers, sps.data(), n, static_cast<cudaStream_t>(cuda_stream));
}

int preserve_decode_step_host(preserve_layer_t *L, const preserve_host_io_t *io, void *cuda_stream)
{
    if (!L || !io)
        return PRESERVE_EINVAL;
    const auto &c = L->cfg;
    if (io->batch < 1 || io->batch > c.max_batch)
        return PRESERVE_ESHAPE;
    if (!io->ctx_len_host || !io->partials_in || !io->residual_in || !io->k_cache || !io->v_cache ||
        !io->residual_out || !io->mlp_partial_out || (c.tp_degree > 1 && !io->attn_peer_partials))
        return PRESERVE_EINVAL;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t BH2 = (size_t)io->batch * c.hidden * 2;
    const size_t slot = (size_t)c.max_batch * c.hidden * 2;
    const void *dparts[kMaxParts], *dpeers[kMaxParts];
    for (int i = 0; i < c.tp_degree; ++i)
        if (!io->partials_in[i])
            return PRESERVE_EINVAL;
    for (int i = 0; i + 1 < c.tp_degree; ++i)
        if (!io->attn_peer_partials[i])
            return PRESERVE_EINVAL;

    // Pinned (page-locked) host buffers are visible to the device: one gather kernel on the layer's
    // transfer stream reads them over PCIe into the staging area - that read IS the host-to-device
    // transfer - while the kernels of the call before this one are still running on `s`; the step
    // then reads device memory.  (2P + 1 separate copy calls would cost more host time than a small
    // layer runs, and window kernels reading host memory themselves put the PCIe latency on the
    // critical path.)  Pageable buffers take the copy-call path.
    auto device_view = [](const void *hp) -> const void * {
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, hp) != cudaSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        if (at.type != cudaMemoryTypeHost || !at.devicePointer ||
            (reinterpret_cast<uintptr_t>(at.devicePointer) & 15))
            return nullptr;
        return at.devicePointer;
    };
    const int n_bufs = 2 * c.tp_degree;      // P partials, P - 1 peers, residual
    const void *views[2 * kMaxParts + 1];
    void *slots[2 * kMaxParts + 1];
    bool direct = BH2 % 16 == 0;
    for (int i = 0; i < n_bufs; ++i)
        slots[i] = L->stage_in + (size_t)i * slot;
    for (int i = 0; i < c.tp_degree && direct; ++i)
        direct = (views[i] = device_view(io->partials_in[i])) != nullptr;
    for (int i = 0; i + 1 < c.tp_degree && direct; ++i)
        direct = (views[c.tp_degree + i] = device_view(io->attn_peer_partials[i])) != nullptr;
    if (direct)
        direct = (views[2 * c.tp_degree - 1] = device_view(io->residual_in)) != nullptr;
    const void *dctx_view = direct ? device_view(io->ctx_len_host) : nullptr;
    if (dctx_view && (reinterpret_cast<uintptr_t>(dctx_view) & 3))
        dctx_view = nullptr;
    // the staging area is free again once the previous call's step has read it
    if (L->in_free_valid)
        CK(L, cudaStreamWaitEvent(direct ? L->xfer : s, L->ev_in_free, 0));
    if (direct) {
        CK(L, launch_stage_inputs(views, slots, n_bufs, BH2, static_cast<const int *>(dctx_view), L->ctx_dev,
                                  dctx_view ? io->batch : 0, L->xfer));
        CK(L, cudaEventRecord(L->ev_in_ready, L->xfer));
        CK(L, cudaStreamWaitEvent(s, L->ev_in_ready, 0));
    } else {
        for (int i = 0; i < c.tp_degree; ++i)
            CK(L, cudaMemcpyAsync(slots[i], io->partials_in[i], BH2, cudaMemcpyHostToDevice, s));
        for (int i = 0; i + 1 < c.tp_degree; ++i)
            CK(L, cudaMemcpyAsync(slots[c.tp_degree + i], io->attn_peer_partials[i], BH2, cudaMemcpyHostToDevice, s));
        CK(L, cudaMemcpyAsync(slots[2 * c.tp_degree - 1], io->residual_in, BH2, cudaMemcpyHostToDevice, s));
    }
    if (!direct || !dctx_view)
        CK(L, cudaMemcpyAsync(L->ctx_dev, io->ctx_len_host, (size_t)io->batch * 4, cudaMemcpyHostToDevice, s));
    for (int i = 0; i < c.tp_degree; ++i)
        dparts[i] = slots[i];
    for (int i = 0; i + 1 < c.tp_degree; ++i)
        dpeers[i] = slots[c.tp_degree + i];
    const void *dres = slots[2 * c.tp_degree - 1];
    const void *dctx = L->ctx_dev;

    preserve_step_io_t dio = {};
    dio.batch = io->batch;
    dio.ctx_len = static_cast<const int32_t *>(dctx);
    dio.ctx_len_host = io->ctx_len_host;
    dio.partials_in = dparts;
    dio.attn_peer_partials = dpeers;
    dio.residual_in = dres;
    dio.k_cache = io->k_cache;
    dio.v_cache = io->v_cache;
    // Results go straight into the caller's pinned buffers when the device can address them (posted
    // writes over PCIe from the kernels that produce them); copy calls otherwise.
    void *out_res = direct ? const_cast<void *>(device_view(io->residual_out)) : nullptr;
    void *out_mlp = direct ? const_cast<void *>(device_view(io->mlp_partial_out)) : nullptr;
    const bool direct_out = out_res && out_mlp;
    dio.residual_out = direct_out ? out_res : L->stage_out;
    dio.mlp_partial_out = direct_out ? out_mlp : L->stage_out + slot;
    dio.attn_partial_out = nullptr;
    int rc = preserve_decode_step(L, &dio, cuda_stream);
    if (rc)
        return rc;
    CK(L, cudaEventRecord(L->ev_in_free, s));
    L->in_free_valid = true;
    if (!direct_out) {
        CK(L, cudaMemcpyAsync(io->residual_out, L->stage_out, BH2, cudaMemcpyDeviceToHost, s));
        CK(L, cudaMemcpyAsync(io->mlp_partial_out, L->stage_out + slot, BH2, cudaMemcpyDeviceToHost, s));
    }
    return PRESERVE_OK;
}

int preserve_profile_step(preserve_layer_t *L, const preserve_step_io_t *io, void *cuda_stream, float *kernel_ms)
{
    if (!kernel_ms)
        return PRESERVE_EINVAL;
    StepPtrs sp = {};
    int rc = check_step(L, io, &sp);
    if (rc)
        return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    StepPlan pl;
    sp.first_of_call = 1;
    plan_step(L, sp, &pl);
    L->profiling = true;
    rc = enqueue_step(L, sp, pl, true, s);
    L->profiling = false;
    if (rc)
        return rc;
    {
        preserve_layer *one[1] = {L};
        rc = join_side_streams(one, 1, s);
        if (rc)
            return rc;
    }
    CK(L, cudaStreamSynchronize(s));
    for (int i = 0; i < PRESERVE_N_KERNELS; ++i)
        CK(L, cudaEventElapsedTime(&kernel_ms[i], L->prof[i], L->prof[i + 1]));
    return PRESERVE_OK;
}

int preserve_run_kernel(preserve_layer_t *L, const preserve_step_io_t *io, int32_t which, void *cuda_stream)
{
    if (which < 0 || which >= PRESERVE_N_KERNELS)
        return PRESERVE_EINVAL;
    StepPtrs sp = {};
    int rc = check_step(L, io, &sp);
    if (rc)
        return rc;
    L->only = which;
    StepPlan pl;
    sp.first_of_call = 1;
    plan_step(L, sp, &pl);
    // (early launch allowed: the buffers the kernel reads hold an earlier step's results by contract)
    rc = enqueue_step(L, sp, pl, false, static_cast<cudaStream_t>(cuda_stream));
    L->only = -1;
    if (rc == PRESERVE_OK && (which == 4 || which == 7) && L->side_pending) {
        // a prefetch queued by preserve_prefetch_window for this block: joined where the block ends
        preserve_layer *one[1] = {L};
        rc = join_side_streams(one, 1, static_cast<cudaStream_t>(cuda_stream));
    }
    return rc;
}

int preserve_prefetch_window(preserve_layer_t *L, const preserve_step_io_t *io, int32_t window, void *cuda_stream)
{
    if (window != 0 && window != 1)
        return PRESERVE_EINVAL;
    StepPtrs sp = {};
    int rc = check_step(L, io, &sp);
    if (rc)
        return rc;
    L->only = window == 0 ? -2 : -3;
    StepPlan pl;
    sp.first_of_call = 1;
    plan_step(L, sp, &pl);
    rc = enqueue_step(L, sp, pl, true, static_cast<cudaStream_t>(cuda_stream));
    L->only = -1;
    return rc;
}

static int reset_trace(preserve_layer *L)
{
    long long init[PRESERVE_N_KERNELS][PRESERVE_TRACE_SLOTS];
    for (auto &r : init) {
        for (auto &v : r)
            v = 0;
        r[0] = r[1] = r[6] = 0x7fffffffffffffffll;     // the slots that take a minimum
    }
    CK(L, cudaMemcpy(L->trace_buf, init, sizeof(init), cudaMemcpyHostToDevice));
    return PRESERVE_OK;
}

int preserve_set_trace(preserve_layer_t *L, int32_t on)
{
    if (!L)
        return PRESERVE_EINVAL;
    L->tracing = on != 0;
    return on ? reset_trace(L) : PRESERVE_OK;
}

int preserve_read_trace(preserve_layer_t *L, int64_t *out)
{
    if (!L || !out)
        return PRESERVE_EINVAL;
    CK(L, cudaDeviceSynchronize());
    CK(L, cudaMemcpy(out, L->trace_buf, sizeof(long long) * PRESERVE_TRACE_SLOTS * PRESERVE_N_KERNELS, cudaMemcpyDeviceToHost));
    return reset_trace(L);
}

int preserve_layer_get_info(const preserve_layer_t *L, preserve_info_t *info)
{
    if (!L || !info)
        return PRESERVE_EINVAL;
    memset(info, 0, sizeof(*info));
    info->sm_count = L->sm_count;
    info->l2_bytes = L->l2_bytes;
    info->max_persisting_l2_bytes = L->max_persist;
    info->max_access_window_bytes = L->max_window;
    info->uses_tensor_path = L->tensor_path ? 1 : 0;
    info->activation_rows = L->rows;
    info->plan_mode = L->plan_mode;
    info->normed_activations_fp16 = L->tensor_path ? 1 : 0;
    info->prefetch_budget = L->budget;
    for (int i = 0; i < 4; ++i)
        info->weight_bytes[i] = L->wbytes[i];
    info->kv_bytes = L->kv_bytes;
    for (int i = 0; i < 2; ++i)
        for (int j = 0; j < 3; ++j)
            info->planned_bytes[i][j] = L->planned[i][j];
    info->algorithmic_bytes = L->alg_bytes;
    return PRESERVE_OK;
}

int preserve_last_status(preserve_layer_t *L)
{
    if (!L)
        return PRESERVE_EINVAL;
    CK(L, cudaSetDevice(L->dev));
    CK(L, cudaDeviceSynchronize());
    int st = 0;
    CK(L, cudaMemcpy(&st, L->status, sizeof(int), cudaMemcpyDeviceToHost));
    return st == ST_OK ? PRESERVE_OK : (st == ST_ITEMS_OVERFLOW ? PRESERVE_ESHAPE : PRESERVE_ETIMEOUT);
}

int preserve_last_status_code(preserve_layer_t *L)
{
    if (!L)
        return PRESERVE_EINVAL;
    CK(L, cudaSetDevice(L->dev));
    CK(L, cudaDeviceSynchronize());
    int st = 0;
    CK(L, cudaMemcpy(&st, L->status, sizeof(int), cudaMemcpyDeviceToHost));
    return st;
}

int preserve_last_cuda_error(const preserve_layer_t *L) { return L ? L->last_cuda : 0; }

int preserve_debug_copy(preserve_layer_t *L, int32_t which, void *dst, size_t bytes, void *cuda_stream)
{
    if (!L || !dst)
        return PRESERVE_EINVAL;
    const auto &c = L->cfg;
    const size_t BH = (size_t)c.max_batch * c.hidden;
    const size_t RH = (size_t)L->rows * c.hidden, Rq = (size_t)L->rows * c.n_q_heads * c.head_dim;
    const void *src[7] = {L->h_f32, L->x, L->q, L->o, L->x2, L->a, L->status + kStatusPlanWord};
    const size_t cap[7] = {BH * 4, 2 * RH * 2, 2 * Rq * 2, 2 * Rq * 2, 2 * RH * 2, 2 * (size_t)L->rows * c.ffn * 2,
                           6 * sizeof(uint64_t)};
    if (which < 0 || which > 6 || bytes > cap[which])
        return PRESERVE_EINVAL;
    CK(L, cudaMemcpyAsync(dst, src[which], bytes, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream)));
    return PRESERVE_OK;
}

}  // extern "C"
