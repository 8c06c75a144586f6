/*
 * preserve.h — C ABI of the B200 (sm_100a) decode-step library.
 *
 * One handle = one tensor-parallel shard of one decoder layer.  A decode step
 * consumes the previous block's partial sums, runs the layer's memory-bound
 * kernels (skinny GEMMs over the shard's QKV / O / gate-up / down weights and
 * grouped-query decode attention over the KV-cache) and emits this shard's
 * partial sums.  While each "communication window" runs, a side stream
 * prefetches the weights and KV-cache entries of the following operators into
 * L2, up to a byte budget.
 *
 * Paper passages behind the entry points:
 *   - prefetching read-only weights and KV-cache into L2 in a stream parallel
 *     to the collective: Section 3, "Execution with the proposed method";
 *   - which operators get a prefetch and the running budget: Algorithm 1
 *     ("Prefetch Operator Insertion") and Section 3, "L2 capacity requirements";
 *   - prefetch stream parallel to the main stream, ordered by events:
 *     Section 3, "PRESERVE" (runtime paragraph);
 *   - the layer's blocks and the tensor-parallel split (heads; MLP
 *     intermediate dimension; one allreduce per block): Section 2.
 * On one GPU the communication window is a local stand-in that computes what
 * the allreduce plus its epilogue would deliver: the sum of P partial-sum
 * buffers already in device memory, the residual add and RMSNorm.
 *
 * General rules
 *   - All tensors are bf16 unless stated; "device" / "host" says where a
 *     pointer must live.  Device pointers must be 16-byte aligned.
 *   - The caller owns every pointer it passes.  Weights are borrowed only for
 *     the duration of preserve_layer_init (the library keeps its own packed
 *     copy).  Buffers named in a step must stay valid until the work queued on
 *     the stream has finished.
 *   - Every call returns PRESERVE_OK (0) or a negative PRESERVE_E* code; no
 *     exception, abort or print crosses the boundary.  preserve_decode_* are
 *     asynchronous on the given stream; a device-side failure (a bounded wait
 *     that gave up) is reported by preserve_last_status.
 *   - Results are a pure function of the inputs: they do not depend, bit for
 *     bit, on the prefetch budget or mode.
 *   - A handle is not thread-safe; distinct handles are independent (the library keeps
 *     no mutable process-wide state besides per-device "attribute already set" marks).
 *   - Buffers of one call: outputs must not overlap each other or the inputs of the same
 *     layer; the KV-caches of different layers of a call must not overlap.  An input of a
 *     layer MAY be an output of an earlier layer of the same preserve_decode_chain call
 *     (layers wired output to input): the library then reads it only after the producer
 *     has finished.  Inputs written by work queued on the stream BEFORE the call are
 *     always read after that work.
 *   - The library needs a device of compute capability 10.x and fails with
 *     PRESERVE_EARCH elsewhere; it has no CPU fallback.
 */
#ifndef PRESERVE_H
#define PRESERVE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* The library is built with hidden visibility; only these entry points are exported. */
#if defined(__GNUC__)
#define PRESERVE_API __attribute__((visibility("default")))
#else
#define PRESERVE_API
#endif

#define PRESERVE_OK        0
#define PRESERVE_EINVAL   (-1)  /* null pointer, bad enum, bad count                */
#define PRESERVE_EALIGN   (-2)  /* a device pointer is not 16-byte aligned          */
#define PRESERVE_ESHAPE   (-3)  /* unsupported sizes (see preserve_layer_config_t)  */
#define PRESERVE_ENOMEM   (-4)  /* device or host allocation failed                 */
#define PRESERVE_ECUDA    (-5)  /* a CUDA call failed; see preserve_last_cuda_error */
#define PRESERVE_EARCH    (-6)  /* no sm_100 device / driver entry point missing    */
#define PRESERVE_ETIMEOUT (-7)  /* a bounded device-side wait gave up               */
#define PRESERVE_ETOOBIG  (-8)  /* problem larger than a fixed-capacity entry point  */

/* Prefetch planning modes. */
#define PRESERVE_PLAN_WHOLE_NODE 0  /* Algorithm 1: a tensor is prefetched whole or not at all      */
#define PRESERVE_PLAN_TRUNCATE   1  /* the first tensor that does not fit is prefetched for its
                                       leading bytes (in the order its consumer reads them)          */

/* flags for preserve_layer_config_t.flags */
#define PRESERVE_FLAG_NO_GRAPH   1u /* launch kernels directly instead of replaying a CUDA graph     */
#define PRESERVE_FLAG_PERSIST_L2 2u /* prefetch kernels run with a persisting access-policy window over the
                                       planned weight range; sets this process's persisting-L2 limit to
                                       3/4 of cudaDevAttrMaxPersistingL2CacheSize at init (off by default) */
#define PRESERVE_FLAG_NO_EARLY_LAUNCH 4u /* ablation: prefetch into L2 only; consumer kernels are not
                                       launched early to stage operands in shared memory              */
#define PRESERVE_FLAG_FORCE_GEMV   8u  /* use the split-K GEMV kernels whatever max_batch is (each launch
                                       covers 16 batch rows)                                          */
#define PRESERVE_FLAG_INT8_WEIGHTS 32u  /* keep the four weight matrices as int8 codes with one fp32 scale per output
                                       feature (symmetric: scale = max |w| / 127 over the feature's inputs, code =
                                       round-to-nearest-even(w / scale), decided in fp32) - the weight precision
                                       of the paper's measurements (Section 4, "Experimental setup"); activations
                                       stay 16-bit (the KV-cache too unless PRESERVE_FLAG_INT8_KV is given).  Both
                                       GEMM paths: the split-K GEMV kernels widen the codes in registers, the
                                       tcgen05 kernels into tensor memory (the MMA's A operand).  ffn a
                                       multiple of 64; PRESERVE_ESHAPE otherwise */
#define PRESERVE_FLAG_INT8_KV 64u      /* the KV-cache is int8 with one fp32 scale per cached vector, i.e. per
                                       (sequence, kv head, slot): scale = max |u| / 127 over the vector's head_dim
                                       values, code = round-to-nearest-even(u / scale), decided in fp32; a cached
                                       value is code * scale (the cache precision of the paper's measurements,
                                       Section 4 "Experimental setup"; the scaling is this library's reading).
                                       k_cache and v_cache then each point to ONE buffer laid out as
                                       preserve_kv8_layout says: the codes, then the scales.  The step quantises its
                                       new key and value, stores them at slot ctx_len[b] and attends over the
                                       cache as stored.  At most 8 query heads per KV head; PRESERVE_ESHAPE
                                       otherwise.  preserve_attention_static does not take this layout.      */
#define PRESERVE_FLAG_FORCE_TENSOR 16u /* use the tcgen05 GEMM kernels although max_batch < 16 (needs ffn
                                       to be a multiple of 128)                                       */

typedef struct preserve_layer preserve_layer_t;   /* opaque, owned by the library */

/* Per-shard sizes.  Supported: head_dim == 128; n_q_heads a multiple of
 * n_kv_heads with at most 16 query heads per KV head; hidden a multiple of 128
 * and at most 16384; ffn a multiple of 32 (128 when max_batch >= 16);
 * 1 <= tp_degree <= 16; 1 <= max_batch <= 128. */
typedef struct {
    int32_t hidden;       /* H                                                       */
    int32_t n_q_heads;    /* query heads held by this shard                          */
    int32_t n_kv_heads;   /* KV heads held by this shard                             */
    int32_t head_dim;     /* d                                                       */
    int32_t ffn;          /* F: this shard's slice of the MLP intermediate dimension */
    int32_t tp_degree;    /* P: partial-sum buffers summed in each window            */
    int32_t max_batch;    /* largest batch of any step                               */
    int32_t max_ctx;      /* most tokens ever cached per sequence; KV capacity is max_ctx + 1 */
    float   rms_eps;      /* RMSNorm epsilon (inside the square root)                */
    float   rope_theta;   /* rotary base; <= 0 disables the rotary embedding         */
    uint32_t flags;       /* PRESERVE_FLAG_*                                         */
} preserve_layer_config_t;

/* Device pointers, row-major [in, out] (y = x W), no biases. */
typedef struct {
    const void *w_q;      /* [hidden, n_q_heads*head_dim]  */
    const void *w_k;      /* [hidden, n_kv_heads*head_dim] */
    const void *w_v;      /* [hidden, n_kv_heads*head_dim] */
    const void *w_o;      /* [n_q_heads*head_dim, hidden]  */
    const void *w_gate;   /* [hidden, ffn]                 */
    const void *w_up;     /* [hidden, ffn]                 */
    const void *w_down;   /* [ffn, hidden]                 */
    const void *g_attn;   /* [hidden] RMSNorm gain before attention */
    const void *g_mlp;    /* [hidden] RMSNorm gain before the MLP   */
} preserve_layer_weights_t;

/* One decode step.  ctx_len[b] = tokens already cached for sequence b; the
 * step writes the new key/value at slot ctx_len[b] and attends over slots
 * 0..ctx_len[b].  The library never advances ctx_len. */
typedef struct {
    int32_t batch;                          /* 1..max_batch                                         */
    const int32_t *ctx_len;                 /* device [batch], each 0..max_ctx                      */
    const int32_t *ctx_len_host;            /* host copy of the same values (used for planning)     */
    const void *const *partials_in;         /* host array of P device pointers, each [batch,hidden]:
                                               the partial sums reduced in the first window         */
    const void *const *attn_peer_partials;  /* host array of P-1 device pointers, [batch,hidden]:
                                               the other shards' attention partial sums (second
                                               window; slot 0 there is this shard's own result)      */
    const void *residual_in;                /* device [batch,hidden]                                */
    void *k_cache;                          /* device [max_batch,n_kv_heads,max_ctx+1,head_dim]     */
    void *v_cache;                          /* same shape; both are read, and written at one slot   */
    void *residual_out;                     /* device [batch,hidden]: residual after the attention block */
    void *mlp_partial_out;                  /* device [batch,hidden]: this shard's MLP partial sum  */
    void *attn_partial_out;                 /* optional (NULL ok) [batch,hidden]: attention partial sum */
} preserve_step_io_t;

/* Same step with HOST activation buffers: the call copies partials, peers and
 * residual to the device, runs the step and copies the two outputs back, all on
 * the given stream.  The KV-cache stays on the device. */
typedef struct {
    int32_t batch;
    const int32_t *ctx_len_host;            /* host [batch]                                          */
    const void *const *partials_in;         /* host array of P HOST pointers, [batch,hidden]         */
    const void *const *attn_peer_partials;  /* host array of P-1 HOST pointers                       */
    const void *residual_in;                /* HOST [batch,hidden]                                   */
    void *k_cache, *v_cache;                /* device                                                */
    void *residual_out;                     /* HOST [batch,hidden]                                   */
    void *mlp_partial_out;                  /* HOST [batch,hidden]                                   */
} preserve_host_io_t;

typedef struct {
    int32_t sm_count;
    int32_t l2_bytes;                 /* cudaDevAttrL2CacheSize                         */
    int32_t max_persisting_l2_bytes;  /* cudaDevAttrMaxPersistingL2CacheSize            */
    int32_t max_access_window_bytes;  /* cudaDevAttrMaxAccessPolicyWindowSize           */
    int32_t uses_tensor_path;         /* 1: tcgen05 GEMM (max_batch >= 16); 0: split-K GEMV */
    int32_t activation_rows;          /* rows per plane of the internal split activations (see preserve_debug_copy) */
    int32_t plan_mode;
    int32_t normed_activations_fp16;  /* 1 (tensor path): o, x2 and a are one fp16 plane each, x two fp16 planes; see preserve_debug_copy */
    uint64_t prefetch_budget;         /* bytes per window                               */
    uint64_t weight_bytes[4];         /* Wqkv, Wo, Wgate|up, Wdown                      */
    uint64_t kv_bytes;                /* K+V bytes read by the last planned step        */
    uint64_t planned_bytes[2][3];     /* last plan: window A {Wqkv,KV,Wo}; window B {Wgate|up,Wdown,-} */
    uint64_t algorithmic_bytes;       /* weights + KV + activations of the last planned step */
} preserve_info_t;

/* Create a layer: validates the sizes, packs the weights into a library-owned
 * arena laid out in the order the kernels consume them, allocates workspaces,
 * a side stream and events on the CURRENT device.  The weight pointers may be
 * freed after the call returns.  *out is NULL on failure.
 * The prefetch budget starts at the library's default (reported by preserve_layer_get_info as
 * prefetch_budget; see preserve_set_prefetch_bytes), mode PRESERVE_PLAN_TRUNCATE. */
PRESERVE_API int preserve_layer_init(const preserve_layer_config_t *cfg, const preserve_layer_weights_t *w,
                        preserve_layer_t **out);

/* Layout of one int8 cache buffer (PRESERVE_FLAG_INT8_KV) for a configuration: bytes [0, S * cap * head_dim)
 * hold the codes, int8 [max_batch, n_kv_heads, cap, head_dim] with cap = max_ctx + 1 and S = max_batch *
 * n_kv_heads; the scales follow at *scale_offset_bytes (the code bytes rounded up to 256): fp32 [max_batch,
 * n_kv_heads, *scale_capacity], *scale_capacity = cap rounded up to 64 (entries at and beyond cap are never
 * used).  *buffer_bytes = the size to allocate for each of k_cache and v_cache (16-byte aligned base).
 * Slots at and beyond ctx_len[b] are never read, whatever they hold.  Host only; no device work. */
PRESERVE_API int preserve_kv8_layout(const preserve_layer_config_t *cfg, uint64_t *scale_offset_bytes,
                                     int32_t *scale_capacity, uint64_t *buffer_bytes);

/* Upper limit, in bytes, on what one window's prefetch may bring into L2
 * (Algorithm 1's C; Section 3 "L2 capacity requirements").
 * 0 = vanilla execution (Section 3, "Vanilla execution"): nothing is fetched ahead of
 * the data dependency - no side-stream work, and every kernel starts only after its
 * predecessor has completed.
 * > 0 = the read-only operands of the operators after a window are brought on chip
 * while the window runs, in two tiers: (1) the consumer kernels are launched early
 * (programmatic dependent launch) and stage the leading part of their weights / cached
 * K and V in shared memory before they wait for the window's result; (2) a side-stream
 * kernel prefetches the planned byte ranges, up to this limit per window, into L2.
 * The library's default is PRESERVE_BUDGET_EARLY_LAUNCH_ONLY: tier 1 alone, which is the fastest
 * setting measured with the single-GPU stand-in windows (they last a few microseconds, too short
 * for off-chip memory to be idle); give a real budget (a sixteenth to a quarter of the L2 size)
 * where the communication window lasts 10 us or more. */
#define PRESERVE_BUDGET_EARLY_LAUNCH_ONLY ((size_t)1)   /* any budget below 128 bytes plans nothing for L2 */
PRESERVE_API int preserve_set_prefetch_bytes(preserve_layer_t *layer, size_t bytes_per_window);

/* How the side-stream kernel brings the planned bytes into L2: mechanism 0 =
 * cp.async.bulk.prefetch.L2 (one instruction per chunk_bytes; the default, with 4096-byte chunks
 * from 128 CTAs), 1 = prefetch.global.L2 per 128-byte line, 2 = plain loads whose values are
 * dropped (the control: completion then implies arrival).  chunk_bytes a multiple of 128, at most
 * 1 MiB; 1 <= ctas <= 1024.  Results never depend on it. */
PRESERVE_API int preserve_set_prefetch_mechanism(preserve_layer_t *layer, int32_t mechanism, uint32_t chunk_bytes,
                                                 int32_t ctas);

/* Modelled communication latency: every window kernel additionally waits (bounded, on
 * the GPU's global timer) until `ns` nanoseconds after its start before it delivers its
 * result, standing in for the network time of a real allreduce, which the single-GPU
 * stand-in does not have.  0 (default) = no added wait.  At most 1,000,000. */
PRESERVE_API int preserve_set_window_delay_ns(preserve_layer_t *layer, int32_t ns);

/* PRESERVE_PLAN_WHOLE_NODE (Algorithm 1 as printed) or PRESERVE_PLAN_TRUNCATE. */
PRESERVE_API int preserve_set_plan_mode(preserve_layer_t *layer, int mode);

/* Queue one decode step of this layer on `cuda_stream` (a cudaStream_t; NULL =
 * the legacy default stream).  Steps: window A (sum of partials_in + residual_in,
 * RMSNorm) || prefetch {Wqkv, K/V, Wo};  QKV projection + rotary embedding + KV
 * append;  split-KV attention;  output projection;  window B (own + peers'
 * attention partials + residual, RMSNorm) || prefetch {Wgate|up, Wdown};  gate/up
 * projection + SwiGLU;  down projection. */
PRESERVE_API int preserve_decode_step(preserve_layer_t *layer, const preserve_step_io_t *io, void *cuda_stream);

/* Queue n layers back to back (a chain): ios[i] describes layer i's buffers as
 * given; when link != 0, layer i+1's partials_in[0] and residual_in are layer
 * i's MLP partial sum and residual, handed over inside the library unrounded
 * (fp32) instead of ios[i+1]'s pointers; layer i's bf16 outputs are still
 * written.  All layers must share batch and hidden.  The whole chain is replayed
 * as one CUDA graph. */
PRESERVE_API int preserve_decode_chain(preserve_layer_t *const *layers, int32_t n, const preserve_step_io_t *ios,
                          int32_t link, void *cuda_stream);

/* The step with host activation buffers (see preserve_host_io_t).  When every
 * input buffer is pinned (page-locked) host memory, one gather kernel on a
 * stream owned by the layer reads the inputs over PCIe into the layer's device
 * staging area (that read is the host-to-device transfer) while whatever was
 * queued on `cuda_stream` before this call is still running, and the step
 * waits only for that gather; pinned output buffers are written directly by
 * the kernels that produce the results.  Pageable buffers are copied with
 * copy calls on `cuda_stream` instead.  As with every entry point the results
 * are complete once the work queued on `cuda_stream` has completed.  Calls on
 * one layer share its staging area: the gather of a call starts when the step
 * of the previous call on that layer has finished. */
PRESERVE_API int preserve_decode_step_host(preserve_layer_t *layer, const preserve_host_io_t *io, void *cuda_stream);

/* Per-kernel device times of one step.  Runs the step with direct launches on
 * `cuda_stream` (prefetch on the side stream as usual), with CUDA events recorded
 * on that stream around each main-stream kernel, waits for the stream, and writes
 * PRESERVE_N_KERNELS durations in milliseconds: window A, QKV projection, split-KV
 * attention, attention merge, output projection, window B, gate/up projection,
 * down projection.  Results of the step are the same as preserve_decode_step's. */
#define PRESERVE_N_KERNELS 8
PRESERVE_API int preserve_profile_step(preserve_layer_t *layer, const preserve_step_io_t *io, void *cuda_stream,
                                       float *kernel_ms);

/* Queue ONE main-stream kernel of the step (index as in preserve_profile_step) with the
 * step's arguments, directly on `cuda_stream`, without prefetch.  For benchmarks that time a
 * kernel on its own; the buffers it reads must hold the results of an earlier full step. */
PRESERVE_API int preserve_run_kernel(preserve_layer_t *layer, const preserve_step_io_t *io, int32_t which,
                                     void *cuda_stream);

/* Queue only the L2 prefetch that belongs beside window `window` (0: {Wqkv, K/V, Wo}; 1: {Wgate|up,
 * Wdown}; planned against the budget as in a full step) on the layer's side stream, forked from
 * `cuda_stream` at this point.  For a caller that runs the communication itself (a library
 * all-reduce between kernels queued with preserve_run_kernel): call this right before the
 * collective, the place Algorithm 1 inserts the prefetch operator.  The side stream is joined
 * again by preserve_run_kernel of the block's last kernel (4 for window 0, 7 for window 1). */
PRESERVE_API int preserve_prefetch_window(preserve_layer_t *layer, const preserve_step_io_t *io, int32_t window,
                                          void *cuda_stream);

/* Timeline trace (diagnostics).  While on, every main-stream kernel of a step records, over all
 * its CTAs, PRESERVE_TRACE_SLOTS values in nanoseconds of the GPU's global timer: {earliest
 * start, earliest and latest return from the wait on the previous kernel, latest end, latest
 * start, latest end of the operand-streaming loop (0 where a kernel has none), earliest end,
 * unused}.  preserve_read_trace synchronises the device, copies PRESERVE_N_KERNELS x
 * PRESERVE_TRACE_SLOTS values (kernel order as in preserve_profile_step) to `out` (host) and
 * clears the slots.  Results of the step do not change. */
#define PRESERVE_TRACE_SLOTS 8
PRESERVE_API int preserve_set_trace(preserve_layer_t *layer, int32_t on);
PRESERVE_API int preserve_read_trace(preserve_layer_t *layer, int64_t *out);

/* Sizes, device attributes and the last plan. */
PRESERVE_API int preserve_layer_get_info(const preserve_layer_t *layer, preserve_info_t *info);

/* Synchronises the device and returns the layer's device status word: PRESERVE_OK;
 * PRESERVE_ETIMEOUT if a bounded wait gave up (the step's results are then undefined, the
 * handle stays usable); PRESERVE_ESHAPE if the device copy of ctx_len described more
 * attention work than the host copy the step was planned with.  The word keeps the first
 * failure until preserve_clear_status. */
PRESERVE_API int preserve_last_status(preserve_layer_t *layer);
PRESERVE_API int preserve_clear_status(preserve_layer_t *layer);

/* The raw device status word behind preserve_last_status (synchronises the device): 0 ok;
 * 1 a wait for operand bytes (TMA / bulk copy / cluster hand-over) gave up; 2 a wait for a free
 * ring slot; 3 a wait for the tensor-core accumulator or a cluster reduction; 4 tensor memory;
 * 5 device ctx_len beyond the host copy; 6 a peer rank never announced its exchange buffer. */
PRESERVE_API int preserve_last_status_code(preserve_layer_t *layer);

/* Graphs captured so far by calls whose first (or only) layer is this handle.  Replays of
 * a cached graph do not count: a decode loop whose contexts advance should see this number
 * grow only when the attention work split changes (about once per 64 tokens at most). */
PRESERVE_API int64_t preserve_graph_captures(const preserve_layer_t *layer);

/* Test hooks.  PRESERVE_DEBUG_WAIT_LIMIT_CYCLES: upper limit, in SM clock cycles, on every
 * bounded device-side wait of this handle's kernels (0 = the built-in limit of 2^31 cycles,
 * about a second; waits shorter than 2^19 cycles are never cut).  PRESERVE_DEBUG_WITHHOLD:
 * 0 = off; otherwise ONE producer of one kernel of the next steps withholds ONE issue - 1: a
 * CTA of the first window's row cluster does not hand over its sum of squares (needs hidden >=
 * 2048); 2: a warp of the QKV GEMV never fills its first ring slot; 3: a CTA of the tcgen05 QKV
 * GEMM never fetches its first weight tile; 4: the first attention CTA never fetches one box of
 * its first tile - so that the consumer's bounded wait runs out, the kernel gives up and returns,
 * and preserve_last_status reports PRESERVE_ETIMEOUT.  Nothing faults or hangs. */
#define PRESERVE_DEBUG_WITHHOLD          0
#define PRESERVE_DEBUG_WAIT_LIMIT_CYCLES 1
PRESERVE_API int preserve_debug_set(preserve_layer_t *layer, int32_t what, int64_t value);

/* The cudaError_t of the most recent failing CUDA call made for this handle. */
PRESERVE_API int preserve_last_cuda_error(const preserve_layer_t *layer);

/* Copy an intermediate of the last step into a caller's device buffer (for
 * kernel-level checks).  which: 0 h (fp32 [max_batch,hidden]); 1 x, 2 q (after the
 * rotary embedding, [.., n_q_heads, head_dim]), 3 o (attention output, same shape),
 * 4 x2, 5 a ([.., ffn]).  1..5 are kept internally as two bf16 planes, value =
 * hi + lo, laid out [2][activation_rows][...] (activation_rows from
 * preserve_layer_get_info); the copy delivers that layout as is.  Exception: where
 * normed_activations_fp16 is set (tensor path), o, x2 and a - an attention output, an RMSNorm output
 * and the SwiGLU output (clamped to +-65504): bounded values - are ONE fp16 plane each,
 * [activation_rows][...] at the start of the buffer, and the two planes of x are fp16 (hi = fp16(x),
 * lo = fp16(x - hi)).  6: uint64 [2][3], the
 * bytes per node that the prefetch kernels of the last step decided to bring in - the same
 * walk as preserve_layer_get_info's planned_bytes, evaluated on the device from the device
 * copy of ctx_len (a window whose host plan is empty launches no kernel and keeps its old
 * values).  `bytes` must not exceed the buffer's size.  Asynchronous on `cuda_stream`. */
PRESERVE_API int preserve_debug_copy(preserve_layer_t *layer, int32_t which, void *dst_device, size_t bytes,
                        void *cuda_stream);

/* Decode attention that allocates nothing.  (The paper has no counterpart to this
 * entry point; it exists for callers of this library.)
 *
 * Who it is for: code that must not, or cannot, call cudaMalloc at the moment it needs
 * attention - a step that runs inside a memory-frozen region of a serving process, a
 * plug-in that is handed device buffers by its host and has no allocator of its own, a
 * caller that is already capturing a stream (allocation is illegal during capture).
 * preserve_layer_init allocates workspaces; this call never does, and needs no handle.
 *
 * What it computes: for every sequence b and query head h, softmax(q . K^T / sqrt(128)) V
 * over cache slots 0..ctx_len[b] (ctx_len[b] + 1 keys: the newest entry must already be
 * in the cache), grouped-query layout as in preserve_step_io_t, by the same split-KV
 * kernel and merge kernel as the layer path.  The split-KV partial results live in a
 * fixed PRESERVE_STATIC_SCRATCH_BYTES array that is part of the library image: every
 * GPU that loads the library holds that much memory until the process exits.
 *
 * Arguments: q_hi/q_lo and o_hi/o_lo are device bf16 [batch, n_q_heads, 128]; a value is
 * hi + lo (pass a zero-filled q_lo for plain bf16 queries; o_lo receives the rounding
 * remainder of the output).  k_cache/v_cache are device bf16
 * [batch, n_kv_heads, kv_capacity, 128].  ctx_len is a device array, ctx_len_host the same
 * values on the host; each 0..kv_capacity-1.  At most 16 query heads per KV head.
 *
 * Limits and errors: the partials of the call's work items (runs of 64-key tiles of one
 * sequence and KV head; at most 8 x SM count + batch x n_kv_heads of them, 520 bytes per query
 * head of the group each) must fit in the scratch array, else PRESERVE_ETOOBIG is returned and nothing is queued; other
 * bad arguments return PRESERVE_EINVAL / _EALIGN / _ESHAPE.
 *
 * Sharing: all calls on one GPU use the same array, and it keeps whatever the previous
 * call left there (the call clears the one word that must start at zero).  Two calls that
 * overlap on the GPU - different streams, or different threads - race on it; serialise them.
 *
 * First call: the first call on each device looks up the array's device address and sets
 * the kernels' shared-memory limit, which are synchronous set-up steps; make that first
 * call outside any stream capture.  Later calls only queue work on `cuda_stream`.
 *
 * Status: the bounded waits of the two kernels report into the first word of the array;
 * preserve_attention_static_status() waits for the current device and returns PRESERVE_OK,
 * PRESERVE_ETIMEOUT (a wait gave up: o is undefined) or PRESERVE_ESHAPE (the device ctx_len
 * described more work than ctx_len_host: the surplus was dropped, nothing was written out
 * of bounds, o is wrong).  It allocates nothing either. */
#define PRESERVE_STATIC_SCRATCH_BYTES (8u << 20)
PRESERVE_API int preserve_attention_static(const void *q_hi, const void *q_lo, const void *k_cache,
                                           const void *v_cache, const int32_t *ctx_len,
                                           const int32_t *ctx_len_host, int32_t batch, int32_t n_q_heads,
                                           int32_t n_kv_heads, int32_t kv_capacity, void *o_hi, void *o_lo,
                                           void *cuda_stream);
PRESERVE_API int preserve_attention_static_status(void);

/* ---- The real communication window (one process per GPU; Section 2, "Multi-device inference":
 * one all-reduce of a [batch, hidden] tensor per attention block and one per MLP block).
 *
 * A preserve_comm_t owns this rank's EXCHANGE BLOCK in device memory: its two partial-sum buffers
 * (window A: what its down projection produced; window B: what its output projection produced),
 * arrival flags and epoch counters.  preserve_comm_create allocates the block on the current
 * device (n_ranks <= 8); the ranks then exchange 64-byte handles (preserve_comm_export on the
 * owner, preserve_comm_import on every other rank; how the bytes travel is the caller's business -
 * the Python layer uses torch.distributed), which maps every peer's block into this process (CUDA
 * IPC, peer access enabled lazily).  Inside ONE process, preserve_comm_set_peer connects blocks
 * directly.  All peers must be connected before preserve_layer_set_comm.
 *
 * With a comm attached (n_ranks must equal tp_degree), a step's two windows become one-shot
 * all-reduces fused into the window kernel: the output / down projections also write this rank's
 * bf16 partial sums into its exchange buffers; each window kernel, once its own buffer is complete,
 * stores the window's epoch number into every peer's flag block, waits - bounded by the handle's
 * wait limit, PRESERVE_ETIMEOUT / status code 6 if a peer never arrives - until every peer has done
 * the same, then reads all n_ranks buffers through the peer mappings with plain 128-bit loads and
 * adds them in rank order (identical bits on every rank), adds the residual and normalises.
 * io->partials_in and io->attn_peer_partials are then ignored.  Window A of a step reads what the
 * down projection of the step before wrote (for the very first step: what preserve_comm_write put
 * there).  Every rank must queue the same sequence of steps.  Several layers may share one comm.
 * No multicast and no bulk / TMA copy ever touches a peer's memory.
 *
 * preserve_comm_write: copy `bytes` of device data into this rank's own buffer of `window` (0 = A,
 * 1 = B), asynchronously on the stream.  preserve_comm_epoch: windows of that kind this rank has
 * completed (synchronises).  preserve_comm_debug_arrive (tests on one GPU, where no second rank
 * runs): marks `from_rank` as having announced every window up to `epoch` in this rank's flag
 * block, from the host. */
typedef struct preserve_comm preserve_comm_t;
PRESERVE_API int preserve_comm_create(int32_t rank, int32_t n_ranks, int32_t max_batch, int32_t hidden,
                                      preserve_comm_t **out);
PRESERVE_API int preserve_comm_export(const preserve_comm_t *comm, void *handle64);
PRESERVE_API int preserve_comm_import(preserve_comm_t *comm, int32_t peer_rank, const void *handle64);
PRESERVE_API int preserve_comm_set_peer(preserve_comm_t *comm, int32_t peer_rank, const preserve_comm_t *peer);
PRESERVE_API int preserve_comm_write(preserve_comm_t *comm, int32_t window, const void *src_device, size_t bytes,
                                     void *cuda_stream);
PRESERVE_API int preserve_comm_debug_arrive(preserve_comm_t *comm, int32_t window, int32_t from_rank, uint32_t epoch);
PRESERVE_API int64_t preserve_comm_epoch(preserve_comm_t *comm, int32_t window);
PRESERVE_API void preserve_comm_destroy(preserve_comm_t *comm);
PRESERVE_API int preserve_layer_set_comm(preserve_layer_t *layer, preserve_comm_t *comm_or_null);

/* For a window whose all-reduce the CALLER performs (the library-collective baseline): window B
 * then takes `reduced_attn_partial` (device bf16 [batch, hidden], e.g. the NCCL all-reduce of
 * attn_partial_out) as its partial 0 instead of this shard's own result; NULL restores the
 * default.  The caller runs the step kernel by kernel (preserve_run_kernel) and reduces between
 * the output projection (4) and window B (5).  Not together with a comm. */
PRESERVE_API int preserve_layer_set_external_attention_sum(preserve_layer_t *layer, const void *reduced_attn_partial);

/* Read-bandwidth microbenchmark (the read roofline next to the copy-bandwidth figure): streams
 * `bytes` (>= 1 MiB, 16-byte aligned) of the caller's device buffer `reps` times (1..1000) with
 * 128-bit loads from 4 CTAs per SM and writes GB/s to *gbs_out.  A buffer several times larger
 * than L2 measures HBM; a buffer well inside L2 measures L2.  Synchronises `cuda_stream`;
 * allocates nothing. */
PRESERVE_API int preserve_measure_read_bandwidth(const void *device_buffer, size_t bytes, int32_t reps,
                                                 void *cuda_stream, float *gbs_out);

/* Streaming-read microbenchmark in ONE launch: `ctas` CTAs each walk their own contiguous slice
 * of the caller's device buffer (128-byte aligned) `passes` times inside the kernel, so launch
 * ramp and tail are paid once.  A buffer well inside L2 with many passes measures L2; a buffer
 * several times larger than L2 measures HBM; ctas = 1 measures what one SM can take in.
 * path 0: 128-bit read-only loads (256 threads, 8 loads in flight each); path 1: bulk async
 * copies of chunk_bytes (multiple of 1024) issued by `producers` (1..8) threads per CTA, each
 * keeping `stages` (1..12) copies in flight in its own shared-memory ring, stages * chunk_bytes *
 * producers <= 200 KiB; path 2: the same with the issuing threads being lanes of one warp.
 * status_block: 64 zeroed device ints (the
 * bounded waits of path 1 report there).  Writes GB/s to *gbs_out; synchronises `cuda_stream`;
 * allocates nothing. */
PRESERVE_API int preserve_measure_stream(const void *device_buffer, size_t bytes, int32_t passes, int32_t path,
                                         int32_t ctas, int32_t stages, uint32_t chunk_bytes, int32_t producers,
                                         int32_t *status_block, void *cuda_stream, float *gbs_out);

/* The same measurement with the tcgen05 GEMM's kind of weight load: 2-D tiled TMA copies (128-byte
 * swizzle) of boxes of 64 columns x box_rows rows (8..256, multiple of 8) out of the buffer viewed as
 * a [bytes / 16384, 8192] bf16 matrix; CTA c walks the 128 column blocks of row tile c mod (number
 * of tiles) `passes` times, its `producers` issuing threads taking every producers-th block. */
PRESERVE_API int preserve_measure_stream_tma(const void *device_buffer, size_t bytes, int32_t passes, int32_t ctas,
                                             int32_t stages, int32_t box_rows, int32_t producers,
                                             int32_t *status_block, void *cuda_stream, float *gbs_out);

/* Frees everything the library allocated for the handle (NULL is allowed). */
PRESERVE_API void preserve_layer_destroy(preserve_layer_t *layer);

/* Static description of a PRESERVE_E* code. */
PRESERVE_API const char *preserve_strerror(int code);

/* Host-only: prefetch planning for one window (Algorithm 1 applied to an
 * ordered list of MatMul / SelfAttention nodes between two communication ops).
 * node_bytes[i] = bytes a prefetch of node i brings in; out_bytes[i] receives
 * what is prefetched (0, the whole node, or in TRUNCATE mode a leading part
 * rounded down to 128 bytes).  Needs no GPU. */
PRESERVE_API int preserve_plan_window(const uint64_t *node_bytes, int32_t n_nodes, uint64_t budget, int32_t mode,
                         uint64_t *out_bytes);

/* Host-only: Algorithm 1 as a pass over an explicit operator graph (the form the paper gives
 * it: for every communication operator, a breadth-first walk over its successors up to the next
 * communication operator or the end of the graph, inserting a prefetch for every MatMul and
 * SelfAttention node while the running sum of their sizes stays below the budget).
 * kind[i] is PRESERVE_NODE_*; mem_bytes[i] what a prefetch of node i brings in (weights, or K+V;
 * ignored for other kinds); successors of node i are succ[succ_off[i] .. succ_off[i+1]).  Writes
 * one (communication op, node, bytes) triple per inserted prefetch, in insertion order, and their
 * number to *n_out; PRESERVE_ETOOBIG (with *n_out set) if there are more than max_out.  A layer's
 * own step plan is this pass applied to the layer's operator chain. */
#define PRESERVE_NODE_COMM      0
#define PRESERVE_NODE_MATMUL    1
#define PRESERVE_NODE_ATTENTION 2
#define PRESERVE_NODE_OTHER     3
PRESERVE_API int preserve_plan_graph(int32_t n_nodes, const int32_t *kind, const uint64_t *mem_bytes,
                                     const int32_t *succ_off, const int32_t *succ, uint64_t budget, int32_t mode,
                                     int32_t max_out, int32_t *out_comm, int32_t *out_node, uint64_t *out_bytes,
                                     int32_t *n_out);

/* Host-only: bytes one step must move once (weights + K/V of the cached tokens
 * + activations), the numerator of the effective-bandwidth figure.
 * sum_ctx = sum over the batch of tokens already cached. */
PRESERVE_API uint64_t preserve_algorithmic_bytes(const preserve_layer_config_t *cfg, int32_t batch, uint64_t sum_ctx);

#ifdef __cplusplus
}
#endif
#endif /* PRESERVE_H */
