/*
 * CPU oracle for one tensor-parallel shard's decode step of a decoder layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA path is checked against.  It shares no code with the CUDA library and
 * must never be called from the product path; only the tests, the smoke check
 * and the benchmark's CPU-baseline leg use it.
 *
 * What it computes.  Prefetching moves read-only weights and KV-cache entries
 * closer to the cores and changes no value (Section 3, "Execution with the
 * proposed method"), so the result of the accelerated step is exactly the
 * result of the plain layer.  The paper names the layer's parts without
 * writing equations (Section 2, "LLM inference workloads": three input
 * projections, a positional embedding, a self-attention kernel, an output
 * projection; three MLP projections and an activation; normalisation layers)
 * and fixes the sharding (Section 2, "Multi-device inference": attention split
 * by heads, MLP split along the intermediate dimension, one allreduce per
 * block).  The readings taken where the paper is silent:
 *   - pre-norm Llama-style layer; the communication window delivers
 *     h = residual + sum of the P partial-sum buffers, followed by RMSNorm;
 *   - RMSNorm: x = h * (mean(h^2) + eps)^(-1/2) * gain, eps inside the root,
 *     the gain is used as given;
 *   - rotary position embedding with half-split pairing (i, i + d/2), angle
 *     t * theta^(-2i/d), position t = number of tokens already cached;
 *     theta <= 0 switches it off;
 *   - the step appends k, v at slot t and attends over slots 0..t with scale
 *     1/sqrt(d), max-subtracted softmax, no other mask;
 *   - grouped-query attention: query head hq reads KV head hq / G;
 *   - SwiGLU: silu(x W_gate) * (x W_up), silu(z) = z / (1 + exp(-z));
 *   - no biases; weights are [in, out] row-major.
 * Precision: inputs are bf16 bit patterns widened exactly to fp32; every
 * intermediate VALUE is stored as fp32 and is never rounded to bf16; every sum
 * (dot products, mean of squares, softmax denominator) is accumulated in
 * double so the result does not depend on summation order.  One rounding is part
 * of the definition: the KV-cache is a bf16 array, the step writes the new key
 * and value into it and the self-attention kernel reads the cache (Section 3,
 * "Execution with the proposed method": the cache is read-only in decode except
 * for the last entry, which the preceding projections update), so attention
 * sees the new entry as stored, i.e. rounded to bf16 (nearest even).  k_new and
 * v_new are reported unrounded.
 *
 * Pins (tests, CPU only): brute-force attention on tiny inputs, softmax rows
 * summing to one, uniform-key and dominant-key special cases, GQA == MHA with
 * repeated KV heads, split-and-merge of the key range, RMSNorm closed forms,
 * identity / one-hot projections, RoPE norm and relative-position invariants,
 * silu constants, sum over both shards == unsharded layer, and an independent
 * torch-CPU restatement of the layer.  The int8 variants (weights per output
 * channel; KV-cache per cached vector) have their own pins: hand-worked vectors,
 * the half-step error bound, symmetry and power-of-two covariance of the
 * quantisers, brute force on the dequantised arrays, agreement with the bf16
 * routines on data that both represent exactly, and the torch restatement with
 * its own quantiser.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t hidden;       /* H */
    int32_t n_q_heads;    /* per shard */
    int32_t n_kv_heads;   /* per shard */
    int32_t head_dim;     /* d */
    int32_t ffn;          /* F, per shard */
    int32_t tp_degree;    /* P */
    int32_t batch;        /* B */
    int32_t kv_capacity;  /* slots per (sequence, kv head) in the cache arrays */
    float rms_eps;
    float rope_theta;
} oracle_cfg_t;

typedef struct {          /* caller-allocated fp32 outputs; any may be NULL */
    float *h;             /* [B,H]  window A sum                          */
    float *x;             /* [B,H]  RMSNorm(h; g_attn)                    */
    float *q;             /* [B,nq,d] after RoPE                          */
    float *k_new;         /* [B,nkv,d] after RoPE (value appended)        */
    float *v_new;         /* [B,nkv,d]                                    */
    float *o;             /* [B,nq,d] attention output                    */
    float *attn_partial;  /* [B,H]  o . W_o                               */
    float *h2;            /* [B,H]  window B sum                          */
    float *x2;            /* [B,H]  RMSNorm(h2; g_mlp)                    */
    float *a;             /* [B,F]  SwiGLU activation                     */
    float *mlp_partial;   /* [B,H]  a . W_down                            */
} oracle_out_t;

typedef struct {          /* int8 KV-cache of a step (see oracle_quantize_rows)              */
    const int8_t *k_codes, *v_codes;    /* [B,nkv,cap,d]                                    */
    const float *k_scales, *v_scales;   /* [B,nkv,cap]                                      */
    int8_t *k_codes_new, *v_codes_new;  /* optional outputs [B,nkv,d]: the appended entry   */
    float *k_scale_new, *v_scale_new;   /* optional outputs [B,nkv]                         */
} oracle_kv8_t;

static inline float bf16f(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* fp32 -> nearest-even bf16, returned widened to fp32 (the value a bf16 cache slot holds) */
static inline float round_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u)
        return f;                       /* NaN stays NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Window: h = r + sum_p part_p ; x = h * (mean h^2 + eps)^(-1/2) * g.
 * parts: [n_parts][B*H] fp32 (contiguous), r: [B*H] fp32, g: bf16 [H]. */
void oracle_window(int B, int H, int n_parts, const float *parts, const float *r,
                   const uint16_t *g, float eps, float *h, float *x)
{
#pragma omp parallel for schedule(static)
    for (int b = 0; b < B; ++b) {
        double ms = 0.0;
        for (int j = 0; j < H; ++j) {
            double s = (double)r[(size_t)b * H + j];
            for (int p = 0; p < n_parts; ++p)
                s += (double)parts[((size_t)p * B + b) * H + j];
            float hv = (float)s;
            h[(size_t)b * H + j] = hv;
            ms += (double)hv * (double)hv;
        }
        double inv = 1.0 / sqrt(ms / (double)H + (double)eps);
        for (int j = 0; j < H; ++j)
            x[(size_t)b * H + j] = (float)((double)h[(size_t)b * H + j] * inv * (double)bf16f(g[j]));
    }
}

/* y[b,n] = sum_k x[b,k] * W[k,n];  W bf16 [K,N] row-major, x fp32 [B,K], y fp32 [B,N]. */
void oracle_matmul(int B, int K, int N, const float *x, const uint16_t *w, float *y)
{
#pragma omp parallel
    {
        /* column n of W, widened once and reused for every batch row */
        float *col = (float *)malloc(sizeof(float) * (size_t)(K ? K : 1));
#pragma omp for schedule(static)
        for (int n = 0; n < N; ++n) {
            for (int k = 0; k < K; ++k)
                col[k] = bf16f(w[(size_t)k * N + n]);
            for (int b = 0; b < B; ++b) {
                double acc = 0.0;
                for (int k = 0; k < K; ++k)
                    acc += (double)x[(size_t)b * K + k] * (double)col[k];
                y[(size_t)b * N + n] = (float)acc;
            }
        }
        free(col);
    }
}

/* ---- int8 weights (the precision of the paper's measurements: Section 4, "Experimental setup").
 * The paper does not say how its int8 weights are scaled; reading: symmetric per-output-channel
 * quantisation.  For output column n of W [K,N]: scale_n = max_k |W[k,n]| / 127 (fp32 division),
 * code q[k,n] = round-to-nearest-even(W[k,n] / scale_n) in fp32, an integer in [-127, 127]; a column of
 * zeros has scale 0 and codes 0.  The layer then computes y[b,n] = scale_n * sum_k x[b,k] q[k,n].
 * The decision of every code is taken in fp32 (one correctly rounded division, one rint), which is
 * what the CUDA side does too, so the codes agree bit for bit. */
void oracle_quantize_weights(int K, int N, const uint16_t *w, int8_t *q, float *scale)
{
    for (int n = 0; n < N; ++n) {
        float mx = 0.f;
        for (int k = 0; k < K; ++k) {
            float v = fabsf(bf16f(w[(size_t)k * N + n]));
            if (v > mx)
                mx = v;
        }
        float sc = mx / 127.0f;
        scale[n] = sc;
        for (int k = 0; k < K; ++k) {
            float v = bf16f(w[(size_t)k * N + n]);
            float r = sc > 0.f ? rintf(v / sc) : 0.f;
            if (r > 127.f) r = 127.f;
            if (r < -127.f) r = -127.f;
            q[(size_t)k * N + n] = (int8_t)r;
        }
    }
}

/* y[b,n] = scale[n] * sum_k x[b,k] q[k,n], sums in double */
void oracle_matmul_q8(int B, int K, int N, const float *x, const int8_t *q, const float *scale, float *y)
{
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int b = 0; b < B; ++b) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k)
                acc += (double)x[(size_t)b * K + k] * (double)q[(size_t)k * N + n];
            y[(size_t)b * N + n] = (float)(acc * (double)scale[n]);
        }
}

/* the projection of the layer: bf16 weights as they are, or quantised to int8 first */
static int layer_matmul(int B, int K, int N, const float *x, const uint16_t *w, float *y, int w8)
{
    if (!w8) {
        oracle_matmul(B, K, N, x, w, y);
        return 0;
    }
    int8_t *q = (int8_t *)malloc((size_t)K * N);
    float *sc = (float *)malloc(sizeof(float) * (size_t)N);
    if (!q || !sc) {
        free(q);
        free(sc);
        return -1;
    }
    oracle_quantize_weights(K, N, w, q, sc);
    oracle_matmul_q8(B, K, N, x, q, sc, y);
    free(q);
    free(sc);
    return 0;
}

/* Rotary embedding in place on u[n_heads][d] at position t (half-split pairs). */
void oracle_rope(int n_heads, int d, int t, float theta, float *u)
{
    if (!(theta > 0.0f))
        return;
    int half = d / 2;
    for (int hd = 0; hd < n_heads; ++hd) {
        float *p = u + (size_t)hd * d;
        for (int i = 0; i < half; ++i) {
            double ang = (double)t * pow((double)theta, -2.0 * (double)i / (double)d);
            double c = cos(ang), s = sin(ang);
            double a = p[i], bb = p[i + half];
            p[i] = (float)(a * c - bb * s);
            p[i + half] = (float)(bb * c + a * s);
        }
    }
}

/* Decode attention for one step.
 * q [B,nq,d] fp32; k_new,v_new [B,nkv,d] fp32 (the entry of slot ctx_len[b]);
 * k_cache,v_cache bf16 [B,nkv,cap,d] (slots < ctx_len[b] are read);
 * o [B,nq,d]; probs (optional) [B,nq,cap] receives the softmax row. */
void oracle_attention(int B, int nq, int nkv, int d, int cap, const int32_t *ctx_len,
                      const float *q, const float *k_new, const float *v_new,
                      const uint16_t *k_cache, const uint16_t *v_cache, float *o, float *probs)
{
    int G = nq / nkv;
    double scale = 1.0 / sqrt((double)d);
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * nq; ++bh) {
        int b = bh / nq, hq = bh % nq, g = hq / G;
        int t = ctx_len[b];
        const float *qv = q + ((size_t)b * nq + hq) * d;
        const uint16_t *kc = k_cache + ((size_t)b * nkv + g) * (size_t)cap * d;
        const uint16_t *vc = v_cache + ((size_t)b * nkv + g) * (size_t)cap * d;
        const float *kn = k_new + ((size_t)b * nkv + g) * d;
        const float *vn = v_new + ((size_t)b * nkv + g) * d;
        double *s = (double *)malloc(sizeof(double) * (size_t)(t + 1));
        double *acc = (double *)calloc((size_t)d, sizeof(double));
        double mx = -INFINITY;
        for (int j = 0; j <= t; ++j) {
            double dot = 0.0;
            if (j < t)
                for (int i = 0; i < d; ++i)
                    dot += (double)qv[i] * (double)bf16f(kc[(size_t)j * d + i]);
            else
                for (int i = 0; i < d; ++i)
                    dot += (double)qv[i] * (double)kn[i];
            s[j] = dot * scale;
            if (s[j] > mx)
                mx = s[j];
        }
        double den = 0.0;
        for (int j = 0; j <= t; ++j) {
            s[j] = exp(s[j] - mx);
            den += s[j];
        }
        for (int j = 0; j <= t; ++j) {
            double p = s[j] / den;
            if (probs)
                probs[((size_t)b * nq + hq) * cap + j] = (float)p;
            if (j < t)
                for (int i = 0; i < d; ++i)
                    acc[i] += p * (double)bf16f(vc[(size_t)j * d + i]);
            else
                for (int i = 0; i < d; ++i)
                    acc[i] += p * (double)vn[i];
        }
        for (int i = 0; i < d; ++i)
            o[((size_t)b * nq + hq) * d + i] = (float)acc[i];
        free(s);
        free(acc);
    }
}

/* ---- int8 KV-cache (the precision of the paper's measurements: Section 4, "Experimental setup").
 * The paper does not say how its int8 cache is scaled; reading: symmetric quantisation with one
 * scale per cached vector, i.e. per (sequence, kv head, slot), keys and values alike.  For a vector
 * u of d values: scale = max_i |u_i| / 127 (fp32 division), code_i = round-to-nearest-even(u_i / scale)
 * in fp32, an integer in [-127, 127]; a vector of zeros has scale 0 and codes 0.  The cache holds
 * the codes and the scales, and the value a slot stands for is code * scale.  Every decision is
 * taken in fp32, so a CUDA side that is given the same fp32 vector produces the same codes. */
void oracle_quantize_rows(size_t n_rows, int d, const float *u, int8_t *q, float *scale)
{
    for (size_t r = 0; r < n_rows; ++r) {
        const float *v = u + r * (size_t)d;
        float mx = 0.f;
        for (int i = 0; i < d; ++i)
            if (fabsf(v[i]) > mx)
                mx = fabsf(v[i]);
        float sc = mx / 127.0f;
        scale[r] = sc;
        for (int i = 0; i < d; ++i) {
            float c = sc > 0.f ? rintf(v[i] / sc) : 0.f;
            if (c > 127.f) c = 127.f;
            if (c < -127.f) c = -127.f;
            q[r * (size_t)d + i] = (int8_t)c;
        }
    }
}

/* Decode attention over an int8 cache.  q [B,nq,d] fp32; the entry of slot ctx_len[b] is given
 * already quantised: kq_new, vq_new int8 [B,nkv,d] with ks_new, vs_new [B,nkv]; the cache is
 * k_codes, v_codes int8 [B,nkv,cap,d] with k_scales, v_scales fp32 [B,nkv,cap] (slots < ctx_len[b]
 * are read).  Every key and value enters as code * scale; o [B,nq,d]; probs optional [B,nq,cap]. */
void oracle_attention_kv8(int B, int nq, int nkv, int d, int cap, const int32_t *ctx_len, const float *q,
                          const int8_t *kq_new, const float *ks_new, const int8_t *vq_new, const float *vs_new,
                          const int8_t *k_codes, const float *k_scales, const int8_t *v_codes,
                          const float *v_scales, float *o, float *probs)
{
    int G = nq / nkv;
    double scale = 1.0 / sqrt((double)d);
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * nq; ++bh) {
        int b = bh / nq, hq = bh % nq, g = hq / G;
        int t = ctx_len[b];
        size_t stream = (size_t)b * nkv + g;
        const float *qv = q + ((size_t)b * nq + hq) * d;
        double *s = (double *)malloc(sizeof(double) * (size_t)(t + 1));
        double *acc = (double *)calloc((size_t)d, sizeof(double));
        double mx = -INFINITY;
        for (int j = 0; j <= t; ++j) {
            const int8_t *kc = j < t ? k_codes + (stream * (size_t)cap + j) * d : kq_new + stream * d;
            double ks = j < t ? (double)k_scales[stream * (size_t)cap + j] : (double)ks_new[stream];
            double dot = 0.0;
            for (int i = 0; i < d; ++i)
                dot += (double)qv[i] * ((double)kc[i] * ks);
            s[j] = dot * scale;
            if (s[j] > mx)
                mx = s[j];
        }
        double den = 0.0;
        for (int j = 0; j <= t; ++j) {
            s[j] = exp(s[j] - mx);
            den += s[j];
        }
        for (int j = 0; j <= t; ++j) {
            const int8_t *vc = j < t ? v_codes + (stream * (size_t)cap + j) * d : vq_new + stream * d;
            double vs = j < t ? (double)v_scales[stream * (size_t)cap + j] : (double)vs_new[stream];
            double p = s[j] / den;
            if (probs)
                probs[((size_t)b * nq + hq) * cap + j] = (float)p;
            for (int i = 0; i < d; ++i)
                acc[i] += p * ((double)vc[i] * vs);
        }
        for (int i = 0; i < d; ++i)
            o[((size_t)b * nq + hq) * d + i] = (float)acc[i];
        free(s);
        free(acc);
    }
}

/* a[i] = silu(gate[i]) * up[i] */
void oracle_swiglu(size_t n, const float *gate, const float *up, float *a)
{
    for (size_t i = 0; i < n; ++i) {
        double z = gate[i];
        a[i] = (float)(z / (1.0 + exp(-z)) * (double)up[i]);
    }
}

static float *falloc(size_t n) { return (float *)malloc(sizeof(float) * (n ? n : 1)); }

/* One decode step of one shard's layer.
 * partials_in [P][B][H] fp32, peer_partials [P-1][B][H] fp32, residual_in [B][H] fp32
 * (the bf16 inputs widened exactly, or a previous layer's unrounded outputs in a chain).
 * Weights bf16 [in,out] row-major; gains bf16 [H]; caches bf16 [B,nkv,cap,d] (read only).
 * Returns 0, or -1 on a bad configuration / allocation failure. */
static int layer_step_impl(const oracle_cfg_t *c, const uint16_t *w_q, const uint16_t *w_k,
                           const uint16_t *w_v, const uint16_t *w_o, const uint16_t *w_gate,
                           const uint16_t *w_up, const uint16_t *w_down, const uint16_t *g_attn,
                           const uint16_t *g_mlp, const int32_t *ctx_len, const float *partials_in,
                           const float *peer_partials, const float *residual_in,
                           const uint16_t *k_cache, const uint16_t *v_cache, oracle_out_t *out, int w8,
                           const oracle_kv8_t *kv8)
{
    int B = c->batch, H = c->hidden, nq = c->n_q_heads, nkv = c->n_kv_heads, d = c->head_dim;
    int F = c->ffn, P = c->tp_degree, cap = c->kv_capacity;
    if (B < 1 || H < 1 || nq < 1 || nkv < 1 || nq % nkv || d < 2 || d % 2 || F < 1 || P < 1)
        return -1;
    for (int b = 0; b < B; ++b)
        if (ctx_len[b] < 0 || ctx_len[b] >= cap)
            return -1;
    size_t BH = (size_t)B * H;
    float *h = falloc(BH), *x = falloc(BH), *q = falloc((size_t)B * nq * d);
    float *kn = falloc((size_t)B * nkv * d), *vn = falloc((size_t)B * nkv * d);
    float *o = falloc((size_t)B * nq * d), *ap = falloc(BH), *h2 = falloc(BH), *x2 = falloc(BH);
    float *gate = falloc((size_t)B * F), *up = falloc((size_t)B * F), *a = falloc((size_t)B * F);
    float *mp = falloc(BH), *parts2 = falloc((size_t)P * BH);
    float *kn_c = falloc((size_t)B * nkv * d), *vn_c = falloc((size_t)B * nkv * d);
    int rc = -1;
    if (!h || !x || !q || !kn || !vn || !o || !ap || !h2 || !x2 || !gate || !up || !a || !mp || !parts2 || !kn_c || !vn_c)
        goto done;

    /* window A: sum of the P partial buffers + residual, then RMSNorm */
    oracle_window(B, H, P, partials_in, residual_in, g_attn, c->rms_eps, h, x);
    /* input projections */
    layer_matmul(B, H, nq * d, x, w_q, q, w8);
    layer_matmul(B, H, nkv * d, x, w_k, kn, w8);
    layer_matmul(B, H, nkv * d, x, w_v, vn, w8);
    /* positional embedding at position ctx_len[b] on q and the new k */
    for (int b = 0; b < B; ++b) {
        oracle_rope(nq, d, ctx_len[b], c->rope_theta, q + (size_t)b * nq * d);
        oracle_rope(nkv, d, ctx_len[b], c->rope_theta, kn + (size_t)b * nkv * d);
    }
    if (!kv8) {
        /* append: the new entry is stored in the bf16 cache; attention reads it from there */
        for (size_t i = 0; i < (size_t)B * nkv * d; ++i) {
            kn_c[i] = round_to_bf16(kn[i]);
            vn_c[i] = round_to_bf16(vn[i]);
        }
        /* self-attention over the cached entries plus the new one */
        oracle_attention(B, nq, nkv, d, cap, ctx_len, q, kn_c, vn_c, k_cache, v_cache, o, NULL);
    } else {
        /* append: the new entry is stored in the int8 cache (codes and one scale per vector);
         * attention reads every entry, the new one included, as code * scale */
        size_t nv = (size_t)B * nkv;
        int8_t *kq = (int8_t *)malloc(nv * d), *vq = (int8_t *)malloc(nv * d);
        float *ks = falloc(nv), *vs = falloc(nv);
        if (!kq || !vq || !ks || !vs) {
            free(kq); free(vq); free(ks); free(vs);
            goto done;
        }
        oracle_quantize_rows(nv, d, kn, kq, ks);
        oracle_quantize_rows(nv, d, vn, vq, vs);
        oracle_attention_kv8(B, nq, nkv, d, cap, ctx_len, q, kq, ks, vq, vs, kv8->k_codes, kv8->k_scales,
                             kv8->v_codes, kv8->v_scales, o, NULL);
        if (kv8->k_codes_new) memcpy(kv8->k_codes_new, kq, nv * d);
        if (kv8->v_codes_new) memcpy(kv8->v_codes_new, vq, nv * d);
        if (kv8->k_scale_new) memcpy(kv8->k_scale_new, ks, sizeof(float) * nv);
        if (kv8->v_scale_new) memcpy(kv8->v_scale_new, vs, sizeof(float) * nv);
        free(kq); free(vq); free(ks); free(vs);
    }
    /* output projection: this shard's partial sum */
    layer_matmul(B, nq * d, H, o, w_o, ap, w8);
    /* window B: own partial + the P-1 peers' partials + h, then RMSNorm */
    memcpy(parts2, ap, sizeof(float) * BH);
    if (P > 1)
        memcpy(parts2 + BH, peer_partials, sizeof(float) * BH * (size_t)(P - 1));
    oracle_window(B, H, P, parts2, h, g_mlp, c->rms_eps, h2, x2);
    /* MLP */
    layer_matmul(B, H, F, x2, w_gate, gate, w8);
    layer_matmul(B, H, F, x2, w_up, up, w8);
    oracle_swiglu((size_t)B * F, gate, up, a);
    layer_matmul(B, F, H, a, w_down, mp, w8);

#define COPY_OUT(dst, src, n) \
    if (out->dst) memcpy(out->dst, src, sizeof(float) * (n))
    COPY_OUT(h, h, BH);
    COPY_OUT(x, x, BH);
    COPY_OUT(q, q, (size_t)B * nq * d);
    COPY_OUT(k_new, kn, (size_t)B * nkv * d);
    COPY_OUT(v_new, vn, (size_t)B * nkv * d);
    COPY_OUT(o, o, (size_t)B * nq * d);
    COPY_OUT(attn_partial, ap, BH);
    COPY_OUT(h2, h2, BH);
    COPY_OUT(x2, x2, BH);
    COPY_OUT(a, a, (size_t)B * F);
    COPY_OUT(mlp_partial, mp, BH);
#undef COPY_OUT
    rc = 0;
done:
    free(h); free(x); free(q); free(kn); free(vn); free(o); free(ap); free(h2); free(x2);
    free(gate); free(up); free(a); free(mp); free(parts2); free(kn_c); free(vn_c);
    return rc;
}

int oracle_layer_step(const oracle_cfg_t *c, const uint16_t *w_q, const uint16_t *w_k,
                      const uint16_t *w_v, const uint16_t *w_o, const uint16_t *w_gate,
                      const uint16_t *w_up, const uint16_t *w_down, const uint16_t *g_attn,
                      const uint16_t *g_mlp, const int32_t *ctx_len, const float *partials_in,
                      const float *peer_partials, const float *residual_in,
                      const uint16_t *k_cache, const uint16_t *v_cache, oracle_out_t *out)
{
    return layer_step_impl(c, w_q, w_k, w_v, w_o, w_gate, w_up, w_down, g_attn, g_mlp, ctx_len, partials_in,
                           peer_partials, residual_in, k_cache, v_cache, out, 0, NULL);
}

/* The same step with every projection's weights quantised to int8 per output channel
 * (oracle_quantize_weights) before use. */
int oracle_layer_step_w8(const oracle_cfg_t *c, const uint16_t *w_q, const uint16_t *w_k,
                         const uint16_t *w_v, const uint16_t *w_o, const uint16_t *w_gate,
                         const uint16_t *w_up, const uint16_t *w_down, const uint16_t *g_attn,
                         const uint16_t *g_mlp, const int32_t *ctx_len, const float *partials_in,
                         const float *peer_partials, const float *residual_in,
                         const uint16_t *k_cache, const uint16_t *v_cache, oracle_out_t *out)
{
    return layer_step_impl(c, w_q, w_k, w_v, w_o, w_gate, w_up, w_down, g_attn, g_mlp, ctx_len, partials_in,
                           peer_partials, residual_in, k_cache, v_cache, out, 1, NULL);
}

/* The same step over an int8 KV-cache (oracle_quantize_rows, oracle_attention_kv8); the weights are
 * bf16 (int8_weights == 0) or quantised per output channel as in oracle_layer_step_w8. */
int oracle_layer_step_kv8(const oracle_cfg_t *c, const uint16_t *w_q, const uint16_t *w_k,
                          const uint16_t *w_v, const uint16_t *w_o, const uint16_t *w_gate,
                          const uint16_t *w_up, const uint16_t *w_down, const uint16_t *g_attn,
                          const uint16_t *g_mlp, const int32_t *ctx_len, const float *partials_in,
                          const float *peer_partials, const float *residual_in, const oracle_kv8_t *kv8,
                          int int8_weights, oracle_out_t *out)
{
    if (!kv8 || !kv8->k_codes || !kv8->v_codes || !kv8->k_scales || !kv8->v_scales)
        return -1;
    return layer_step_impl(c, w_q, w_k, w_v, w_o, w_gate, w_up, w_down, g_attn, g_mlp, ctx_len, partials_in,
                           peer_partials, residual_in, NULL, NULL, out, int8_weights ? 1 : 0, kv8);
}
