/*
 * CPU oracle for the cloud-side verification step of Synera (arxiv 2511.07423).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, definition-level restatement of
 * what the step computes, used to check the CUDA library and to provide the timed CPU
 * baseline.  Only tests, the smoke check and the benchmark's CPU-baseline leg may call
 * it; the product never does, and the two share no code.
 *
 * What is computed (paper passages):
 *   - A verification request = cached tokens + uncached device-accepted tokens +
 *     pending-verify tokens (Sec. 3.4); the uncached and pending tokens are forwarded
 *     "like a prefill, but with an existing KV-cached prefix": partial prefill (Sec. 3.4,
 *     Takeaway-3; Sec. 4.5).
 *   - Attention(Q,K,V) = softmax(Q K^T / sqrt(d_k)) V (Sec. 3.2, unnumbered equation),
 *     causal inside the chunk, over the cached prefix read through the page table.
 *   - After the forward pass, verification uses the engine outputs
 *     q(x|prefix), ..., q(x|prefix, x~_1..x~_gamma) (Sec. 4.5): gamma+1 distributions for
 *     gamma drafts.  Greedy "draft & verify" (Sec. 3.1, Fig. "Draft & verify"): accept
 *     drafts while they equal the LLM's argmax; the LLM's argmax at the first mismatch
 *     is the correction; if all are accepted the last distribution gives a bonus token.
 *
 * The paper does not fix the model internals; the decoder is the Llama family it
 * evaluates (RMSNorm, rotary embedding with rotate-half pairing, grouped-query attention,
 * SwiGLU), no biases.  All arithmetic is in `real` (double by default; -DORC_F32 builds the
 * single-precision variant).  Weights arrive as bf16 bit patterns and are widened exactly.
 * Sums run in index order except the long dot products, which use ORC_LANES interleaved
 * partial sums combined in lane order (a fixed summation order, nothing else is blocked,
 * fused or reordered).
 *
 * Pins (tests/test_oracle_*.py): dense full-matrix attention on a contiguous rebuild of the
 * sequence, paged == contiguous and page-permutation invariance, chunk == token-by-token,
 * batch-composition invariance, hand-worked accept cases and slot maps, closed forms
 * (zeroed projections, q = 0, equal V rows, RoPE at position 0 and relative-position
 * property), greedy losslessness, and the capped-geometric acceptance expectation
 * (Sec. 5).  Absolute logit values at the large shapes have no external pin
 * ("parity unpinned" for those magnitudes): they rest on the small-shape pins plus
 * shape-generic code.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef ORC_F32
typedef float real;
#define ORC_REAL_BYTES 4
#else
typedef double real;
#define ORC_REAL_BYTES 8
#endif

#define ORC_LANES 8

typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    double rope_base, rms_eps;
    int32_t bf16_operands; /* 0: every intermediate stays in `real`.  1: the model as a bf16 model
                              ("bf16 weights and activations, fp32 accumulation"): every activation
                              that enters a matrix product or the KV cache is first rounded to bf16
                              (normalised hidden states, rotated q and k, v, the attention output,
                              the SwiGLU output); sums, softmax and the residual stream stay wide. */
} orc_desc;

int orc_real_bytes(void) { return ORC_REAL_BYTES; }

static inline real bf16_widen(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return (real)f;
}

/* round to the nearest bf16 (ties to even), returned in `real` */
static inline real bf16_round(real v) {
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) != 0x7F800000u) u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    memcpy(&f, &u, 4);
    return (real)f;
}
static void round_all(real *a, size_t n) {
    for (size_t i = 0; i < n; ++i) a[i] = bf16_round(a[i]);
}

void orc_bf16_round_array(const real *in, real *out, int n) {
    for (int i = 0; i < n; ++i) out[i] = bf16_round(in[i]);
}

/* x_j = E[c_j]  (token embedding lookup) */
void orc_embed(const uint16_t *E, int d, const int32_t *tok, int n, real *x) {
    for (int j = 0; j < n; ++j)
        for (int i = 0; i < d; ++i) x[(size_t)j * d + i] = bf16_widen(E[(size_t)tok[j] * d + i]);
}

/* RMSNorm: out = x / sqrt(mean(x^2) + eps) * g, row by row */
void orc_rmsnorm(const real *x, const uint16_t *g, int n, int d, double eps, real *out) {
    for (int j = 0; j < n; ++j) {
        real ss = 0;
        for (int i = 0; i < d; ++i) ss += x[(size_t)j * d + i] * x[(size_t)j * d + i];
        real r = (real)1 / (real)sqrt((double)(ss / (real)d) + eps);
        for (int i = 0; i < d; ++i) out[(size_t)j * d + i] = x[(size_t)j * d + i] * r * bf16_widen(g[i]);
    }
}

static inline real dot_w(const real *x, const uint16_t *w, int K) {
    real acc[ORC_LANES];
    for (int l = 0; l < ORC_LANES; ++l) acc[l] = 0;
    int k = 0;
    for (; k + ORC_LANES <= K; k += ORC_LANES)
        for (int l = 0; l < ORC_LANES; ++l) acc[l] += x[k + l] * bf16_widen(w[k + l]);
    for (int l = 0; k < K; ++k, ++l) acc[l] += x[k] * bf16_widen(w[k]);
    real s = 0;
    for (int l = 0; l < ORC_LANES; ++l) s += acc[l];
    return s;
}

/* y[j][o] = sum_k x[j][k] * W[o][k];  W is [N][K] row-major bf16 (out-features by in-features) */
void orc_linear(const real *x, const uint16_t *W, int n, int K, int N, real *y) {
#pragma omp parallel for schedule(static)
    for (int o = 0; o < N; ++o)
        for (int j = 0; j < n; ++j) y[(size_t)j * N + o] = dot_w(x + (size_t)j * K, W + (size_t)o * K, K);
}

/* Rotary embedding of one token's heads, rotate-half pairing (i, i + hd/2),
 * theta_i = base^(-2i/hd), angle = pos * theta_i, evaluated in double. */
void orc_rope(real *v, int n_heads, int hd, int pos, double base) {
    int half = hd / 2;
    for (int h = 0; h < n_heads; ++h) {
        real *p = v + (size_t)h * hd;
        for (int i = 0; i < half; ++i) {
            double ang = (double)pos * pow(base, -2.0 * (double)i / (double)hd);
            real c = (real)cos(ang), s = (real)sin(ang);
            real a = p[i], b = p[i + half];
            p[i] = a * c - b * s;
            p[i + half] = b * c + a * s;
        }
    }
}

/* KV pool of one layer: [n_pages][2 (K,V)][n_kv_heads][page_size][head_dim].
 * Position p of a request lives in physical page page_table[p / P], row p % P. */
static inline size_t pool_index(const orc_desc *m, int P, int page, int which, int kvh, int row) {
    return ((((size_t)page * 2 + which) * m->n_kv_heads + kvh) * P + row) * (size_t)m->head_dim;
}

void orc_slot(const int32_t *page_table, int P, int pos, int32_t *page, int32_t *row) {
    *page = page_table[pos / P];
    *row = pos % P;
}

void orc_kv_write(const orc_desc *m, real *pool, const int32_t *page_table, int P, int pos,
                  const real *k, const real *v) {
    int32_t page, row;
    orc_slot(page_table, P, pos, &page, &row);
    for (int h = 0; h < m->n_kv_heads; ++h) {
        memcpy(pool + pool_index(m, P, page, 0, h, row), k + (size_t)h * m->head_dim, sizeof(real) * m->head_dim);
        memcpy(pool + pool_index(m, P, page, 1, h, row), v + (size_t)h * m->head_dim, sizeof(real) * m->head_dim);
    }
}

/* Chunk token j (position ctx + j) attends to positions 0 .. ctx + j.
 * q: [n][Hq*hd] (already rotated); out: [n][Hq*hd]. */
void orc_attention(const orc_desc *m, const real *q, const real *pool, const int32_t *page_table, int P,
                   int ctx, int n, real *out) {
    int hd = m->head_dim, G = m->n_q_heads / m->n_kv_heads;
    real scale = (real)(1.0 / sqrt((double)hd));
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int j = 0; j < n; ++j)
        for (int h = 0; h < m->n_q_heads; ++h) {
            int len = ctx + j + 1, kvh = h / G;
            const real *qv = q + ((size_t)j * m->n_q_heads + h) * hd;
            real *s = (real *)malloc(sizeof(real) * (size_t)len);
            real mx = -INFINITY;
            for (int t = 0; t < len; ++t) {
                const real *kv = pool + pool_index(m, P, page_table[t / P], 0, kvh, t % P);
                real a = 0;
                for (int i = 0; i < hd; ++i) a += qv[i] * kv[i];
                s[t] = a * scale;
                if (s[t] > mx) mx = s[t];
            }
            real den = 0;
            for (int t = 0; t < len; ++t) {
                s[t] = (real)exp((double)(s[t] - mx));
                den += s[t];
            }
            real *o = out + ((size_t)j * m->n_q_heads + h) * hd;
            for (int i = 0; i < hd; ++i) o[i] = 0;
            for (int t = 0; t < len; ++t) {
                const real *vv = pool + pool_index(m, P, page_table[t / P], 1, kvh, t % P);
                real w = s[t] / den;
                for (int i = 0; i < hd; ++i) o[i] += w * vv[i];
            }
            free(s);
        }
}

typedef struct {
    const uint16_t *wq, *wk, *wv, *wo, *wg, *wu, *wd, *norm1, *norm2;
} orc_layer_weights;

/* One decoder layer over one request's chunk: x [n][d] is updated in place, the chunk's
 * K and V are appended to the pool at positions ctx .. ctx+n-1. */
void orc_layer(const orc_desc *m, const orc_layer_weights *w, real *x, real *pool,
               const int32_t *page_table, int P, int ctx, int n) {
    int d = m->d_model, qd = m->n_q_heads * m->head_dim, kd = m->n_kv_heads * m->head_dim, f = m->d_ffn;
    real *h = (real *)malloc(sizeof(real) * (size_t)n * d);
    real *q = (real *)malloc(sizeof(real) * (size_t)n * qd);
    real *k = (real *)malloc(sizeof(real) * (size_t)n * kd);
    real *v = (real *)malloc(sizeof(real) * (size_t)n * kd);
    real *a = (real *)malloc(sizeof(real) * (size_t)n * qd);
    real *o = (real *)malloc(sizeof(real) * (size_t)n * d);
    real *g = (real *)malloc(sizeof(real) * (size_t)n * f);
    real *u = (real *)malloc(sizeof(real) * (size_t)n * f);

    const int rb = m->bf16_operands;
    orc_rmsnorm(x, w->norm1, n, d, m->rms_eps, h);
    if (rb) round_all(h, (size_t)n * d);
    orc_linear(h, w->wq, n, d, qd, q);
    orc_linear(h, w->wk, n, d, kd, k);
    orc_linear(h, w->wv, n, d, kd, v);
    for (int j = 0; j < n; ++j) {
        orc_rope(q + (size_t)j * qd, m->n_q_heads, m->head_dim, ctx + j, m->rope_base);
        orc_rope(k + (size_t)j * kd, m->n_kv_heads, m->head_dim, ctx + j, m->rope_base);
        if (rb) {
            round_all(q + (size_t)j * qd, (size_t)qd);
            round_all(k + (size_t)j * kd, (size_t)kd);
            round_all(v + (size_t)j * kd, (size_t)kd);
        }
        orc_kv_write(m, pool, page_table, P, ctx + j, k + (size_t)j * kd, v + (size_t)j * kd);
    }
    orc_attention(m, q, pool, page_table, P, ctx, n, a);
    if (rb) round_all(a, (size_t)n * qd);
    orc_linear(a, w->wo, n, qd, d, o);
    for (size_t i = 0; i < (size_t)n * d; ++i) x[i] += o[i];

    orc_rmsnorm(x, w->norm2, n, d, m->rms_eps, h);
    if (rb) round_all(h, (size_t)n * d);
    orc_linear(h, w->wg, n, d, f, g);
    orc_linear(h, w->wu, n, d, f, u);
    for (size_t i = 0; i < (size_t)n * f; ++i) {
        real z = g[i];
        g[i] = z / ((real)1 + (real)exp((double)-z)) * u[i]; /* silu(gate) * up */
    }
    if (rb) round_all(g, (size_t)n * f);
    orc_linear(g, w->wd, n, f, d, o);
    for (size_t i = 0; i < (size_t)n * d; ++i) x[i] += o[i];

    free(h); free(q); free(k); free(v); free(a); free(o); free(g); free(u);
}

/* Final norm, vocabulary projection, greedy argmax (lowest id on ties), and the runner-up.
 * logits may be NULL.  top2/gap describe the second-largest logit (lowest id on ties). */
void orc_logits(const orc_desc *m, const uint16_t *final_norm, const uint16_t *lm_head, const real *x, int n,
                real *logits, int32_t *top1, int32_t *top2, real *gap) {
    int d = m->d_model, V = m->vocab;
    real *h = (real *)malloc(sizeof(real) * (size_t)n * d);
    real *l = logits ? logits : (real *)malloc(sizeof(real) * (size_t)n * V);
    orc_rmsnorm(x, final_norm, n, d, m->rms_eps, h);
    if (m->bf16_operands) round_all(h, (size_t)n * d);
    orc_linear(h, lm_head, n, d, V, l);
    for (int j = 0; j < n; ++j) {
        const real *r = l + (size_t)j * V;
        int b1 = 0;
        for (int t = 1; t < V; ++t) if (r[t] > r[b1]) b1 = t;
        int b2 = -1;
        for (int t = 0; t < V; ++t) if (t != b1 && (b2 < 0 || r[t] > r[b2])) b2 = t;
        top1[j] = b1;
        if (top2) top2[j] = b2;
        if (gap) gap[j] = b2 >= 0 ? r[b1] - r[b2] : (real)INFINITY;
    }
    free(h);
    if (!logits) free(l);
}

/* Greedy verification of one request.  chunk = [u accepted tokens | n-u drafts]; the
 * distribution at chunk index u-1+j judges draft j.  accept_len = number of leading
 * drafts equal to the argmax; correction = argmax at the first mismatch, or the bonus
 * token (argmax after the last draft) when every draft is accepted. */
void orc_verify(const int32_t *top1, const int32_t *chunk, int n, int u, int32_t *accept_len,
                int32_t *correction) {
    int a = 0;
    while (a < n - u && top1[u - 1 + a] == chunk[u + a]) ++a;
    *accept_len = a;
    *correction = top1[u - 1 + a];
}
