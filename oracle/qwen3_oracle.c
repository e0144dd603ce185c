/*
 * qwen3_oracle.c -- CPU oracle for the Qwen3-architecture decoder forward pass.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA library is checked against.
 * Only the tests, the smoke check and the benchmark's cpu-baseline leg may build or call it; the product
 * path never does.  It shares no code, header, table or helper with the CUDA sources.
 *
 * What it follows.  The paper (Section 4, "Evaluation") fixes the workload only: Qwen3 decoder-only models,
 * batch 1, a prompt phase followed by token-by-token decoding, F32 as the reference precision.  It does not
 * restate the model's arithmetic; that comes from the public Qwen3 architecture the paper cites, with the
 * readings listed beside each function below.  Arithmetic is fp32 on bf16-valued weights; the K/V cache is
 * bf16 (round-to-nearest-even on write).  Compiling with -DORC_ACC_DOUBLE makes every reduction accumulate
 * in double: the difference between the two builds is the oracle's own rounding-order error bar.
 *
 * Pins (tests/test_oracle_*.py): closed forms and invariants of each function, and an independently written
 * unfused float64 numpy forward on small shapes.  The paper prints no logits or tokens, so end-to-end values
 * are "parity unpinned" by the paper itself; they are pinned by those invariants and the numpy forward only.
 *
 * Layouts: every matrix is row-major W[out][in], y = W x.  bf16 values travel as uint16_t bit patterns.
 * There is no blocking, fusion or reordering here beyond "for each layer, for each token".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef ORC_ACC_DOUBLE
typedef double acc_t;
#define ORC_SQRT sqrt
#define ORC_EXP exp
#else
typedef float acc_t;
#define ORC_SQRT sqrtf
#define ORC_EXP expf
#endif

/* ------------------------------------------------------------------------------------------------ bf16 */

float orc_bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round-to-nearest-even; NaN stays NaN (quiet) */
uint16_t orc_f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

int orc_acc_is_double(void) { return (int)(sizeof(acc_t) == 8); }

/* --------------------------------------------------------------------------------------------- RMSNorm */
/* y_i = x_i * (1 / sqrt(mean_j x_j^2 + eps)) * g_i ; eps inside the root, no mean subtraction, no bias. */
void orc_rmsnorm(const float *x, const uint16_t *gain, int n, float eps, float *y) {
    acc_t ss = 0;
    for (int i = 0; i < n; ++i) ss += (acc_t)x[i] * (acc_t)x[i];
    acc_t inv = (acc_t)1 / ORC_SQRT(ss / (acc_t)n + (acc_t)eps);
    for (int i = 0; i < n; ++i) y[i] = (float)((acc_t)x[i] * inv * (acc_t)orc_bf16_to_f32(gain[i]));
}

/* ------------------------------------------------------------------------------------------------ RoPE */
/* Table row p, pair i (i < d/2): cos and sin of p * theta^(-2i/d), evaluated in double, rounded once to fp32.
 * Layout table[p][i][0] = cos, table[p][i][1] = sin. */
void orc_rope_table(int n_pos, int d, double theta, float *table) {
    int half = d / 2;
    for (int p = 0; p < n_pos; ++p)
        for (int i = 0; i < half; ++i) {
            double inv_freq = pow(theta, -2.0 * (double)i / (double)d);
            double phi = (double)p * inv_freq;
            table[((size_t)p * half + i) * 2 + 0] = (float)cos(phi);
            table[((size_t)p * half + i) * 2 + 1] = (float)sin(phi);
        }
}

/* Half-split pairing: element i rotates with element i + d/2.
 *   y_i       = x_i cos - x_{i+d/2} sin
 *   y_{i+d/2} = x_{i+d/2} cos + x_i sin                                                             */
void orc_rope_apply(float *x, int d, const float *row) {
    int half = d / 2;
    for (int i = 0; i < half; ++i) {
        float c = row[2 * i], s = row[2 * i + 1];
        float a = x[i], b = x[i + half];
        x[i] = a * c - b * s;
        x[i + half] = b * c + a * s;
    }
}

/* ---------------------------------------------------------------------------------------------- matmul */
static inline float dot_bf16_f32(const uint16_t *w, const float *x, int n) {
    acc_t acc = 0;
#pragma omp simd reduction(+ : acc)
    for (int k = 0; k < n; ++k) acc += (acc_t)orc_bf16_to_f32(w[k]) * (acc_t)x[k];
    return (float)acc;
}

/* Y[t][o] = sum_k W[o][k] X[t][k] */
void orc_matmul(const uint16_t *W, const float *X, int T, int n_out, int n_in, float *Y) {
#pragma omp parallel for schedule(static)
    for (int o = 0; o < n_out; ++o)
        for (int t = 0; t < T; ++t)
            Y[(size_t)t * n_out + o] = dot_bf16_f32(W + (size_t)o * n_in, X + (size_t)t * n_in, n_in);
}

/* ------------------------------------------------------ second weight precision: FP8 E4M3, row scales */
/* The paper evaluates two weight precisions of the same models (Section 4.1: F32 and F16 variants).  The second
 * precision of this build is weight-only FP8: every weight row is stored as E4M3 codes (1 sign, 4 exponent bits
 * with bias 7, 3 mantissa bits; exponent 0 = subnormal m * 2^-9; no infinities, S.1111.111 = NaN, largest finite
 * value 448) times one power-of-two scale 2^e per output row.  Reading taken (the paper is silent on quantisation):
 *   e     = the smallest integer with max_k |W[o][k]| <= 448 * 2^e  (0 for an all-zero row),
 *   code  = round-to-nearest-even of W[o][k] / 2^e onto the E4M3 grid, saturating at +-448,
 *   value = e4m3(code) * 2^e -- at most 4 significant bits times a power of two, hence exactly a bf16 value.
 * A model "in FP8" is the same forward pass on the dequantised bf16 matrices, so every other function of this
 * file applies unchanged. */
float orc_e4m3_to_f32(uint8_t c) {
    const int sign = c >> 7, e = (c >> 3) & 15, m = c & 7;
    float v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexpf((float)m, -9);
    else v = ldexpf(1.0f + (float)m / 8.0f, e - 7);
    return sign ? -v : v;
}

uint8_t orc_f32_to_e4m3(float x) {
    const uint8_t sign = signbit(x) ? 0x80 : 0;
    const float a = fabsf(x);
    if (isnan(x)) return 0x7f;
    if (a > 448.0f) return sign | 0x7e;                       /* saturate: 0x7e is 448 */
    if (a < 0.015625f) {                                      /* below 2^-6: the subnormal grid, step 2^-9 */
        const int q = (int)rintf(ldexpf(a, 9));               /* exact scaling; rintf rounds to nearest even */
        return sign | (uint8_t)q;                             /* q == 8 is the smallest normal, code 0x08 */
    }
    int E;
    const float f = frexpf(a, &E);                            /* a = f * 2^E, f in [0.5, 1) */
    int q = (int)rintf((2.0f * f - 1.0f) * 8.0f);             /* mantissa steps of 1/8 above 2^(E-1) */
    int e = E - 1 + 7;
    if (q == 8) { q = 0; ++e; }
    return sign | (uint8_t)((e << 3) | q);                    /* a <= 448 keeps this at or below 0x7e */
}

/* W bf16 [n_out][n_in] -> codes [n_out][n_in], exps [n_out] */
void orc_quantise_rows_e4m3(const uint16_t *W, int n_out, int n_in, uint8_t *codes, int8_t *exps) {
#pragma omp parallel for schedule(static)
    for (int o = 0; o < n_out; ++o) {
        const uint16_t *row = W + (size_t)o * n_in;
        float amax = 0.0f;
        for (int k = 0; k < n_in; ++k) {
            const float a = fabsf(orc_bf16_to_f32(row[k]));
            if (a > amax) amax = a;
        }
        int e = 0;
        if (amax > 0.0f) {
            int E;
            const float f = frexpf(amax, &E);                 /* 448 = 0.875 * 2^9 */
            e = (f <= 0.875f) ? E - 9 : E - 8;
            if (e < -127) e = -127;
            if (e > 127) e = 127;
        }
        exps[o] = (int8_t)e;
        for (int k = 0; k < n_in; ++k)
            codes[(size_t)o * n_in + k] = orc_f32_to_e4m3(ldexpf(orc_bf16_to_f32(row[k]), -e));
    }
}

void orc_dequantise_rows_e4m3(const uint8_t *codes, const int8_t *exps, int n_out, int n_in, uint16_t *W) {
#pragma omp parallel for schedule(static)
    for (int o = 0; o < n_out; ++o)
        for (int k = 0; k < n_in; ++k)
            W[(size_t)o * n_in + k] = orc_f32_to_bf16(ldexpf(orc_e4m3_to_f32(codes[(size_t)o * n_in + k]), exps[o]));
}

/* ------------------------------------------------------------------------------------- softmax / SwiGLU */
float orc_silu(float z) { return (float)((acc_t)z / ((acc_t)1 + ORC_EXP(-(acc_t)z))); }

/* in place: subtract the maximum, exponentiate, divide by the sum */
void orc_softmax(float *s, int n) {
    float m = s[0];
    for (int i = 1; i < n; ++i) m = s[i] > m ? s[i] : m;
    acc_t sum = 0;
    for (int i = 0; i < n; ++i) {
        s[i] = (float)ORC_EXP((acc_t)s[i] - (acc_t)m);
        sum += (acc_t)s[i];
    }
    for (int i = 0; i < n; ++i) s[i] = (float)((acc_t)s[i] / sum);
}

/* One query against n cached positions of one KV head.
 *   s_t = (q . K[t]) / sqrt(d),  w = softmax(s),  o = sum_t w_t V[t]
 * K, V: bf16 [n][d] with row stride `stride` elements.  scratch: n floats. */
void orc_attend(const float *q, const uint16_t *K, const uint16_t *V, int n, int d, size_t stride,
                float *scratch, float *o) {
    acc_t scale = (acc_t)1 / ORC_SQRT((acc_t)d);
    for (int t = 0; t < n; ++t) {
        acc_t acc = 0;
#pragma omp simd reduction(+ : acc)
        for (int i = 0; i < d; ++i) acc += (acc_t)q[i] * (acc_t)orc_bf16_to_f32(K[t * stride + i]);
        scratch[t] = (float)(acc * scale);
    }
    orc_softmax(scratch, n);
    for (int i = 0; i < d; ++i) {
        acc_t acc = 0;
        for (int t = 0; t < n; ++t) acc += (acc_t)scratch[t] * (acc_t)orc_bf16_to_f32(V[t * stride + i]);
        o[i] = (float)acc;
    }
}

/* argmax with lowest index on ties, and the gap between the two largest values.  Logits must be finite: a NaN
 * or an infinity anywhere is reported as index -1 with a NaN margin, never silently ranked. */
void orc_argmax_margin(const float *v, int n, int32_t *idx, float *margin) {
    for (int i = 0; i < n; ++i)
        if (!isfinite(v[i])) {
            *idx = -1;
            *margin = NAN;
            return;
        }
    int best = 0;
    for (int i = 1; i < n; ++i)
        if (v[i] > v[best]) best = i;
    float second = -INFINITY;
    for (int i = 0; i < n; ++i)
        if (i != best && v[i] > second) second = v[i];
    *idx = best;
    *margin = n > 1 ? v[best] - second : INFINITY;
}

/* ----------------------------------------------------------------------------------------------- model */
typedef struct {
    int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, intermediate, vocab, max_seq;
    float rms_eps;
    double rope_theta;
} orc_config;

typedef struct {
    const uint16_t *wq, *wk, *wv, *wo, *w_gate, *w_up, *w_down; /* [nq*d][H] [nkv*d][H] [nkv*d][H] [H][nq*d] [I][H] [I][H] [H][I] */
    const uint16_t *g_in, *g_post, *g_q, *g_k;                  /* [H] [H] [d] [d] */
} orc_layer;

typedef struct orc_model {
    orc_config c;
    const uint16_t *embed, *lm_head, *g_final; /* lm_head == embed when tied */
    orc_layer *layers;
    uint16_t *kc, *vc; /* [L][nkv][max_seq][d] */
    float *rope;       /* [max_seq][d/2][2] */
    int len;           /* cached positions */
} orc_model;

/* Weight arrays stay owned by the caller and must outlive the model.  lm_head may be NULL (tied). */
orc_model *orc_create(const orc_config *c, const uint16_t *embed, const uint16_t *lm_head,
                      const uint16_t *g_final, const orc_layer *layers) {
    if (c->n_q_heads % c->n_kv_heads || c->head_dim % 2) return NULL;
    orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
    m->c = *c;
    m->embed = embed;
    m->lm_head = lm_head ? lm_head : embed;
    m->g_final = g_final;
    m->layers = (orc_layer *)malloc(sizeof(orc_layer) * c->n_layers);
    memcpy(m->layers, layers, sizeof(orc_layer) * c->n_layers);
    size_t kv = (size_t)c->n_layers * c->n_kv_heads * c->max_seq * c->head_dim;
    m->kc = (uint16_t *)calloc(kv, 2);
    m->vc = (uint16_t *)calloc(kv, 2);
    m->rope = (float *)malloc(sizeof(float) * (size_t)c->max_seq * c->head_dim);
    orc_rope_table(c->max_seq, c->head_dim, c->rope_theta, m->rope);
    m->len = 0;
    return m;
}

void orc_destroy(orc_model *m) {
    if (!m) return;
    free(m->layers); free(m->kc); free(m->vc); free(m->rope); free(m);
}

void orc_reset(orc_model *m) { m->len = 0; }
int orc_length(const orc_model *m) { return m->len; }
const float *orc_rope_ptr(const orc_model *m) { return m->rope; }

static size_t kv_off(const orc_model *m, int layer, int head, int pos) {
    return (((size_t)layer * m->c.n_kv_heads + head) * m->c.max_seq + pos) * m->c.head_dim;
}

/* Set the raw cache contents of one layer: k, v bf16 [nkv][n_pos][d]; the cache length becomes n_pos. */
int orc_kv_import(orc_model *m, int layer, const uint16_t *k, const uint16_t *v, int n_pos) {
    if (layer < 0 || layer >= m->c.n_layers || n_pos > m->c.max_seq) return -1;
    int d = m->c.head_dim;
    for (int j = 0; j < m->c.n_kv_heads; ++j) {
        memcpy(m->kc + kv_off(m, layer, j, 0), k + (size_t)j * n_pos * d, (size_t)n_pos * d * 2);
        memcpy(m->vc + kv_off(m, layer, j, 0), v + (size_t)j * n_pos * d, (size_t)n_pos * d * 2);
    }
    m->len = n_pos;
    return 0;
}

/* Copy out the cache of one layer, positions [0, n_pos): k, v bf16 [nkv][n_pos][d]. */
int orc_kv_export(const orc_model *m, int layer, uint16_t *k, uint16_t *v, int n_pos) {
    if (layer < 0 || layer >= m->c.n_layers || n_pos > m->c.max_seq) return -1;
    int d = m->c.head_dim;
    for (int j = 0; j < m->c.n_kv_heads; ++j) {
        memcpy(k + (size_t)j * n_pos * d, m->kc + kv_off(m, layer, j, 0), (size_t)n_pos * d * 2);
        memcpy(v + (size_t)j * n_pos * d, m->vc + kv_off(m, layer, j, 0), (size_t)n_pos * d * 2);
    }
    return 0;
}

/* One decoder layer over T new tokens at positions p0 .. p0+T-1; X[T][H] is updated in place.
 *   h = RMSNorm(x; g_in);  q,k,v = Wq h, Wk h, Wv h
 *   per head: q_i <- RoPE_p(RMSNorm_d(q_i; g_q)),  k_j <- RoPE_p(RMSNorm_d(k_j; g_k))   (norm before rotation)
 *   cache[p] <- bf16(k), bf16(v);  o_i = attention(q_i, cache of head i / G over positions 0..p)  (causal)
 *   x += Wo o;  h = RMSNorm(x; g_post);  x += Wd (silu(Wg h) * (Wu h))                                 */
static void layer_forward(orc_model *m, int l, float *X, int T, int p0) {
    const orc_config *c = &m->c;
    const orc_layer *w = &m->layers[l];
    int H = c->hidden, d = c->head_dim, nq = c->n_q_heads, nkv = c->n_kv_heads, I = c->intermediate;
    int G = nq / nkv, qd = nq * d, kd = nkv * d;
    float *Hn = (float *)malloc(sizeof(float) * (size_t)T * H);
    float *Q = (float *)malloc(sizeof(float) * (size_t)T * qd);
    float *K = (float *)malloc(sizeof(float) * (size_t)T * kd);
    float *V = (float *)malloc(sizeof(float) * (size_t)T * kd);
    float *O = (float *)malloc(sizeof(float) * (size_t)T * qd);
    float *Y = (float *)malloc(sizeof(float) * (size_t)T * H);
    float *Gt = (float *)malloc(sizeof(float) * (size_t)T * I);
    float *U = (float *)malloc(sizeof(float) * (size_t)T * I);

    for (int s = 0; s < T; ++s) orc_rmsnorm(X + (size_t)s * H, w->g_in, H, c->rms_eps, Hn + (size_t)s * H);
    orc_matmul(w->wq, Hn, T, qd, H, Q);
    orc_matmul(w->wk, Hn, T, kd, H, K);
    orc_matmul(w->wv, Hn, T, kd, H, V);

    for (int s = 0; s < T; ++s) {
        int p = p0 + s;
        const float *row = m->rope + (size_t)p * d;
        for (int i = 0; i < nq; ++i) {
            float *q = Q + (size_t)s * qd + (size_t)i * d;
            orc_rmsnorm(q, w->g_q, d, c->rms_eps, q);
            orc_rope_apply(q, d, row);
        }
        for (int j = 0; j < nkv; ++j) {
            float *k = K + (size_t)s * kd + (size_t)j * d;
            const float *v = V + (size_t)s * kd + (size_t)j * d;
            orc_rmsnorm(k, w->g_k, d, c->rms_eps, k);
            orc_rope_apply(k, d, row);
            uint16_t *kc = m->kc + kv_off(m, l, j, p), *vc = m->vc + kv_off(m, l, j, p);
            for (int e = 0; e < d; ++e) {
                kc[e] = orc_f32_to_bf16(k[e]);
                vc[e] = orc_f32_to_bf16(v[e]);
            }
        }
    }

#pragma omp parallel
    {
        float *scratch = (float *)malloc(sizeof(float) * (size_t)(p0 + T));
#pragma omp for collapse(2) schedule(dynamic)
        for (int s = 0; s < T; ++s)
            for (int i = 0; i < nq; ++i) {
                int j = i / G, n = p0 + s + 1;
                orc_attend(Q + (size_t)s * qd + (size_t)i * d, m->kc + kv_off(m, l, j, 0),
                           m->vc + kv_off(m, l, j, 0), n, d, (size_t)d, scratch,
                           O + (size_t)s * qd + (size_t)i * d);
            }
        free(scratch);
    }

    orc_matmul(w->wo, O, T, H, qd, Y);
    for (size_t e = 0; e < (size_t)T * H; ++e) X[e] += Y[e];

    for (int s = 0; s < T; ++s) orc_rmsnorm(X + (size_t)s * H, w->g_post, H, c->rms_eps, Hn + (size_t)s * H);
    orc_matmul(w->w_gate, Hn, T, I, H, Gt);
    orc_matmul(w->w_up, Hn, T, I, H, U);
    for (size_t e = 0; e < (size_t)T * I; ++e) Gt[e] = orc_silu(Gt[e]) * U[e];
    orc_matmul(w->w_down, Gt, T, H, I, Y);
    for (size_t e = 0; e < (size_t)T * H; ++e) X[e] += Y[e];

    free(Hn); free(Q); free(K); free(V); free(O); free(Y); free(Gt); free(U);
}

/* Process T new tokens (a prompt, or T = 1 for a decode step) after the `len` positions already cached.
 *   logits: [T][vocab] if all_positions else [vocab] (last token only)
 *   taps:   NULL or [n_layers + 1][T][hidden]: the residual stream after the embedding (index 0) and after
 *           each layer (index l + 1)
 * Returns 0, or -1 if the cache would overflow or a token id is out of range. */
int orc_forward(orc_model *m, const int32_t *tokens, int T, float *logits, int all_positions, float *taps) {
    const orc_config *c = &m->c;
    int H = c->hidden;
    if (T < 1 || m->len + T > c->max_seq) return -1;
    for (int s = 0; s < T; ++s)
        if (tokens[s] < 0 || tokens[s] >= c->vocab) return -1;
    float *X = (float *)malloc(sizeof(float) * (size_t)T * H);
    for (int s = 0; s < T; ++s)
        for (int e = 0; e < H; ++e) X[(size_t)s * H + e] = orc_bf16_to_f32(m->embed[(size_t)tokens[s] * H + e]);
    if (taps) memcpy(taps, X, sizeof(float) * (size_t)T * H);
    for (int l = 0; l < c->n_layers; ++l) {
        layer_forward(m, l, X, T, m->len);
        if (taps) memcpy(taps + (size_t)(l + 1) * T * H, X, sizeof(float) * (size_t)T * H);
    }
    int first = all_positions ? 0 : T - 1, cnt = T - first;
    float *Hn = (float *)malloc(sizeof(float) * (size_t)cnt * H);
    for (int s = 0; s < cnt; ++s)
        orc_rmsnorm(X + (size_t)(first + s) * H, m->g_final, H, c->rms_eps, Hn + (size_t)s * H);
    orc_matmul(m->lm_head, Hn, cnt, c->vocab, H, logits);
    m->len += T;
    free(Hn); free(X);
    return 0;
}

/* One layer, one decode step on a given residual-stream vector (no embedding, no lm_head): the new token
 * sits at position `len`; its k, v are appended and the cache length grows by one. */
int orc_layer_decode(orc_model *m, int layer, const float *x_in, float *x_out) {
    if (layer < 0 || layer >= m->c.n_layers || m->len + 1 > m->c.max_seq) return -1;
    memcpy(x_out, x_in, sizeof(float) * m->c.hidden);
    layer_forward(m, layer, x_out, 1, m->len);
    m->len += 1;
    return 0;
}
