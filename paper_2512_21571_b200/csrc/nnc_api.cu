// The C ABI of libnnc (include/nnc.h): model object, workspace plan, one-time repack, and the two forward
// paths -- the batch-1 decode step (GEMV kernels, captured in a CUDA graph) and the token-batch path (tcgen05
// GEMMs) that serves the prompt phase and batched decode.  Host logic only; every arithmetic step of the
// model runs in the kernels of the neighbouring files.
#include <cuda_runtime.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <tuple>
#include <vector>

#include "common.cuh"
#include "nnc_internal.h"

using namespace nnc;

namespace {

constexpr size_t kAlign = 256;
constexpr int kHostLogitRows = 64;  // rows of logits the *_host variants can stage

struct LayerW {
    bf16 *wqkv, *wo, *wgu, *wd, *g_in, *g_post, *g_q, *g_k;
    // fp16 copies for the prompt-phase GEMMs (null without them), each scaled by a power of two; sc_* point at the
    // DEVICE pair {2^e, 2^-e} of the matrix
    void *wo16, *wgu16, *wd16;
    float *sc_o, *sc_gu, *sc_d;
    // weight_format 1: FP8 E4M3 codes and per-row scales of the four matrices (null otherwise)
    uint8_t *q_qkv, *q_o, *q_gu, *q_d;
    float *s_qkv, *s_o, *s_gu, *s_d;
};

struct Plan {
    size_t total = 0;
    // offsets
    std::vector<size_t> l_wqkv, l_wo, l_wgu, l_wd, l_gin, l_gpost, l_gq, l_gk, l_wo16, l_wgu16, l_wd16;
    std::vector<size_t> l_q8, l_s8;   // FP8: codes of the four matrices back to back, then their row scales
    size_t f16_scales, f16_word, lm_q8, lm_s8, k16, v16;
    size_t embed, lm_head, g_final, kcache, vcache, rope;
    size_t gemv_ctr, gemm_part, gemm_tickets, x, qkv, attn_out, act, part, tickets, am_val, am_idx, am_ticket, d_len, d_status, d_tokens, d_argmax;
    size_t xt, hb, hb_lo, qkvt, ob, ob_lo, ab, ab_lo, logits_stage;
    size_t take(size_t bytes) {
        const size_t o = total;
        total += (bytes + kAlign - 1) / kAlign * kAlign;
        return o;
    }
};

bool valid_config(const nnc_config &c) {
    if (c.n_layers <= 0 || c.hidden <= 0 || c.n_q_heads <= 0 || c.n_kv_heads <= 0 || c.intermediate <= 0 ||
        c.vocab <= 0 || c.max_seq <= 0 || c.max_batch <= 0 || c.max_tokens < c.max_batch)
        return false;
    if (c.head_dim != 128) return false;
    if (c.n_q_heads % c.n_kv_heads) return false;
    const int G = c.n_q_heads / c.n_kv_heads;
    if (!(G == 1 || G == 2 || G == 4 || G == 8)) return false;
    if (c.hidden % 64 || c.intermediate % 64 || c.vocab % 8) return false;
    if ((size_t)c.intermediate * 4 > 200 * 1024 || (size_t)c.n_q_heads * 128 * 4 > 200 * 1024) return false;
    if (!(c.rms_eps > 0.f) || !(c.rope_theta > 1.f)) return false;
    if (c.tc_operands < 0 || c.tc_operands > 2) return false;
    if (c.weight_format < 0 || c.weight_format > 1) return false;
    if (c.weight_format == 1 && (c.hidden % 128 || c.intermediate % 128)) return false;   // the FP8 GEMV's K slices
    return true;
}

// fp16 copies of Wo, Wgate/up and Wdown exist when the model may see calls of more than 128 tokens in operand mode 0
bool wants_f16_copies(const nnc_config &c) { return c.tc_operands == 0 && c.max_tokens > 128; }

void make_plan(const nnc_config &c, Plan &p) {
    const size_t H = c.hidden, qd = (size_t)c.n_q_heads * 128, kd = (size_t)c.n_kv_heads * 128, I = c.intermediate;
    const size_t qkvd = qd + 2 * kd, V = c.vocab, B = c.max_batch, R = c.max_tokens;
    for (int l = 0; l < c.n_layers; ++l) {
        p.l_wqkv.push_back(p.take(qkvd * H * 2));
        p.l_wo.push_back(p.take(H * qd * 2));
        p.l_wgu.push_back(p.take(2 * I * H * 2));
        p.l_wd.push_back(p.take(H * I * 2));
        p.l_gin.push_back(p.take(H * 2));
        p.l_gpost.push_back(p.take(H * 2));
        p.l_gq.push_back(p.take(128 * 2));
        p.l_gk.push_back(p.take(128 * 2));
        if (c.weight_format == 1) {
            p.l_q8.push_back(p.take(qkvd * H + H * qd + 2 * I * H + H * I));
            p.l_s8.push_back(p.take((qkvd + H + 2 * I + H) * sizeof(float)));
        }
        if (wants_f16_copies(c)) {
            p.l_wo16.push_back(p.take(H * qd * 2));
            p.l_wgu16.push_back(p.take(2 * I * H * 2));
            p.l_wd16.push_back(p.take(H * I * 2));
        }
    }
    p.lm_q8 = p.take(c.weight_format == 1 ? V * H : 0);
    p.lm_s8 = p.take(c.weight_format == 1 ? V * sizeof(float) : 0);
    // fp16 image of ONE layer's K/V rows, rebuilt per layer by the prompt phase (its attention runs in fp16)
    p.k16 = p.take(wants_f16_copies(c) ? B * kd * c.max_seq * 2 : 0);
    p.v16 = p.take(wants_f16_copies(c) ? B * kd * c.max_seq * 2 : 0);
    p.f16_scales = p.take((size_t)c.n_layers * 3 * 2 * sizeof(float));
    p.f16_word = p.take(4);
    p.embed = p.take(V * H * 2);
    p.lm_head = c.tie_embeddings ? p.embed : p.take(V * H * 2);
    p.g_final = p.take(H * 2);
    const size_t kv = (size_t)c.n_layers * B * kd * c.max_seq * 2;
    p.kcache = p.take(kv);
    p.vcache = p.take(kv);
    p.rope = p.take((size_t)c.max_seq * 128 * 4);
    p.gemv_ctr = p.take(((size_t)c.n_layers * 4 + 2) * 16);
    p.gemm_part = p.take(c.max_tokens > 0 ? kGemmPartBytes : 0);
    p.gemm_tickets = p.take((size_t)kGemmTickets * 4);
    p.x = p.take(H * 4);
    p.qkv = p.take(qkvd * 4);
    p.attn_out = p.take(qd * 4);
    p.act = p.take(I * 4);
    p.part = p.take(attn_decode_scratch_floats((int)B, c.n_q_heads, kAttnMaxSplits) * 4);
    p.tickets = p.take(B * c.n_kv_heads * 4);
    p.am_val = p.take(kArgmaxMaxBlocks * 4);
    p.am_idx = p.take(kArgmaxMaxBlocks * 4);
    p.am_ticket = p.take(4);
    p.d_len = p.take(4);
    p.d_status = p.take(4);
    p.d_tokens = p.take(R * 4);
    p.d_argmax = p.take(B * 4);
    p.xt = p.take(R * H * 4);
    p.hb = p.take(R * H * 2);
    p.hb_lo = p.take(R * H * 2);
    p.qkvt = p.take(R * qkvd * 4);
    p.ob = p.take(R * qd * 2);
    p.ob_lo = p.take(R * qd * 2);
    p.ab = p.take(R * I * 2);
    p.ab_lo = p.take(R * I * 2);
    p.logits_stage = p.take((size_t)kHostLogitRows * V * 4);
}

}  // namespace

struct nnc_model {
    nnc_config c;
    cudaStream_t stream;
    cudaStream_t capture_stream;  // graphs are captured here (the caller's stream may be the legacy stream, which cannot capture)
    int device, sm_count;
    char *ws;
    Plan plan;
    std::vector<LayerW> layers;
    bf16 *embed, *lm_head, *g_final, *kcache, *vcache;
    float *rope, *x, *qkv, *attn_out, *act, *part;
    uint32_t *tickets;
    GemmScratch gemm_scratch;  // split-K partial tiles and tickets of the token-batch GEMMs
    uint32_t *gemv_ctr;  // 4 words per GEMV call site (4 per layer + lm_head): dynamic work counters, zero at rest
    ArgmaxScratch am;
    int32_t *d_len, *d_status, *d_tokens, *d_argmax;
    float *xt, *qkvt, *logits_stage;
    bf16 *hb, *ob, *ab;
    bf16 *hb_lo, *ob_lo, *ab_lo;  // bf16 rounding residuals of the GEMM activations (null in the one-term mode)
    bool f16_copies;              // the layers hold fp16 copies of Wo, Wgate/up, Wdown
    void *k16, *v16;              // fp16 image of one layer's K/V rows (prompt phase with fp16 operands; null otherwise)
    uint8_t *lm_q8;               // weight_format 1: FP8 codes and row scales of the lm_head (null otherwise)
    float *lm_s8;
    int len;
    float *taps;
    bool pdl;
    int64_t launches;
    struct Graph {
        cudaGraphExec_t exec;
        int64_t nodes;
    };
    std::map<std::tuple<const void *, const void *, const void *, int>, Graph> graphs;
    char err[512];

    size_t kv_layer_stride() const { return (size_t)c.max_batch * c.n_kv_heads * c.max_seq * 128; }
    size_t kv_seq_stride() const { return (size_t)c.n_kv_heads * c.max_seq * 128; }
    int qd() const { return c.n_q_heads * 128; }
    int kd() const { return c.n_kv_heads * 128; }
    int qkvd() const { return qd() + 2 * kd(); }
};

namespace {

int fail(nnc_model *m, int code, const char *fmt, ...) {
    if (m) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(m->err, sizeof(m->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

#define NNC_CUDA(m, expr)                                                                                  \
    do {                                                                                                   \
        cudaError_t e__ = (expr);                                                                          \
        if (e__ != cudaSuccess)                                                                            \
            return fail(m, NNC_ERR_CUDA, "%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), __FILE__, __LINE__); \
    } while (0)

LaunchCtx ctx(nnc_model *m, bool pdl) { return LaunchCtx{m->stream, m->sm_count, pdl, &m->launches, m->d_status}; }

// One decoder layer for a single token (batch 1) on the residual stream m->x.
int layer_decode_b1(nnc_model *m, int l, const LaunchCtx &lc, int n_splits) {
    const nnc_config &c = m->c;
    const LayerW &w = m->layers[l];
    bf16 *kc = m->kcache + (size_t)l * m->kv_layer_stride();
    bf16 *vc = m->vcache + (size_t)l * m->kv_layer_stride();
    uint32_t *ctr = m->gemv_ctr + (size_t)l * 16;
    const bool q8 = c.weight_format == 1;
    NNC_CUDA(m, launch_gemv(lc, q8 ? (const void *)w.q_qkv : w.wqkv, w.s_qkv, m->x, m->qkv, m->qkvd(), c.hidden, w.g_in, c.rms_eps, kGemvStore, nullptr, ctr));
    const AttnFused fused{w.g_q, w.g_k, m->rope, c.rms_eps};
    NNC_CUDA(m, launch_attn_decode(lc, m->qkv, m->qkvd(), kc, vc, m->attn_out, nullptr, nullptr, m->qd(), m->part, m->tickets,
                                   m->d_len, 1, 1, c.n_q_heads, c.n_kv_heads, c.max_seq, n_splits, &fused));
    NNC_CUDA(m, launch_gemv(lc, q8 ? (const void *)w.q_o : w.wo, w.s_o, m->attn_out, m->x, c.hidden, m->qd(), nullptr, 0.f, kGemvResidual, nullptr, ctr + 4));
    NNC_CUDA(m, launch_gemv(lc, q8 ? (const void *)w.q_gu : w.wgu, w.s_gu, m->x, m->act, 2 * c.intermediate, c.hidden, w.g_post, c.rms_eps, kGemvSwiglu, nullptr, ctr + 8));
    NNC_CUDA(m, launch_gemv(lc, q8 ? (const void *)w.q_d : w.wd, w.s_d, m->act, m->x, c.hidden, c.intermediate, nullptr, 0.f, kGemvResidual, nullptr, ctr + 12));
    return NNC_OK;
}

int decode_b1_launches(nnc_model *m, const int32_t *tokens, float *logits, int32_t *argmax, const LaunchCtx &lc) {
    const nnc_config &c = m->c;
    const int n_splits = attn_decode_splits(m->sm_count, 1, c.n_kv_heads, c.max_seq);
    NNC_CUDA(m, launch_embed(lc, m->embed, tokens, m->x, 1, c.hidden, c.vocab, m->taps));
    for (int l = 0; l < c.n_layers; ++l) {
        int rc = layer_decode_b1(m, l, lc, n_splits);
        if (rc) return rc;
        if (m->taps) NNC_CUDA(m, launch_copy_f32(lc, m->x, m->taps + (size_t)(l + 1) * c.hidden, c.hidden));
    }
    ArgmaxScratch am = m->am;
    am.out = argmax;
    NNC_CUDA(m, launch_gemv(lc, m->lm_q8 ? (const void *)m->lm_q8 : m->lm_head, m->lm_s8, m->x, logits, c.vocab, c.hidden, m->g_final, c.rms_eps, kGemvLogits, &am,
                            m->gemv_ctr + (size_t)c.n_layers * 16));
    NNC_CUDA(m, launch_add_len(lc, m->d_len, 1));
    return NNC_OK;
}

// Token-batch path: rows = batch * T tokens; T == 1 with decode attention is a batched decode step.
int forward_tokens(nnc_model *m, const int32_t *tokens, int batch, int T, float *logits, int all_positions, const LaunchCtx &lc) {
    const nnc_config &c = m->c;
    const int R = batch * T, H = c.hidden, I = c.intermediate, qd = m->qd(), qkvd = m->qkvd();
    NNC_CUDA(m, launch_embed(lc, m->embed, tokens, m->xt, R, H, c.vocab, m->taps));
    const int n_splits = attn_decode_splits(m->sm_count, batch, c.n_kv_heads, c.max_seq);
    // prompt-phase calls of more than 128 tokens: attention output, MLP input and SwiGLU output travel as one fp16 term
    // and meet the fp16 weight copies; the QKV input keeps two bf16 terms (see nnc_config::tc_operands)
    const bool f16 = m->f16_copies && T > 1 && R > 128;
    for (int l = 0; l < c.n_layers; ++l) {
        const LayerW &w = m->layers[l];
        bf16 *kc = m->kcache + (size_t)l * m->kv_layer_stride();
        bf16 *vc = m->vcache + (size_t)l * m->kv_layer_stride();
        NNC_CUDA(m, launch_rmsnorm_rows(lc, m->xt, w.g_in, m->hb, m->hb_lo, R, H, c.rms_eps, 0, 1));
        NNC_CUDA(m, launch_gemm(lc, m->hb, m->hb_lo, w.wqkv, m->qkvt, nullptr, R, qkvd, H, qkvd, kEpiStoreF32, m->d_status, &m->gemm_scratch));
        if (T == 1) {
            const AttnFused fused{w.g_q, w.g_k, m->rope, c.rms_eps};
            NNC_CUDA(m, launch_attn_decode(lc, m->qkvt, qkvd, kc, vc, nullptr, m->ob, m->ob_lo, qd, m->part, m->tickets, m->d_len, 1,
                                           batch, c.n_q_heads, c.n_kv_heads, c.max_seq, n_splits, &fused));
        } else {
            // K/V heads: norm, rotation, append; the query heads are normalised and rotated by the attention kernel
            // With fp16 operands the attention reads an fp16 image of this layer's K/V rows: the new rows are written
            // there by the append kernel, rows of earlier calls are converted first.
            if (f16 && m->len > 0) {
                NNC_CUDA(m, launch_kv_rows_to_f16(lc, kc, m->k16, batch * c.n_kv_heads, c.max_seq, m->len));
                NNC_CUDA(m, launch_kv_rows_to_f16(lc, vc, m->v16, batch * c.n_kv_heads, c.max_seq, m->len));
            }
            NNC_CUDA(m, launch_qk_norm_rope_append(lc, m->qkvt, R, T, w.g_q, w.g_k, c.rms_eps, m->rope, kc, vc, c.n_q_heads,
                                                   c.n_kv_heads, c.max_seq, m->d_len, true, f16 ? m->k16 : nullptr, f16 ? m->v16 : nullptr));
            const AttnFused fused{w.g_q, w.g_k, m->rope, c.rms_eps};
            NNC_CUDA(m, launch_attn_prefill(lc, m->qkvt, R, T, f16 ? (const void *)m->k16 : kc, f16 ? (const void *)m->v16 : vc, f16, m->ob,
                                            f16 ? nullptr : m->ob_lo, f16, c.n_q_heads, c.n_kv_heads, c.max_seq, m->len, &fused));
        }
        if (f16) {
            NNC_CUDA(m, launch_gemm(lc, m->ob, nullptr, (const bf16 *)w.wo16, m->xt, nullptr, R, H, qd, H, kEpiAccumF32, m->d_status, nullptr, true, w.sc_o + 1));
            NNC_CUDA(m, launch_rmsnorm_rows(lc, m->xt, w.g_post, m->hb, nullptr, R, H, c.rms_eps, 0, 1, true));
            NNC_CUDA(m, launch_gemm(lc, m->hb, nullptr, (const bf16 *)w.wgu16, m->ab, nullptr, R, 2 * I, H, I, kEpiSwigluBf16, m->d_status, nullptr, true, w.sc_gu + 1));
            NNC_CUDA(m, launch_gemm(lc, m->ab, nullptr, (const bf16 *)w.wd16, m->xt, nullptr, R, H, I, H, kEpiAccumF32, m->d_status, nullptr, true, w.sc_d + 1));
        } else {
            NNC_CUDA(m, launch_gemm(lc, m->ob, m->ob_lo, w.wo, m->xt, nullptr, R, H, qd, H, kEpiAccumF32, m->d_status, &m->gemm_scratch));
            NNC_CUDA(m, launch_rmsnorm_rows(lc, m->xt, w.g_post, m->hb, m->hb_lo, R, H, c.rms_eps, 0, 1));
            NNC_CUDA(m, launch_gemm(lc, m->hb, m->hb_lo, w.wgu, m->ab, m->ab_lo, R, 2 * I, H, I, kEpiSwigluBf16, m->d_status, &m->gemm_scratch));
            NNC_CUDA(m, launch_gemm(lc, m->ab, m->ab_lo, w.wd, m->xt, nullptr, R, H, I, H, kEpiAccumF32, m->d_status, &m->gemm_scratch));
        }
        if (m->taps) NNC_CUDA(m, launch_copy_f32(lc, m->xt, m->taps + (size_t)(l + 1) * R * H, (size_t)R * H));
    }
    if (logits) {
        if (all_positions || T == 1) {
            NNC_CUDA(m, launch_rmsnorm_rows(lc, m->xt, m->g_final, m->hb, m->hb_lo, R, H, c.rms_eps, 0, 1));
            NNC_CUDA(m, launch_gemm(lc, m->hb, m->hb_lo, m->lm_head, logits, nullptr, R, c.vocab, H, c.vocab, kEpiStoreF32, m->d_status, &m->gemm_scratch));
        } else if (batch == 1) {
            // last position only: the streaming GEMV keeps the activation in fp32
            NNC_CUDA(m, launch_gemv(lc, m->lm_q8 ? (const void *)m->lm_q8 : m->lm_head, m->lm_s8, m->xt + (size_t)(T - 1) * H, logits, c.vocab, H, m->g_final, c.rms_eps,
                                    kGemvLogits, nullptr));
        } else {
            NNC_CUDA(m, launch_rmsnorm_rows(lc, m->xt, m->g_final, m->hb, m->hb_lo, batch, H, c.rms_eps, T - 1, T));
            NNC_CUDA(m, launch_gemm(lc, m->hb, m->hb_lo, m->lm_head, logits, nullptr, batch, c.vocab, H, c.vocab, kEpiStoreF32, m->d_status, &m->gemm_scratch));
        }
    }
    NNC_CUDA(m, launch_add_len(lc, m->d_len, T));
    return NNC_OK;
}

int check_step(nnc_model *m, int batch, int n_tokens) {
    if (batch < 1 || n_tokens < 1) return fail(m, NNC_ERR_INVALID_ARG, "batch and n_tokens must be positive");
    if (batch > m->c.max_batch) return fail(m, NNC_ERR_CAPACITY, "batch %d exceeds max_batch %d", batch, m->c.max_batch);
    if ((long)batch * n_tokens > m->c.max_tokens)
        return fail(m, NNC_ERR_CAPACITY, "%d tokens exceed max_tokens %d", batch * n_tokens, m->c.max_tokens);
    if (m->len + n_tokens > m->c.max_seq)
        return fail(m, NNC_ERR_CAPACITY, "cache length %d + %d new tokens exceeds max_seq %d", m->len, n_tokens, m->c.max_seq);
    return NNC_OK;
}

}  // namespace

extern "C" {

size_t nnc_workspace_bytes(const nnc_config *config) {
    if (!config || !valid_config(*config)) return 0;
    Plan p;
    make_plan(*config, p);
    return p.total;
}

int nnc_model_create(const nnc_config *config, const nnc_weights *weights, void *workspace, size_t workspace_bytes,
                     void *cuda_stream, nnc_model **out) {
    if (!config || !weights || !workspace || !out) return NNC_ERR_INVALID_ARG;
    if (!valid_config(*config)) return NNC_ERR_INVALID_ARG;
    if (!weights->embed || !weights->g_final || !weights->layers) return NNC_ERR_INVALID_ARG;
    if (!config->tie_embeddings && !weights->lm_head) return NNC_ERR_INVALID_ARG;
    for (int l = 0; l < config->n_layers; ++l) {
        const nnc_layer_weights &w = weights->layers[l];
        if (!w.wq || !w.wk || !w.wv || !w.wo || !w.w_gate || !w.w_up || !w.w_down || !w.g_in || !w.g_post || !w.g_q || !w.g_k)
            return NNC_ERR_INVALID_ARG;
    }
    nnc_model *m = new nnc_model();
    m->capture_stream = nullptr;
    m->c = *config;
    m->err[0] = 0;
    make_plan(m->c, m->plan);
    if (workspace_bytes < m->plan.total || ((uintptr_t)workspace % kAlign)) {
        delete m;
        return NNC_ERR_WORKSPACE;
    }
    int rc = NNC_OK;
    auto body = [&]() -> int {
        NNC_CUDA(m, cudaGetDevice(&m->device));
        NNC_CUDA(m, cudaDeviceGetAttribute(&m->sm_count, cudaDevAttrMultiProcessorCount, m->device));
        int major = 0;
        NNC_CUDA(m, cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, m->device));
        if (major != 10) return fail(m, NNC_ERR_CUDA, "this library is built for sm_100a only (device is sm_%d*)", major);
        m->stream = (cudaStream_t)cuda_stream;
        NNC_CUDA(m, cudaStreamCreateWithFlags(&m->capture_stream, cudaStreamNonBlocking));
        m->ws = (char *)workspace;
        const Plan &p = m->plan;
        const nnc_config &c = m->c;
        auto at = [&](size_t off) { return m->ws + off; };
        m->layers.resize(c.n_layers);
        for (int l = 0; l < c.n_layers; ++l) {
            LayerW &w = m->layers[l];
            w.wqkv = (bf16 *)at(p.l_wqkv[l]); w.wo = (bf16 *)at(p.l_wo[l]); w.wgu = (bf16 *)at(p.l_wgu[l]);
            w.wd = (bf16 *)at(p.l_wd[l]); w.g_in = (bf16 *)at(p.l_gin[l]); w.g_post = (bf16 *)at(p.l_gpost[l]);
            w.g_q = (bf16 *)at(p.l_gq[l]); w.g_k = (bf16 *)at(p.l_gk[l]);
            w.wo16 = w.wgu16 = w.wd16 = nullptr;
            w.sc_o = (float *)at(p.f16_scales) + (size_t)l * 6;
            w.sc_gu = w.sc_o + 2; w.sc_d = w.sc_o + 4;
            if (wants_f16_copies(c)) { w.wo16 = at(p.l_wo16[l]); w.wgu16 = at(p.l_wgu16[l]); w.wd16 = at(p.l_wd16[l]); }
            w.q_qkv = w.q_o = w.q_gu = w.q_d = nullptr;
            w.s_qkv = w.s_o = w.s_gu = w.s_d = nullptr;
            if (c.weight_format == 1) {
                const size_t qkvd = (size_t)m->qkvd(), Hs = c.hidden, qds = m->qd(), Is = c.intermediate;
                w.q_qkv = (uint8_t *)at(p.l_q8[l]); w.q_o = w.q_qkv + qkvd * Hs; w.q_gu = w.q_o + Hs * qds; w.q_d = w.q_gu + 2 * Is * Hs;
                w.s_qkv = (float *)at(p.l_s8[l]); w.s_o = w.s_qkv + qkvd; w.s_gu = w.s_o + Hs; w.s_d = w.s_gu + 2 * Is;
            }
        }
        m->k16 = wants_f16_copies(c) ? at(p.k16) : nullptr;
        m->v16 = wants_f16_copies(c) ? at(p.v16) : nullptr;
        m->lm_q8 = c.weight_format == 1 ? (uint8_t *)at(p.lm_q8) : nullptr;
        m->lm_s8 = c.weight_format == 1 ? (float *)at(p.lm_s8) : nullptr;
        m->embed = (bf16 *)at(p.embed); m->lm_head = (bf16 *)at(p.lm_head); m->g_final = (bf16 *)at(p.g_final);
        m->kcache = (bf16 *)at(p.kcache); m->vcache = (bf16 *)at(p.vcache); m->rope = (float *)at(p.rope);
        m->x = (float *)at(p.x); m->qkv = (float *)at(p.qkv); m->attn_out = (float *)at(p.attn_out);
        m->act = (float *)at(p.act); m->part = (float *)at(p.part); m->tickets = (uint32_t *)at(p.tickets);
        m->gemv_ctr = (uint32_t *)at(p.gemv_ctr);
        m->gemm_scratch = GemmScratch{(float *)at(p.gemm_part), kGemmPartBytes, (uint32_t *)at(p.gemm_tickets), kGemmTickets};
        m->am = ArgmaxScratch{(float *)at(p.am_val), (int32_t *)at(p.am_idx), (uint32_t *)at(p.am_ticket), nullptr};
        m->d_len = (int32_t *)at(p.d_len); m->d_status = (int32_t *)at(p.d_status);
        m->d_tokens = (int32_t *)at(p.d_tokens); m->d_argmax = (int32_t *)at(p.d_argmax);
        m->xt = (float *)at(p.xt); m->hb = (bf16 *)at(p.hb); m->qkvt = (float *)at(p.qkvt);
        m->ob = (bf16 *)at(p.ob); m->ab = (bf16 *)at(p.ab); m->logits_stage = (float *)at(p.logits_stage);
        const bool fast = c.tc_operands == 2;
        m->f16_copies = wants_f16_copies(c);
        m->hb_lo = fast ? nullptr : (bf16 *)at(p.hb_lo);
        m->ob_lo = fast ? nullptr : (bf16 *)at(p.ob_lo);
        m->ab_lo = fast ? nullptr : (bf16 *)at(p.ab_lo);
        m->len = 0;
        m->taps = nullptr;
        m->launches = 0;
        m->pdl = c.serial_launches == 0;

        // ---- repack: bit moves on the device ----
        LaunchCtx lc = ctx(m, false);
        const int H = c.hidden, qd = m->qd(), kd = m->kd(), I = c.intermediate;
        for (int l = 0; l < c.n_layers; ++l) {
            const nnc_layer_weights &s = weights->layers[l];
            LayerW &w = m->layers[l];
            NNC_CUDA(m, launch_copy_rows(lc, (const bf16 *)s.wq, w.wqkv, qd, H, 0, 1, 0, 1));
            NNC_CUDA(m, launch_copy_rows(lc, (const bf16 *)s.wk, w.wqkv, kd, H, qd, 1, 0, 1));
            NNC_CUDA(m, launch_copy_rows(lc, (const bf16 *)s.wv, w.wqkv, kd, H, qd + kd, 1, 0, 1));
            NNC_CUDA(m, launch_copy_rows(lc, (const bf16 *)s.wo, w.wo, H, qd, 0, 1, 0, 1));
            NNC_CUDA(m, launch_copy_rows(lc, (const bf16 *)s.w_gate, w.wgu, I, H, 0, 2, 0, 1));
            NNC_CUDA(m, launch_copy_rows(lc, (const bf16 *)s.w_up, w.wgu, I, H, 1, 2, 0, 1));
            NNC_CUDA(m, launch_copy_rows(lc, (const bf16 *)s.w_down, w.wd, H, I, 0, 1, 0, 1));
            NNC_CUDA(m, cudaMemcpyAsync(w.g_in, s.g_in, (size_t)H * 2, cudaMemcpyDeviceToDevice, m->stream));
            NNC_CUDA(m, cudaMemcpyAsync(w.g_post, s.g_post, (size_t)H * 2, cudaMemcpyDeviceToDevice, m->stream));
            NNC_CUDA(m, cudaMemcpyAsync(w.g_q, s.g_q, 256, cudaMemcpyDeviceToDevice, m->stream));
            NNC_CUDA(m, cudaMemcpyAsync(w.g_k, s.g_k, 256, cudaMemcpyDeviceToDevice, m->stream));
            if (c.weight_format == 1) {   // quantise; the bf16 store keeps the dequantised values
                NNC_CUDA(m, launch_quantise_rows_e4m3(lc, w.wqkv, w.q_qkv, w.s_qkv, w.wqkv, m->qkvd(), H));
                NNC_CUDA(m, launch_quantise_rows_e4m3(lc, w.wo, w.q_o, w.s_o, w.wo, H, qd));
                NNC_CUDA(m, launch_quantise_rows_e4m3(lc, w.wgu, w.q_gu, w.s_gu, w.wgu, 2 * I, H));
                NNC_CUDA(m, launch_quantise_rows_e4m3(lc, w.wd, w.q_d, w.s_d, w.wd, H, I));
            }
            if (m->f16_copies) {
                uint32_t *word = (uint32_t *)at(p.f16_word);
                NNC_CUDA(m, launch_to_f16_scaled(lc, w.wo, w.wo16, (size_t)H * qd, w.sc_o, word));
                NNC_CUDA(m, launch_to_f16_scaled(lc, w.wgu, w.wgu16, (size_t)2 * I * H, w.sc_gu, word));
                NNC_CUDA(m, launch_to_f16_scaled(lc, w.wd, w.wd16, (size_t)H * I, w.sc_d, word));
            }
        }
        NNC_CUDA(m, launch_copy_rows(lc, (const bf16 *)weights->embed, m->embed, c.vocab, H, 0, 1, 0, 1));
        if (!c.tie_embeddings)
            NNC_CUDA(m, launch_copy_rows(lc, (const bf16 *)weights->lm_head, m->lm_head, c.vocab, H, 0, 1, 0, 1));
        NNC_CUDA(m, cudaMemcpyAsync(m->g_final, weights->g_final, (size_t)H * 2, cudaMemcpyDeviceToDevice, m->stream));
        if (c.weight_format == 1)   // a tied embedding is this same matrix: the gather then reads the dequantised rows
            NNC_CUDA(m, launch_quantise_rows_e4m3(lc, m->lm_head, m->lm_q8, m->lm_s8, m->lm_head, c.vocab, H));

        // ---- RoPE table: cos/sin of p * theta^(-2i/128) in double, rounded once to fp32 ----
        {
            std::vector<float> tab((size_t)c.max_seq * 128);
            std::vector<double> inv_freq(64);
            for (int i = 0; i < 64; ++i) inv_freq[i] = pow((double)c.rope_theta, -2.0 * i / 128.0);
            for (int pos = 0; pos < c.max_seq; ++pos)
                for (int i = 0; i < 64; ++i) {
                    const double phi = (double)pos * inv_freq[i];
                    tab[((size_t)pos * 64 + i) * 2] = (float)cos(phi);
                    tab[((size_t)pos * 64 + i) * 2 + 1] = (float)sin(phi);
                }
            NNC_CUDA(m, cudaMemcpyAsync(m->rope, tab.data(), tab.size() * 4, cudaMemcpyHostToDevice, m->stream));
            NNC_CUDA(m, cudaStreamSynchronize(m->stream));
        }
        NNC_CUDA(m, cudaMemsetAsync(m->tickets, 0, (size_t)c.max_batch * c.n_kv_heads * 4, m->stream));
        NNC_CUDA(m, cudaMemsetAsync(m->am.ticket, 0, 4, m->stream));
        NNC_CUDA(m, cudaMemsetAsync(m->gemm_scratch.tickets, 0, (size_t)kGemmTickets * 4, m->stream));
        NNC_CUDA(m, cudaMemsetAsync(m->gemv_ctr, 0, ((size_t)c.n_layers * 4 + 2) * 16, m->stream));
        NNC_CUDA(m, cudaMemsetAsync(m->d_len, 0, 4, m->stream));
        NNC_CUDA(m, cudaMemsetAsync(m->d_status, 0, 4, m->stream));
        NNC_CUDA(m, cudaStreamSynchronize(m->stream));
        return NNC_OK;
    };
    rc = body();
    if (rc != NNC_OK) {
        fprintf(stderr, "nnc_model_create: %s\n", m->err);
        if (m->capture_stream) cudaStreamDestroy(m->capture_stream);
        delete m;
        return rc;
    }
    *out = m;
    return NNC_OK;
}

void nnc_model_destroy(nnc_model *m) {
    if (!m) return;
    cudaStreamSynchronize(m->stream);
    for (auto &g : m->graphs) cudaGraphExecDestroy(g.second.exec);
    if (m->capture_stream) cudaStreamDestroy(m->capture_stream);
    delete m;
}

int nnc_prefill(nnc_model *m, const int32_t *tokens, int32_t batch, int32_t n_tokens, float *logits,
                int32_t all_positions) {
    if (!m || !tokens) return fail(m, NNC_ERR_INVALID_ARG, "null argument");
    int rc = check_step(m, batch, n_tokens);
    if (rc) return rc;
    rc = forward_tokens(m, tokens, batch, n_tokens, logits, all_positions, ctx(m, m->pdl));
    if (rc == NNC_OK) m->len += n_tokens;
    return rc;
}

int nnc_decode_step(nnc_model *m, const int32_t *tokens, int32_t batch, float *logits, int32_t *argmax) {
    if (!m || !tokens || !logits) return fail(m, NNC_ERR_INVALID_ARG, "null argument");
    int rc = check_step(m, batch, 1);
    if (rc) return rc;
    if (batch > 1 && argmax) return fail(m, NNC_ERR_INVALID_ARG, "argmax output is only available at batch 1");
    if (m->taps) {  // instrumented: kernel by kernel
        rc = batch > 1 ? forward_tokens(m, tokens, batch, 1, logits, 0, ctx(m, false))
                       : decode_b1_launches(m, tokens, logits, argmax, ctx(m, false));
        if (rc == NNC_OK) m->len += 1;
        return rc;
    }
    // one graph per (buffers, batch): the position is read from device memory, so a graph serves every step
    auto key = std::make_tuple((const void *)tokens, (const void *)logits, (const void *)argmax, (int)batch);
    auto it = m->graphs.find(key);
    if (it == m->graphs.end()) {
        // capture the step once for this set of buffers
        cudaGraphExec_t exec = nullptr;
        cudaGraph_t graph = nullptr;
        const int64_t before = m->launches;
        NNC_CUDA(m, cudaStreamBeginCapture(m->capture_stream, cudaStreamCaptureModeThreadLocal));
        LaunchCtx cap = ctx(m, m->pdl);
        cap.stream = m->capture_stream;
        rc = batch > 1 ? forward_tokens(m, tokens, batch, 1, logits, 0, cap) : decode_b1_launches(m, tokens, logits, argmax, cap);
        cudaError_t e = cudaStreamEndCapture(m->capture_stream, &graph);
        const int64_t nodes = m->launches - before;
        m->launches = before;
        if (rc == NNC_OK && e == cudaSuccess) e = cudaGraphInstantiate(&exec, graph, 0);
        if (graph) cudaGraphDestroy(graph);
        if (rc != NNC_OK || e != cudaSuccess) {
            cudaGetLastError();
            if (rc != NNC_OK) return rc;
            return fail(m, NNC_ERR_CUDA, "graph capture / instantiate failed: %s", cudaGetErrorString(e));
        }
        if (m->graphs.size() >= 16) {  // callers that keep changing buffers should not leak graphs
            for (auto &g : m->graphs) cudaGraphExecDestroy(g.second.exec);
            m->graphs.clear();
        }
        it = m->graphs.emplace(key, nnc_model::Graph{exec, nodes}).first;
    }
    NNC_CUDA(m, cudaGraphLaunch(it->second.exec, m->stream));
    m->launches += it->second.nodes;
    m->len += 1;
    return NNC_OK;
}

int nnc_decode_step_host(nnc_model *m, const int32_t *tokens_host, int32_t batch, float *logits_host,
                         int32_t *argmax_host) {
    if (!m || !tokens_host) return fail(m, NNC_ERR_INVALID_ARG, "null argument");
    int rc = check_step(m, batch, 1);
    if (rc) return rc;
    if (batch > kHostLogitRows) return fail(m, NNC_ERR_CAPACITY, "host variant stages at most %d rows of logits", kHostLogitRows);
    NNC_CUDA(m, cudaMemcpyAsync(m->d_tokens, tokens_host, (size_t)batch * 4, cudaMemcpyHostToDevice, m->stream));
    rc = nnc_decode_step(m, m->d_tokens, batch, m->logits_stage, (argmax_host && batch == 1) ? m->d_argmax : nullptr);
    if (rc) return rc;
    if (logits_host)
        NNC_CUDA(m, cudaMemcpyAsync(logits_host, m->logits_stage, (size_t)batch * m->c.vocab * 4, cudaMemcpyDeviceToHost, m->stream));
    if (argmax_host) {
        if (batch != 1) return fail(m, NNC_ERR_INVALID_ARG, "argmax output is only available at batch 1");
        NNC_CUDA(m, cudaMemcpyAsync(argmax_host, m->d_argmax, 4, cudaMemcpyDeviceToHost, m->stream));
    }
    NNC_CUDA(m, cudaStreamSynchronize(m->stream));
    return NNC_OK;
}

int nnc_prefill_host(nnc_model *m, const int32_t *tokens_host, int32_t batch, int32_t n_tokens, float *logits_host,
                     int32_t all_positions) {
    if (!m || !tokens_host) return fail(m, NNC_ERR_INVALID_ARG, "null argument");
    int rc = check_step(m, batch, n_tokens);
    if (rc) return rc;
    const long rows = all_positions ? (long)batch * n_tokens : batch;
    if (logits_host && rows > kHostLogitRows)
        return fail(m, NNC_ERR_CAPACITY, "host variant stages at most %d rows of logits", kHostLogitRows);
    NNC_CUDA(m, cudaMemcpyAsync(m->d_tokens, tokens_host, (size_t)batch * n_tokens * 4, cudaMemcpyHostToDevice, m->stream));
    rc = nnc_prefill(m, m->d_tokens, batch, n_tokens, logits_host ? m->logits_stage : nullptr, all_positions);
    if (rc) return rc;
    if (logits_host)
        NNC_CUDA(m, cudaMemcpyAsync(logits_host, m->logits_stage, (size_t)rows * m->c.vocab * 4, cudaMemcpyDeviceToHost, m->stream));
    NNC_CUDA(m, cudaStreamSynchronize(m->stream));
    return NNC_OK;
}

static int kv_copy(nnc_model *m, int layer, int b, void *k, void *v, int n_pos, bool import) {
    if (!m || !k || !v) return fail(m, NNC_ERR_INVALID_ARG, "null argument");
    if (layer < 0 || layer >= m->c.n_layers || b < 0 || b >= m->c.max_batch || n_pos < 0)
        return fail(m, NNC_ERR_INVALID_ARG, "layer / batch index out of range");
    if (n_pos > m->c.max_seq) return fail(m, NNC_ERR_CAPACITY, "n_pos %d exceeds max_seq %d", n_pos, m->c.max_seq);
    if (n_pos == 0) return NNC_OK;
    const size_t off = (size_t)layer * m->kv_layer_stride() + (size_t)b * m->kv_seq_stride();
    const size_t row = (size_t)n_pos * 128 * 2, pitch = (size_t)m->c.max_seq * 128 * 2;
    for (int which = 0; which < 2; ++which) {
        char *cache = (char *)((which ? m->vcache : m->kcache) + off);
        char *user = (char *)(which ? v : k);
        if (import)
            NNC_CUDA(m, cudaMemcpy2DAsync(cache, pitch, user, row, row, m->c.n_kv_heads, cudaMemcpyDeviceToDevice, m->stream));
        else
            NNC_CUDA(m, cudaMemcpy2DAsync(user, row, cache, pitch, row, m->c.n_kv_heads, cudaMemcpyDeviceToDevice, m->stream));
    }
    return NNC_OK;
}

int nnc_kv_import(nnc_model *m, int32_t layer, int32_t b, const void *k, const void *v, int32_t n_pos) {
    return kv_copy(m, layer, b, const_cast<void *>(k), const_cast<void *>(v), n_pos, true);
}
int nnc_kv_export(nnc_model *m, int32_t layer, int32_t b, void *k, void *v, int32_t n_pos) {
    return kv_copy(m, layer, b, k, v, n_pos, false);
}

int nnc_set_length(nnc_model *m, int32_t n_pos) {
    if (!m) return NNC_ERR_INVALID_ARG;
    if (n_pos < 0 || n_pos > m->c.max_seq) return fail(m, NNC_ERR_CAPACITY, "length %d outside [0, %d]", n_pos, m->c.max_seq);
    // a 4-byte async copy from the stack is unsafe, a memset cannot set an arbitrary int: add the difference
    LaunchCtx lc = ctx(m, false);
    NNC_CUDA(m, launch_add_len(lc, m->d_len, n_pos - m->len));
    m->len = n_pos;
    return NNC_OK;
}

int32_t nnc_get_length(const nnc_model *m) { return m ? m->len : -1; }

int nnc_set_hidden_tap(nnc_model *m, float *taps) {
    if (!m) return NNC_ERR_INVALID_ARG;
    m->taps = taps;
    return NNC_OK;
}

int nnc_layer_decode(nnc_model *m, int32_t layer, const float *x_in, float *x_out) {
    if (!m || !x_in || !x_out) return fail(m, NNC_ERR_INVALID_ARG, "null argument");
    if (layer < 0 || layer >= m->c.n_layers) return fail(m, NNC_ERR_INVALID_ARG, "layer out of range");
    if (m->len + 1 > m->c.max_seq) return fail(m, NNC_ERR_CAPACITY, "cache full");
    LaunchCtx lc = ctx(m, false);
    NNC_CUDA(m, cudaMemcpyAsync(m->x, x_in, (size_t)m->c.hidden * 4, cudaMemcpyDeviceToDevice, m->stream));
    const int n_splits = attn_decode_splits(m->sm_count, 1, m->c.n_kv_heads, m->c.max_seq);
    int rc = layer_decode_b1(m, layer, lc, n_splits);
    if (rc) return rc;
    NNC_CUDA(m, cudaMemcpyAsync(x_out, m->x, (size_t)m->c.hidden * 4, cudaMemcpyDeviceToDevice, m->stream));
    return NNC_OK;
}

int nnc_unrepack(nnc_model *m, int32_t layer, int32_t which, void *out) {
    if (!m || !out) return fail(m, NNC_ERR_INVALID_ARG, "null argument");
    if (layer < 0 || layer >= m->c.n_layers) return fail(m, NNC_ERR_INVALID_ARG, "layer out of range");
    LaunchCtx lc = ctx(m, false);
    const LayerW &w = m->layers[layer];
    const int H = m->c.hidden, qd = m->qd(), kd = m->kd(), I = m->c.intermediate;
    bf16 *o = (bf16 *)out;
    switch (which) {
        case 0: NNC_CUDA(m, launch_copy_rows(lc, w.wqkv, o, qd, H, 0, 1, 0, 1)); break;
        case 1: NNC_CUDA(m, launch_copy_rows(lc, w.wqkv, o, kd, H, 0, 1, qd, 1)); break;
        case 2: NNC_CUDA(m, launch_copy_rows(lc, w.wqkv, o, kd, H, 0, 1, qd + kd, 1)); break;
        case 3: NNC_CUDA(m, launch_copy_rows(lc, w.wo, o, H, qd, 0, 1, 0, 1)); break;
        case 4: NNC_CUDA(m, launch_copy_rows(lc, w.wgu, o, I, H, 0, 1, 0, 2)); break;
        case 5: NNC_CUDA(m, launch_copy_rows(lc, w.wgu, o, I, H, 0, 1, 1, 2)); break;
        case 6: NNC_CUDA(m, launch_copy_rows(lc, w.wd, o, H, I, 0, 1, 0, 1)); break;
        default: return fail(m, NNC_ERR_INVALID_ARG, "which must be 0..6");
    }
    return NNC_OK;
}

int nnc_device_status(nnc_model *m, int32_t *status_out) {
    if (!m || !status_out) return NNC_ERR_INVALID_ARG;
    NNC_CUDA(m, cudaMemcpyAsync(status_out, m->d_status, 4, cudaMemcpyDeviceToHost, m->stream));
    NNC_CUDA(m, cudaMemsetAsync(m->d_status, 0, 4, m->stream));
    NNC_CUDA(m, cudaStreamSynchronize(m->stream));
    return *status_out ? NNC_ERR_DEVICE_STATUS : NNC_OK;
}

int64_t nnc_launch_count(const nnc_model *m) { return m ? m->launches : 0; }

const char *nnc_last_error(const nnc_model *m) { return m ? m->err : "no model"; }

const char *nnc_status_string(int status) {
    switch (status) {
        case NNC_OK: return "ok";
        case NNC_ERR_INVALID_ARG: return "invalid argument";
        case NNC_ERR_WORKSPACE: return "workspace too small or misaligned";
        case NNC_ERR_CAPACITY: return "capacity exceeded";
        case NNC_ERR_CUDA: return "CUDA error";
        case NNC_ERR_DEVICE_STATUS: return "a kernel reported a bounded wait that ran out";
    }
    return "unknown status";
}

#ifdef NNC_BOUNDS_CHECK
}  // extern "C"
namespace nnc {
static std::vector<void (*)(unsigned *, unsigned *)> &bc_readers() {
    static std::vector<void (*)(unsigned *, unsigned *)> v;
    return v;
}
void bc_register(void (*read_and_clear)(unsigned *, unsigned *)) { bc_readers().push_back(read_and_clear); }
}  // namespace nnc
extern "C" {
#endif

int nnc_bounds_check_report(int32_t *misses_out, int32_t *first_code_out) {
    if (!misses_out || !first_code_out) return NNC_ERR_INVALID_ARG;
#ifdef NNC_BOUNDS_CHECK
    if (cudaDeviceSynchronize() != cudaSuccess) return NNC_ERR_CUDA;
    unsigned total = 0, first = 0;
    for (auto rd : nnc::bc_readers()) {
        unsigned n = 0, code = 0;
        rd(&n, &code);
        if (n && !first) first = code;
        total += n;
    }
    *misses_out = (int32_t)total;
    *first_code_out = (int32_t)first;
#else
    *misses_out = -1;   // not a checked build
    *first_code_out = 0;
#endif
    return NNC_OK;
}

#ifdef NNC_TRACE
}  // extern "C"
namespace nnc {
static std::vector<void (*)(TraceRec *, unsigned *)> &trace_binders() {
    static std::vector<void (*)(TraceRec *, unsigned *)> v;
    return v;
}
void trace_register(void (*bind)(TraceRec *, unsigned *)) { trace_binders().push_back(bind); }
static TraceRec *g_trace_dev;
static unsigned *g_trace_cnt_dev;
}  // namespace nnc
extern "C" {
// tracing builds only.  enable: allocates the record buffer (cudaMalloc -- tracing builds are not the product)
// and points every translation unit at it.  dump: copies the records out, resets the count, returns it.
int nnc_trace_enable(void) {
    if (!nnc::g_trace_dev) {
        if (cudaMalloc(&nnc::g_trace_dev, sizeof(nnc::TraceRec) * nnc::kTraceMax) != cudaSuccess) return -1;
        if (cudaMalloc(&nnc::g_trace_cnt_dev, 4) != cudaSuccess) return -1;
        cudaMemset(nnc::g_trace_cnt_dev, 0, 4);
    }
    for (auto b : nnc::trace_binders()) b(nnc::g_trace_dev, nnc::g_trace_cnt_dev);
    return (int)nnc::trace_binders().size();
}
int nnc_trace_dump(void *out, int max_records) {
    unsigned n = 0;
    cudaDeviceSynchronize();
    cudaMemcpy(&n, nnc::g_trace_cnt_dev, 4, cudaMemcpyDeviceToHost);
    if (n > nnc::kTraceMax) n = nnc::kTraceMax;
    if ((int)n > max_records) n = max_records;
    if (out && n) cudaMemcpy(out, nnc::g_trace_dev, (size_t)n * sizeof(nnc::TraceRec), cudaMemcpyDeviceToHost);
    cudaMemset(nnc::g_trace_cnt_dev, 0, 4);
    return (int)n;
}
#endif

// ---- single operations ------------------------------------------------------------------------------

static __device__ int g_op_status;
static __device__ uint32_t g_op_gemv_ctr[8][4];   // work counters of the last 8 nnc_op_gemv calls, used in rotation

static int op_ctx(LaunchCtx &lc, void *stream) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return NNC_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return NNC_ERR_CUDA;
    int *status = nullptr;
    if (cudaGetSymbolAddress((void **)&status, g_op_status) != cudaSuccess) return NNC_ERR_CUDA;
    lc = LaunchCtx{(cudaStream_t)stream, sms, false, nullptr, status};
    return NNC_OK;
}

int nnc_bounds_check_selftest(int32_t code, void *cuda_stream) {
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    return launch_bounds_check_selftest(lc, code) == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_gemm(const void *X, const void *X_lo, const void *W, void *Y, int32_t T, int32_t n_out, int32_t n_in,
                int32_t out_f32, int32_t accumulate, void *cuda_stream) {
    if (!X || !W || !Y) return NNC_ERR_INVALID_ARG;
    if (accumulate && !out_f32) return NNC_ERR_INVALID_ARG;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    int *status = nullptr;
    if (cudaGetSymbolAddress((void **)&status, g_op_status) != cudaSuccess) return NNC_ERR_CUDA;
    const int epi = out_f32 ? (accumulate ? kEpiAccumF32 : kEpiStoreF32) : kEpiStoreBf16;
    cudaError_t e = launch_gemm(lc, (const bf16 *)X, (const bf16 *)X_lo, (const bf16 *)W, Y, nullptr, T, n_out, n_in, n_out, epi, status);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_gemm_swiglu(const void *X, const void *X_lo, const void *W, void *Y, void *Y_lo, int32_t T, int32_t n_out,
                       int32_t n_in, void *cuda_stream) {
    if (!X || !W || !Y || n_out % 2) return NNC_ERR_INVALID_ARG;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    int *status = nullptr;
    if (cudaGetSymbolAddress((void **)&status, g_op_status) != cudaSuccess) return NNC_ERR_CUDA;
    cudaError_t e = launch_gemm(lc, (const bf16 *)X, (const bf16 *)X_lo, (const bf16 *)W, Y, Y_lo, T, n_out, n_in, n_out / 2, kEpiSwigluBf16, status);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_gemm_splitk(const void *X, const void *X_lo, const void *W, void *Y, int32_t T, int32_t n_out, int32_t n_in,
                       int32_t out_f32, int32_t accumulate, void *scratch, size_t scratch_bytes, void *cuda_stream) {
    if (!X || !W || !Y || !scratch || ((uintptr_t)scratch & 255)) return NNC_ERR_INVALID_ARG;
    if (accumulate && !out_f32) return NNC_ERR_INVALID_ARG;
    const size_t ticket_bytes = (size_t)kGemmTickets * 4;
    if (scratch_bytes < ticket_bytes + (1u << 20)) return NNC_ERR_WORKSPACE;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    const GemmScratch sc{(float *)((char *)scratch + ticket_bytes), scratch_bytes - ticket_bytes, (uint32_t *)scratch, kGemmTickets};
    const int epi = out_f32 ? (accumulate ? kEpiAccumF32 : kEpiStoreF32) : kEpiStoreBf16;
    cudaError_t e = launch_gemm(lc, (const bf16 *)X, (const bf16 *)X_lo, (const bf16 *)W, Y, nullptr, T, n_out, n_in, n_out, epi,
                                lc.status, &sc);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_gemm_f16(const void *X, const void *W, float *Y, int32_t T, int32_t n_out, int32_t n_in, int32_t accumulate,
                    const float *out_scale, void *cuda_stream) {
    if (!X || !W || !Y) return NNC_ERR_INVALID_ARG;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    cudaError_t e = launch_gemm(lc, (const bf16 *)X, nullptr, (const bf16 *)W, Y, nullptr, T, n_out, n_in, n_out,
                                accumulate ? kEpiAccumF32 : kEpiStoreF32, lc.status, nullptr, true, out_scale);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_gemm_swiglu_f16(const void *X, const void *W, void *Y, int32_t T, int32_t n_out, int32_t n_in,
                           const float *out_scale, void *cuda_stream) {
    if (!X || !W || !Y || n_out % 2) return NNC_ERR_INVALID_ARG;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    cudaError_t e = launch_gemm(lc, (const bf16 *)X, nullptr, (const bf16 *)W, Y, nullptr, T, n_out, n_in, n_out / 2,
                                kEpiSwigluBf16, lc.status, nullptr, true, out_scale);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_to_f16_scaled(const void *src, void *dst, size_t n, float *scales, uint32_t *scratch_word, void *cuda_stream) {
    if (!src || !dst || !scales || !scratch_word || n == 0 || n % 8) return NNC_ERR_INVALID_ARG;
    if (((uintptr_t)src | (uintptr_t)dst) & 15) return NNC_ERR_INVALID_ARG;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    cudaError_t e = launch_to_f16_scaled(lc, (const bf16 *)src, dst, n, scales, scratch_word);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_status(int32_t *status_out) {
    if (!status_out) return NNC_ERR_INVALID_ARG;
    int zero = 0;
    if (cudaMemcpyFromSymbol(status_out, g_op_status, 4) != cudaSuccess) return NNC_ERR_CUDA;
    if (cudaMemcpyToSymbol(g_op_status, &zero, 4) != cudaSuccess) return NNC_ERR_CUDA;
    return *status_out ? NNC_ERR_DEVICE_STATUS : NNC_OK;
}

int nnc_op_gemv(const void *W, const float *x, float *y, int32_t n_out, int32_t n_in, const void *gain, float eps,
                int32_t mode, void *cuda_stream) {
    const bool chained = (mode & NNC_GEMV_CHAINED) != 0;
    mode &= ~NNC_GEMV_CHAINED;
    if (!W || !x || !y || mode < 0 || mode > 2) return NNC_ERR_INVALID_ARG;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    lc.pdl = chained;
    uint32_t *ctrs = nullptr;
    if (cudaGetSymbolAddress((void **)&ctrs, g_op_gemv_ctr) != cudaSuccess) return NNC_ERR_CUDA;
    static unsigned rotation = 0;   // call sites taken in turn; atomic so that concurrent host threads get distinct ones
    const unsigned site = __atomic_fetch_add(&rotation, 1u, __ATOMIC_RELAXED) % 8;
    cudaError_t e = launch_gemv(lc, W, nullptr, x, y, n_out, n_in, (const bf16 *)gain, eps, mode, nullptr, ctrs + 4 * site);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_attn_prefill_f16(const float *qkv, const void *k16, const void *v16, void *out, int32_t batch, int32_t T,
                            int32_t n_q_heads, int32_t n_kv_heads, int32_t max_seq, int32_t n_past, void *cuda_stream) {
    if (!qkv || !k16 || !v16 || !out) return NNC_ERR_INVALID_ARG;
    if (batch <= 0 || T <= 0 || n_kv_heads <= 0 || n_q_heads <= 0 || n_q_heads % n_kv_heads || n_past < 0) return NNC_ERR_INVALID_ARG;
    if ((long)n_past + T > max_seq) return NNC_ERR_CAPACITY;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    cudaError_t e = launch_attn_prefill(lc, qkv, batch * T, T, k16, v16, true, out, nullptr, true, n_q_heads, n_kv_heads, max_seq, n_past);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_gemv_fp8(const void *codes, const float *scales, const float *x, float *y, int32_t n_out, int32_t n_in,
                    const void *gain, float eps, int32_t mode, void *cuda_stream) {
    const bool chained = (mode & NNC_GEMV_CHAINED) != 0;
    mode &= ~NNC_GEMV_CHAINED;
    if (!codes || !scales || !x || !y || mode < 0 || mode > 2) return NNC_ERR_INVALID_ARG;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    lc.pdl = chained;
    cudaError_t e = launch_gemv(lc, codes, scales, x, y, n_out, n_in, (const bf16 *)gain, eps, mode, nullptr, nullptr);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_quantise_rows_e4m3(const void *W, void *codes, float *scales, void *dequant, int32_t n_out, int32_t n_in,
                              void *cuda_stream) {
    if (!W || !codes || !scales) return NNC_ERR_INVALID_ARG;
    if (((uintptr_t)W | (uintptr_t)codes | (uintptr_t)dequant) & 15) return NNC_ERR_INVALID_ARG;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    cudaError_t e = launch_quantise_rows_e4m3(lc, (const bf16 *)W, (uint8_t *)codes, scales, (bf16 *)dequant, n_out, n_in);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

size_t nnc_attn_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t n_ctx) {
    (void)n_ctx;
    if (batch <= 0 || n_q_heads <= 0) return 0;
    // partials for the largest split count, then one ticket word per (sequence, KV head <= query heads)
    return (attn_decode_scratch_floats(batch, n_q_heads, kAttnMaxSplits) * 4 + 255) / 256 * 256 + (size_t)batch * n_q_heads * 4;
}

int nnc_op_attn_decode(const float *q, const void *kcache, const void *vcache, float *out, int32_t batch,
                       int32_t n_q_heads, int32_t n_kv_heads, int32_t max_seq, int32_t n_ctx, void *scratch,
                       void *cuda_stream) {
    if (!q || !kcache || !vcache || !out || !scratch) return NNC_ERR_INVALID_ARG;
    if (batch <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads || n_ctx <= 0 || n_ctx > max_seq) return NNC_ERR_INVALID_ARG;
    const int G = n_q_heads / n_kv_heads;
    if (!(G == 1 || G == 2 || G == 4 || G == 8) || ((uintptr_t)scratch & 255)) return NNC_ERR_INVALID_ARG;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    const int n_splits = attn_decode_splits(lc.sm_count, batch, n_kv_heads, n_ctx);
    float *part = (float *)scratch;
    uint32_t *tickets = (uint32_t *)((char *)scratch + (attn_decode_scratch_floats(batch, n_q_heads, kAttnMaxSplits) * 4 + 255) / 256 * 256);
    if (cudaMemsetAsync(tickets, 0, (size_t)batch * n_kv_heads * 4, lc.stream) != cudaSuccess) return NNC_ERR_CUDA;
    cudaError_t e = launch_attn_decode(lc, q, n_q_heads * 128, (bf16 *)const_cast<void *>(kcache), (bf16 *)const_cast<void *>(vcache),
                                       out, nullptr, nullptr, n_q_heads * 128, part, tickets, nullptr, n_ctx, batch, n_q_heads,
                                       n_kv_heads, max_seq, n_splits, nullptr);
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

int nnc_op_attn_prefill(const float *qkv, const void *kcache, const void *vcache, void *out, void *out_lo, int32_t batch,
                        int32_t T, int32_t n_q_heads, int32_t n_kv_heads, int32_t max_seq, int32_t n_past, void *cuda_stream) {
    if (!qkv || !kcache || !vcache || !out) return NNC_ERR_INVALID_ARG;
    if (batch <= 0 || T <= 0 || n_kv_heads <= 0 || n_q_heads <= 0 || n_q_heads % n_kv_heads || n_past < 0) return NNC_ERR_INVALID_ARG;
    if ((long)n_past + T > max_seq) return NNC_ERR_CAPACITY;
    LaunchCtx lc;
    if (op_ctx(lc, cuda_stream)) return NNC_ERR_CUDA;
    cudaError_t e = launch_attn_prefill(lc, qkv, batch * T, T, kcache, vcache, false, out, out_lo, false, n_q_heads, n_kv_heads,
                                        max_seq, n_past);
    if (e == cudaErrorInvalidValue) return NNC_ERR_INVALID_ARG;
    return e == cudaSuccess ? NNC_OK : NNC_ERR_CUDA;
}

}  // extern "C"
