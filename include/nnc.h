/*
 * nnc.h -- C ABI of the B200-native Qwen3 forward pass (libnnc.so).
 *
 * The paper frames LLM deployment as "prepare the model once ahead of time, then run a prompt phase followed
 * by token-by-token decoding at batch 1, reporting decode tokens/s" (Section 4, Evaluation; Section 3.3.1 for
 * laying constants out once where the kernels read them).  The three main calls mirror that framing:
 *
 *     nnc_model_create(config, weights)   one-time weight repack + workspace carve-up
 *     nnc_prefill(tokens)                 the prompt phase
 *     nnc_decode_step(token) -> logits    one decoding step (the HBM-bound hot path)
 *
 * Conventions
 *   - Plain C, no exceptions.  Every function that can fail returns an int status: NNC_OK (0) or a negative
 *     nnc_status.  nnc_last_error() gives a human-readable line for the last failure of that model.
 *   - "DEVICE pointer" = CUDA global memory on the device that was current in nnc_model_create.
 *     "HOST pointer" = ordinary host memory.  Unless a parameter says HOST it is a DEVICE pointer.
 *   - The library never allocates or frees device memory: the caller supplies one workspace at create time
 *     (nnc_workspace_bytes tells how large) and owns it; it must stay alive until nnc_model_destroy.
 *   - All work is enqueued on the CUDA stream given at create time (a cudaStream_t passed as void*; NULL =
 *     the legacy default stream) and is asynchronous unless a function says it synchronises.
 *   - Errors that the host can see (bad configuration, null pointers, cache overflow, batch too large,
 *     workspace too small) are returned before anything is launched and leave the model unchanged.  Launch
 *     errors reported by the CUDA runtime are returned as NNC_ERR_CUDA.  Kernels never trap or assert; every
 *     device-side wait is bounded and reports through a status word that nnc_device_status() reads.
 *   - All matrices are bf16, row-major W[out][in] (y = W x); bf16 values are IEEE bfloat16 bit patterns.
 *   - The sequences of a batch advance in lock step: they all hold the same number of cached positions.
 */
#ifndef NNC_H_
#define NNC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    NNC_OK = 0,
    NNC_ERR_INVALID_ARG = -1,   /* null pointer, non-positive size, unsupported shape */
    NNC_ERR_WORKSPACE = -2,     /* workspace smaller than nnc_workspace_bytes(), or misaligned */
    NNC_ERR_CAPACITY = -3,      /* cache length + new tokens > max_seq, batch > max_batch, tokens > max_tokens */
    NNC_ERR_CUDA = -4,          /* a CUDA runtime / driver call failed; see nnc_last_error */
    NNC_ERR_DEVICE_STATUS = -5  /* a kernel reported a bounded wait that ran out */
} nnc_status;

typedef struct nnc_model nnc_model; /* opaque; host struct owned by the library */

/* Model and capacity description.  Supported: head_dim == 128; n_q_heads a multiple of n_kv_heads with at
 * most 8 query heads per KV head; hidden, intermediate multiples of 64; everything positive. */
typedef struct {
    int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, intermediate, vocab;
    int32_t max_seq;        /* KV-cache capacity in positions per sequence */
    int32_t max_batch;      /* sequences held in the cache */
    int32_t max_tokens;     /* most tokens one nnc_prefill call may carry (batch * n_tokens); >= max_batch */
    int32_t tie_embeddings; /* 1: the lm_head is the embedding matrix */
    float rms_eps;          /* 1e-6 for Qwen3 */
    float rope_theta;       /* 1e6 for Qwen3 */
    int32_t tc_operands;    /* operand feed of the tensor-core path (prompt phase, batched decode).  The residual stream
                             * stays fp32 everywhere; this only says how an activation matrix enters a tcgen05.mma.
                             * 0 (default): calls with more than 128 tokens multiply the attention output, the MLP input and
                             *    the SwiGLU output as ONE fp16 term with fp16 copies of Wo, Wgate/up and Wdown (made at
                             *    create time when max_tokens > 128; scaled by a power of two per matrix, exact for bf16
                             *    weights), and the QKV input -- the operand deep models are sensitive to -- as TWO bf16
                             *    terms (value + rounding residual, ~16 mantissa bits).  Calls with at most 128 tokens use
                             *    two bf16 terms throughout (they are bound by streaming the weights, not by the MMAs).
                             * 1: two bf16 terms throughout, no fp16 weight copies (smaller workspace, ~1.8x the tensor work
                             *    of mode 0 in the prompt phase).
                             * 2: one bf16 term throughout (half the tensor work of mode 1; 2^-9 per operand accumulates to
                             *    a few percent of hidden-state error over ~30 layers, outside the parity tolerance). */
    int32_t weight_format;  /* 0 (default): bf16 weights.  1: the second weight precision (the paper evaluates two, Section
                             * 4.1) -- weight-only FP8: at create time every matrix that is multiplied (QKV, O, gate/up,
                             * down, lm_head; a tied embedding is that same matrix) is quantised row by row to E4M3 codes
                             * times a power-of-two scale 2^e per output row (e the smallest integer with max|w| <= 448 *
                             * 2^e, round to nearest even, saturating), and the bf16 copy in the workspace is replaced by
                             * the dequantised values (exact in bf16).  Batch-1 decode streams the codes (half the bytes per
                             * step); the tensor-core paths multiply the dequantised bf16 matrices, so every path computes
                             * the same model: the forward pass on the dequantised weights. */
    int32_t serial_launches; /* 0 (default): kernels are launched with programmatic stream serialization, so a
                             * kernel's set-up and weight prefetch overlap its predecessor's tail.  1: plain stream
                             * order (for debugging and for timing the overlap's worth). */
} nnc_config;

/* Per-layer weights: DEVICE pointers, bf16.  Read only during nnc_model_create (they are repacked into the
 * workspace) and may be freed by the caller afterwards.
 *   wq [n_q_heads*128][hidden]   wk, wv [n_kv_heads*128][hidden]   wo [hidden][n_q_heads*128]
 *   w_gate, w_up [intermediate][hidden]   w_down [hidden][intermediate]
 *   g_in, g_post [hidden] (RMSNorm gains before attention / before the MLP)   g_q, g_k [128] (per-head
 *   query / key RMSNorm gains, shared by the heads of the layer) */
typedef struct {
    const void *wq, *wk, *wv, *wo, *w_gate, *w_up, *w_down;
    const void *g_in, *g_post, *g_q, *g_k;
} nnc_layer_weights;

typedef struct {
    const void *embed;               /* DEVICE [vocab][hidden] */
    const void *lm_head;             /* DEVICE [vocab][hidden]; NULL when tie_embeddings */
    const void *g_final;             /* DEVICE [hidden] */
    const nnc_layer_weights *layers; /* HOST array of n_layers entries (holding DEVICE pointers) */
} nnc_weights;

/* Bytes of workspace nnc_model_create needs for this configuration (repacked weights, KV cache, RoPE table,
 * activations, split-K scratch).  Returns 0 for an invalid configuration.  Pure host arithmetic. */
size_t nnc_workspace_bytes(const nnc_config *config);

/* Ahead-of-time preparation (the paper's "constants laid out once", Section 3.3.1): validates the
 * configuration, carves the workspace (256-byte aligned DEVICE pointer, at least nnc_workspace_bytes), builds
 * the RoPE table on the host in double precision, and repacks the weights on the device: Wq|Wk|Wv are
 * concatenated row-wise, gate/up rows are interleaved pairwise (row 2i = gate_i, row 2i+1 = up_i) so that one
 * warp owns both halves of a SwiGLU output.  Synchronises the stream before returning.  *out is set only on
 * success.  The cache starts empty. */
int nnc_model_create(const nnc_config *config, const nnc_weights *weights, void *workspace,
                     size_t workspace_bytes, void *cuda_stream, nnc_model **out);

/* Releases the host struct, CUDA graphs and tensor maps.  Synchronises the stream.  NULL is ignored. */
void nnc_model_destroy(nnc_model *model);

/* Prompt phase (Section 4: a prompt is processed, then decoding starts).  tokens: int32 [batch][n_tokens],
 * ids in [0, vocab); out-of-range ids are clamped on the device.  The tokens take positions len .. len +
 * n_tokens - 1 of every sequence, their K/V are appended, and len grows by n_tokens.
 * logits: fp32 [batch][vocab] (last position of each sequence), or [batch][n_tokens][vocab] when
 * all_positions != 0; may be NULL to skip the lm_head. */
int nnc_prefill(nnc_model *model, const int32_t *tokens, int32_t batch, int32_t n_tokens, float *logits,
                int32_t all_positions);

/* One decoding step (Section 4: throughput is measured over this stage).  tokens: int32 [batch]; each
 * sequence's token takes position len; len grows by one.  logits: fp32 [batch][vocab].  argmax: int32
 * [batch] or NULL (batch 1 only); lowest index wins ties.  The whole step is one CUDA graph launch, captured on
 * first use for the given buffers and batch size and re-used while they stay the same. */
int nnc_decode_step(nnc_model *model, const int32_t *tokens, int32_t batch, float *logits, int32_t *argmax);

/* End-to-end variants with HOST buffers: copy the tokens to the device, run the step, copy logits (and the
 * argmax, if not NULL) back, and synchronise the stream before returning.  HOST pointers throughout; pinned
 * memory makes the copies faster but is not required.  logits_host may be NULL when only argmax is wanted. */
int nnc_decode_step_host(nnc_model *model, const int32_t *tokens_host, int32_t batch, float *logits_host,
                         int32_t *argmax_host);
int nnc_prefill_host(nnc_model *model, const int32_t *tokens_host, int32_t batch, int32_t n_tokens,
                     float *logits_host, int32_t all_positions);

/* Set the raw cache contents of one layer of one sequence, positions [0, n_pos): k, v DEVICE bf16
 * [n_kv_heads][n_pos][128] (K as the cache stores it: already normalised and rotated).  nnc_set_length then
 * declares how many positions are valid. */
int nnc_kv_import(nnc_model *model, int32_t layer, int32_t batch_index, const void *k, const void *v,
                  int32_t n_pos);
/* Copy the cache of one layer of one sequence, positions [0, n_pos), to k, v (DEVICE, same layout). */
int nnc_kv_export(nnc_model *model, int32_t layer, int32_t batch_index, void *k, void *v, int32_t n_pos);

int nnc_set_length(nnc_model *model, int32_t n_pos); /* cached positions := n_pos (0 empties the cache) */
int32_t nnc_get_length(const nnc_model *model);

/* Parity instrumentation.  taps: DEVICE fp32 [n_layers + 1][rows][hidden] (rows = batch for a decode step,
 * batch * n_tokens for a prefill), receiving the residual stream after the embedding and after every layer of
 * each following call; NULL switches it off.  While a tap is set, decode steps run kernel by kernel instead
 * of through the captured graph (same kernels, same order). */
int nnc_set_hidden_tap(nnc_model *model, float *taps);

/* One decoder layer, one step, batch 1, on a caller-supplied residual-stream vector: x_in, x_out DEVICE fp32
 * [hidden].  The token sits at position len; its K/V are appended to that layer's cache; len is NOT changed
 * (call nnc_set_length to advance). */
int nnc_layer_decode(nnc_model *model, int32_t layer, const float *x_in, float *x_out);

/* Write the ORIGINAL (caller-layout) matrix back from the repacked store: which = 0 wq, 1 wk, 2 wv, 3 wo,
 * 4 w_gate, 5 w_up, 6 w_down; out DEVICE bf16 of that matrix's shape.  Lets a test check that the repack
 * loses nothing (with weight_format 1 the store holds the dequantised values, and those are what comes back). */
int nnc_unrepack(nnc_model *model, int32_t layer, int32_t which, void *out);

/* Reads (and clears) the device status word; synchronises the stream.  0 = no kernel gave up on a wait. */
int nnc_device_status(nnc_model *model, int32_t *status_out /* HOST */);

/* Number of kernels this library launched on behalf of `model` since creation (graph nodes count once per
 * graph launch). */
int64_t nnc_launch_count(const nnc_model *model);

/* Debugging aid.  A library built with -DNNC_BOUNDS_CHECK compares, inside the kernels, the indices that rest on the
 * host's capacity checks (cache positions, matrix row ranges, scratch slots) with their extents; a miss is counted and
 * the access skipped (no trap, no out-of-range access).  This call synchronises the device and returns the number of
 * misses since the last call and the code of the first one (HOST pointers); in a normal build *misses_out is -1.
 * nnc_bounds_check_selftest launches a kernel that touches no memory and, in a checked build, reports one miss with
 * `code` (nothing in a normal build): it shows the counter at work. */
int nnc_bounds_check_report(int32_t *misses_out, int32_t *first_code_out);
int nnc_bounds_check_selftest(int32_t code, void *cuda_stream);

const char *nnc_last_error(const nnc_model *model); /* never NULL; valid until the next call on the model */
const char *nnc_status_string(int status);

/* ---- single operations, exposed for kernel-level tests and isolated timing ----------------------------
 * Each runs on `cuda_stream`, allocates nothing, and returns an nnc_status. */

/* y[T][n_out] = (X + X_lo)[T][n_in] * W[n_out][n_in]^T on the tensor cores (tcgen05, fp32 accumulation in
 * tensor memory).  X, W bf16 row-major (n_in contiguous), n_in a multiple of 64, n_out a multiple of 8.
 * X_lo: NULL, or a second bf16 [T][n_in] matrix (the rounding residual of the activations) multiplied with
 * the same weights into the same accumulator.
 * out_f32 != 0: Y is fp32 (and, if accumulate != 0, Y += product); otherwise Y is bf16. */
int nnc_op_gemm(const void *X, const void *X_lo, const void *W, void *Y, int32_t T, int32_t n_out, int32_t n_in,
                int32_t out_f32, int32_t accumulate, void *cuda_stream);
/* The same product with the SwiGLU epilogue of the MLP: W rows interleaved (row 2i = gate_i, row 2i+1 = up_i),
 * Y bf16 [T][n_out/2], Y[t][i] = silu(gate) * up; n_out a multiple of 16 (rows of Y stay 16-byte aligned). */
int nnc_op_gemm_swiglu(const void *X, const void *X_lo, const void *W, void *Y, void *Y_lo, int32_t T,
                       int32_t n_out, int32_t n_in, void *cuda_stream); /* Y_lo: NULL or the residual of Y */
/* nnc_op_gemm for few tokens (T <= 128), where the product is bound by streaming W: the (output tile, K block)
 * space is cut into one equal contiguous range per SM, so every SM streams the same share of W.  A tile whose K
 * range straddles a cut is finished through fp32 partial tiles in `scratch`: the CTA holding the tile's first K
 * piece waits (bounded; on expiry the status word is set) for the others and adds the pieces in K order
 * (deterministic).  scratch: DEVICE, 256-byte aligned, at least 16 KiB + 2 * 64 KiB * (number of SMs) to cover
 * every T (a smaller one makes large T fall back to whole tiles); its first 16 KiB are flags that must be zero
 * before the first call and are left zero by every call that ends without error.  Calls that share a scratch
 * must not overlap on the device.  With T > 128 it behaves as nnc_op_gemm. */
int nnc_op_gemm_splitk(const void *X, const void *X_lo, const void *W, void *Y, int32_t T, int32_t n_out, int32_t n_in,
                       int32_t out_f32, int32_t accumulate, void *scratch, size_t scratch_bytes, void *cuda_stream);
/* The fp16 forms used by the prompt phase: X fp16 [T][n_in] (T > 128), W fp16 [n_out][n_in], one term.  out_scale: NULL
 * or a DEVICE float multiplied into every accumulator before the epilogue (undoes the scale of an fp16 weight copy).
 * nnc_op_gemm_f16: Y fp32 [T][n_out], Y += product when accumulate != 0.  nnc_op_gemm_swiglu_f16: W rows interleaved
 * gate/up, Y fp16 [T][n_out/2] (values beyond +-65504 saturate). */
int nnc_op_gemm_f16(const void *X, const void *W, float *Y, int32_t T, int32_t n_out, int32_t n_in, int32_t accumulate,
                    const float *out_scale, void *cuda_stream);
int nnc_op_gemm_swiglu_f16(const void *X, const void *W, void *Y, int32_t T, int32_t n_out, int32_t n_in,
                           const float *out_scale, void *cuda_stream);
/* dst (fp16) = src (bf16) * 2^e, n elements (a multiple of 8), with e chosen so that the largest magnitude lands in
 * [2^14, 2^15): exact for every element down to 2^-32 of the largest (smaller ones round with an error below 2^-39 of the largest).  scales: DEVICE float[2] receiving {2^e, 2^-e};
 * scratch_word: DEVICE uint32 used during the call. */
int nnc_op_to_f16_scaled(const void *src, void *dst, size_t n, float *scales, uint32_t *scratch_word, void *cuda_stream);

/* Status word of the nnc_op_* tensor-core kernels (0 = no bounded wait ran out); synchronises the device and
 * clears the word.  status_out is a HOST pointer. */
int nnc_op_status(int32_t *status_out);

/* y[n_out] = W[n_out][n_in] x (batch-1 streaming GEMV, fp32 accumulate).  x fp32 [n_in]; y fp32.
 * If gain != NULL (bf16 [n_in]) x is first RMS-normalised with that gain and eps.
 * mode 0: y = Wx;  mode 1: y += Wx (residual);  mode 2: rows interleaved gate/up, y[n_out/2] = silu(g)*u.
 * mode | NNC_GEMV_CHAINED: launch the way the decode step does, with programmatic stream serialization, so that
 * back-to-back calls on one stream overlap the next kernel's weight prefetch with the previous kernel's tail
 * (x and y of consecutive chained calls must then not depend on each other's weights buffer being rewritten). */
#define NNC_GEMV_CHAINED 0x100
int nnc_op_gemv(const void *W, const float *x, float *y, int32_t n_out, int32_t n_in, const void *gain,
                float eps, int32_t mode, void *cuda_stream);

/* FP8 E4M3 row quantisation (nnc_config::weight_format 1): W bf16 [n_out][n_in] -> codes uint8 [n_out][n_in] and
 * scales fp32 [n_out] (= 2^e per row); dequant: NULL, or bf16 [n_out][n_in] receiving code * 2^e (may be W itself).
 * n_in a multiple of 8. */
int nnc_op_quantise_rows_e4m3(const void *W, void *codes, float *scales, void *dequant, int32_t n_out, int32_t n_in,
                              void *cuda_stream);
/* nnc_op_gemv on FP8 weights: y = diag(scales) * codes * x with the same modes, gain and chaining flag; n_in a multiple
 * of 16 (up to 16384; 8192 with mode 2). */
int nnc_op_gemv_fp8(const void *codes, const float *scales, const float *x, float *y, int32_t n_out, int32_t n_in,
                    const void *gain, float eps, int32_t mode, void *cuda_stream);

/* Split-K flash-decode for one query token per sequence over a contiguous cache.
 *   q fp32 [batch][n_q_heads][128] (already normalised and rotated);  kcache, vcache bf16
 *   [batch][n_kv_heads][max_seq][128];  n_ctx positions are attended;  out fp32 [batch][n_q_heads][128].
 *   scratch: DEVICE, at least nnc_attn_scratch_bytes(batch, n_q_heads, n_ctx) bytes, 256-byte aligned. */
size_t nnc_attn_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t n_ctx);
int nnc_op_attn_decode(const float *q, const void *kcache, const void *vcache, float *out, int32_t batch,
                       int32_t n_q_heads, int32_t n_kv_heads, int32_t max_seq, int32_t n_ctx, void *scratch,
                       void *cuda_stream);

/* Causal attention of the prompt phase for T new tokens per sequence (tcgen05 tensor cores; the score and
 * probability tile stays in tensor memory between the two products, cf. the pass-through layout of Section 3.1.2).
 *   qkv fp32 [batch * T][(n_q_heads + 2 n_kv_heads) * 128]: only the query heads are read (already normalised and
 *   rotated);  kcache, vcache bf16 [batch][n_kv_heads][max_seq][128] must already hold the new tokens' K/V at
 *   positions n_past .. n_past + T - 1;  the query of token s attends to positions 0 .. n_past + s.  Cache rows at
 *   positions >= n_past + T are never read (they may hold anything).
 *   out (and out_lo, NULL or the bf16 rounding residual): bf16 [batch * T][n_q_heads * 128], 16-byte aligned.
 *   n_past: cached positions before these tokens, a host value; n_past + T > max_seq returns NNC_ERR_CAPACITY. */
int nnc_op_attn_prefill(const float *qkv, const void *kcache, const void *vcache, void *out, void *out_lo, int32_t batch,
                        int32_t T, int32_t n_q_heads, int32_t n_kv_heads, int32_t max_seq, int32_t n_past,
                        void *cuda_stream);

/* The one-term form the prompt phase uses: k16, v16 fp16 images of the cache rows (same layout; exact for bf16 values
 * inside the fp16 range), queries and probabilities travel as one fp16 term each (half the tensor-core work of the form
 * above), out fp16 [batch * T][n_q_heads * 128]. */
int nnc_op_attn_prefill_f16(const float *qkv, const void *k16, const void *v16, void *out, int32_t batch, int32_t T,
                            int32_t n_q_heads, int32_t n_kv_heads, int32_t max_seq, int32_t n_past, void *cuda_stream);

/* The same operation for callers that cannot allocate device memory (the paper has no counterpart: this is a
 * deployment convenience of this library).  A plug-in that is handed only its inputs and outputs, or a process
 * whose device memory is owned by another runtime's pool, cannot produce the scratch buffer above; here the
 * scratch lives in a fixed array inside the library image (NNC_ATTN_STATIC_SCRATCH_BYTES per GPU, held from
 * library load until process exit) and the call allocates nothing.
 *   - Needs above that size (nnc_attn_scratch_bytes(batch, n_q_heads, n_ctx) > NNC_ATTN_STATIC_SCRATCH_BYTES,
 *     i.e. roughly batch * n_q_heads > 120) return NNC_ERR_CAPACITY, print one line to stderr, launch nothing.
 *   - Every call on a device shares the array and finds the previous call's contents in it; the call clears
 *     what must start at zero itself.  Calls that overlap on the GPU (two streams, two threads) race on the
 *     array: serialise them.
 *   - The first call on each device looks up the array's device address; issue that first call outside any
 *     stream capture. */
#define NNC_ATTN_STATIC_SCRATCH_BYTES (4u << 20)
int nnc_op_attn_decode_static(const float *q, const void *kcache, const void *vcache, float *out, int32_t batch,
                              int32_t n_q_heads, int32_t n_kv_heads, int32_t max_seq, int32_t n_ctx,
                              void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* NNC_H_ */
