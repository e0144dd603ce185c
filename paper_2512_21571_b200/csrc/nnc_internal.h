// Host-side internals of libnnc: launch context, kernel launchers, and the launch helper they share.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/nnc.h"

namespace nnc {

typedef __nv_bfloat16 bf16;

struct LaunchCtx {
    cudaStream_t stream;
    int sm_count;
    bool pdl;           // launch with programmatic stream serialization (kernels call pdl_wait themselves)
    int64_t *launches;  // bumped once per kernel launch (may be null)
    int *status;        // device status word raised by kernels whose bounded waits run out (may be null)
};

template <typename... KArgs, typename... Args>
inline cudaError_t launch(const LaunchCtx &lc, void (*kern)(KArgs...), dim3 grid, dim3 block, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = lc.stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = lc.pdl ? 1 : 0;
    if (lc.launches) ++*lc.launches;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Raises a kernel's dynamic shared-memory limit once per device (the attribute belongs to the device's copy of the
// function, so a process that drives several GPUs needs it on each).  `done` is a per-kernel bit mask of devices.
template <typename K>
inline cudaError_t ensure_dynamic_smem(K kern, int bytes, unsigned long long *done) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = 1ull << (dev & 63);
    if (__atomic_load_n(done, __ATOMIC_ACQUIRE) & bit) return cudaSuccess;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) __atomic_fetch_or(done, bit, __ATOMIC_RELEASE);
    return e;
}

// ---- decode GEMV family (decode_gemv.cu) --------------------------------------------------------------
enum GemvMode { kGemvStore = 0, kGemvResidual = 1, kGemvSwiglu = 2, kGemvLogits = 3 };

constexpr int kArgmaxMaxBlocks = 4096;
struct ArgmaxScratch {
    float *part_val;    // [kArgmaxMaxBlocks]
    int32_t *part_idx;  // [kArgmaxMaxBlocks]
    uint32_t *ticket;   // one counter, zero between launches
    int32_t *out;       // result; null = no arg-max
};

// ctr (nullable): two zeroed words owned by this call site, used by the streaming form to hand out work
// dynamically; a call site may be launched again only after ~4 later GEMVs of the same stream have started.
// Weights: bf16 W[n_out][n_in] (wscale null), or FP8 E4M3 codes W[n_out][n_in] with wscale[n_out] (one scale per row).
cudaError_t launch_gemv(const LaunchCtx &lc, const void *W, const float *wscale, const float *x, float *y, int n_out, int n_in,
                        const bf16 *gain, float eps, int mode, const ArgmaxScratch *am, uint32_t *ctr = nullptr);

// streaming form (decode_gemv_stream.cu): n_in a multiple of 8 up to 16384 (8192 for SwiGLU) for bf16, a multiple of
// 16 for FP8 (wb = bytes per weight); launch_gemv uses it whenever the shape allows and, for bf16, falls back to the
// plain-load kernel otherwise
bool gemv_stream_supported(int n_out, int n_in, int mode, int wb = 2);
cudaError_t launch_gemv_stream(const LaunchCtx &lc, const void *W, const float *wscale, int wb, const float *x, float *y,
                               int n_out, int n_in, const bf16 *gain, float eps, int mode, const ArgmaxScratch *am,
                               uint32_t *ctr);

// FP8 E4M3 row quantisation (repack.cu): codes[n_out][n_in], scales[n_out] = 2^e with e the smallest integer such that
// the row's largest magnitude is at most 448 * 2^e; round to nearest even, saturating.  If dequant is not null it
// receives code * 2^e as bf16 (exact); it may alias W.
cudaError_t launch_quantise_rows_e4m3(const LaunchCtx &lc, const bf16 *W, uint8_t *codes, float *scales, bf16 *dequant,
                                      int n_out, int n_in);

// ---- row-wise kernels (decode_misc.cu) ----------------------------------------------------------------
cudaError_t launch_embed(const LaunchCtx &lc, const bf16 *E, const int32_t *tokens, float *x, int rows, int H,
                         int vocab, float *tap);
// skip_q: only the key and value heads are processed (the consumer of the queries normalises and rotates them itself)
// k16 / v16 (nullable): fp16 images of one layer's cache (same layout); the appended rows are written there as well
cudaError_t launch_qk_norm_rope_append(const LaunchCtx &lc, float *qkv, int rows, int rows_per_seq,
                                       const bf16 *g_q, const bf16 *g_k, float eps, const float *rope,
                                       bf16 *kcache_layer, bf16 *vcache_layer, int nq, int nkv, int max_seq,
                                       const int32_t *d_len, bool skip_q, void *k16 = nullptr, void *v16 = nullptr);
// out_f16: `out` receives one fp16 matrix (saturating) instead of a bf16 value (+ residual in out_lo)
cudaError_t launch_rmsnorm_rows(const LaunchCtx &lc, const float *x, const bf16 *gain, bf16 *out, bf16 *out_lo, int rows,
                                int H, float eps, int first, int step, bool out_f16 = false);
cudaError_t launch_copy_f32(const LaunchCtx &lc, const float *src, float *dst, size_t n);
cudaError_t launch_add_len(const LaunchCtx &lc, int32_t *d_len, int delta);

// ---- attention ----------------------------------------------------------------------------------------
constexpr int kAttnMaxSplits = 64;
int attn_decode_splits(int sm_count, int batch, int nkv, int max_ctx);
size_t attn_decode_scratch_floats(int batch, int nq, int n_splits);
// fused != null: q points at the raw fused QKV activation of the new token (query heads, then key heads, then
// value heads); the kernel applies the per-head RMSNorm + RoPE to q and k itself and appends the bf16 K/V row
// at position *d_len + len_add - 1 before attending to it.
struct AttnFused {
    const bf16 *g_q, *g_k;
    const float *rope;
    float eps;
};
cudaError_t launch_attn_decode(const LaunchCtx &lc, const float *q, int q_row_stride, bf16 *kcache, bf16 *vcache,
                               float *out_f32, bf16 *out_bf16, bf16 *out_bf16_lo, int out_row_stride, float *part,
                               uint32_t *tickets, const int32_t *d_len, int len_add, int batch, int nq, int nkv,
                               int max_seq, int n_splits, const AttnFused *fused);
// prompt-phase causal attention on the tcgen05 path (attn_prefill_tc.cu); out: bf16 value (+ residual in out_lo, nullable)
// or, with out_fp16, one fp16 matrix.  n_past (cached positions before this call) is a host value: it sizes the tensor maps.
// fused != null: the query heads of qkv are raw projections and the kernel applies the per-head RMSNorm (g_q) and RoPE
// itself (the K/V rows must already be in the cache: launch_qk_norm_rope_append with skip_q).
// kv_f16: kcache / vcache point at an fp16 image of the cache rows (same [batch][nkv][max_seq][128] layout) and Q and P
// travel as one fp16 term each; otherwise they are the bf16 cache and Q and P travel as two bf16 terms.
cudaError_t launch_attn_prefill(const LaunchCtx &lc, const float *qkv, int rows, int rows_per_seq, const void *kcache,
                                const void *vcache, bool kv_f16, void *out, void *out_lo, bool out_fp16, int nq, int nkv,
                                int max_seq, int n_past, const AttnFused *fused = nullptr);
// fp16 image of cache rows [0, n_pos) of every (sequence, KV head): dst and src share the [heads][max_seq][128] layout
cudaError_t launch_kv_rows_to_f16(const LaunchCtx &lc, const bf16 *src, void *dst, int heads, int max_seq, int n_pos);

// ---- GEMM (gemm_tc.cu) --------------------------------------------------------------------------------
enum GemmEpi { kEpiStoreF32 = 0, kEpiStoreBf16 = 1, kEpiAccumF32 = 2, kEpiSwigluBf16 = 3 };
bool gemm_tc_available();
// X_lo (nullable): bf16 rounding residual of the activations; the product is then (X + X_lo) W^T.
// Y_lo (nullable, SwiGLU epilogue only): receives the rounding residual of the bf16 output.
// scratch (nullable): lets products with at most 128 tokens split K across CTAs (fp32 partial tiles + one ticket
// word per output tile, zero at rest); without it every output tile is computed by one CTA.
struct GemmScratch {
    float *part;
    size_t part_bytes;
    uint32_t *tickets;
    int n_tickets;
};
constexpr size_t kGemmPartBytes = 48u << 20;
constexpr int kGemmTickets = 4096;
// f16: X and W hold fp16 (single term, T > 128 only) and the SwiGLU epilogue writes fp16; out_scale (nullable): DEVICE
// scalar multiplied into the accumulators, undoing the power-of-two scale of an fp16 weight copy.
cudaError_t launch_gemm(const LaunchCtx &lc, const bf16 *X, const bf16 *X_lo, const bf16 *W, void *Y, void *Y_lo, int T,
                        int N, int K, int ldy, int epi, int *status, const GemmScratch *scratch = nullptr, bool f16 = false,
                        const float *out_scale = nullptr);

// ---- repack (repack.cu) -------------------------------------------------------------------------------
// dst rows [row0, row0 + rows) <- src rows [0, rows), row length K (plain row copy into a taller matrix)
cudaError_t launch_copy_rows(const LaunchCtx &lc, const bf16 *src, bf16 *dst, int rows, int K, int dst_row0,
                             int dst_row_step, int src_row0, int src_row_step);

cudaError_t launch_bounds_check_selftest(const LaunchCtx &lc, int code);   // reports one miss with `code` in a checked build

// fp16 copy of a bf16 matrix scaled by a power of two (see repack.cu); scales: DEVICE float[2] <- {2^e, 2^-e}
cudaError_t launch_to_f16_scaled(const LaunchCtx &lc, const bf16 *src, void *dst, size_t n, float *scales, uint32_t *max_bits);

}  // namespace nnc
