// GQA split-K flash-decode: one query token per sequence against a contiguous bf16 KV cache, optionally fused
// with the per-head QK-RMSNorm + RoPE of the new token and the append of its K/V row.
//
// HBM-bound on K/V bytes (2 * 2 * n_kv_heads * 128 bytes per cached position), so the kernel is arranged for
// wide loads and few instructions per byte:
//   - grid (n_splits, n_kv_heads, batch), 4 warps.  A CTA owns one KV head and one contiguous range of
//     positions; its G query heads ride along, so every K/V byte is loaded once and feeds G dot products.
//   - the two products run on the warp-level tensor-core path (mma.sync m16n8k16, bf16 in, fp32 accumulate) in
//     transposed form: S^T = K Q^T and O^T = V^T P^T, so 16 cached positions (resp. 16 head-dimension elements)
//     fill the 16-row operand and the G <= 8 query heads are the 8-column operand -- no padding rows.  Q and the
//     probabilities are fed as two bf16 terms each (value + rounding residual), so the result keeps fp32-level
//     accuracy.  K and V fragments are loaded straight from global memory as 16-byte vectors: the contraction
//     index of K Q^T (the head dimension) and the row index of V^T P^T are permuted so that what a thread needs
//     is contiguous in the cache row.
//   - every warp walks its own blocks of 16 positions with a private online softmax; warps, then CTAs, are
//     merged through (m, l, o~) partials.  The CTA that finishes last for a (sequence, KV head) folds the
//     partials in split order (a ticket counter; nobody waits), so the result does not depend on arrival order.
//   - before waiting on the preceding kernel, the CTA asks for its K/V range to be brought into L2
//     (cp.async.bulk.prefetch): the cache rows of earlier positions do not depend on that kernel.
#include "attn_decode_body.cuh"

namespace nnc {

namespace {

template <int G, bool FUSED>
__global__ void __launch_bounds__(kAttnWarps * 32) attn_decode_kernel(const AttnParams p) {
    NNC_TRACE_SCOPE(30);
    __shared__ AttnSmem<G> sm;
    const int split = blockIdx.x, j = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x;

    pdl_launch_dependents();
    // ---- before the dependency: ask for this CTA's K/V range in L2 (rows of earlier positions are stable) ----
    {
        const size_t head_off = ((size_t)b * p.nkv + j) * (size_t)p.max_seq * kHeadDim;
        const int n_guess = (p.d_len ? *p.d_len : 0) + p.len_add;   // only a hint here; read again after the wait
        int chunk = (n_guess + p.n_splits - 1) / p.n_splits;
        chunk = (chunk + 15) & ~15;
        if (chunk < 16) chunk = 16;
        if (n_guess <= kSingleRange) chunk = kSingleRange;
        const int c0 = split * chunk, c1 = min(c0 + chunk, min(n_guess, p.max_seq));
        if (tid < 2 && c1 > c0) {
            const bf16 *src = (tid ? p.vcache : p.kcache) + head_off + (size_t)c0 * kHeadDim;
            // short ranges whole; long ranges only their head (the body prefetches ahead of itself as it goes)
            const uint32_t bytes = (uint32_t)min(c1 - c0, kPrefetchAhead * kAttnWarps * 16) * kHeadDim * 2u;
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
        }
    }
    pdl_wait();
    NNC_TRACE_MARK();
    attn_decode_body<G, FUSED>(p, split, j, b, tid, sm, 1);
}


}  // namespace

int attn_decode_splits(int sm_count, int batch, int nkv, int max_ctx) {
    // Two CTAs are resident per SM.  Among the split counts that keep ranges at 64 positions or more, take the one
    // whose CTA count fills whole rounds of those slots best (a last round that is mostly empty costs a full range's
    // time), with a small charge per split.
    const int slots = 2 * sm_count, heads = batch * nkv;
    int s_max = (max_ctx + 63) / 64;
    if (s_max > kAttnMaxSplits) s_max = kAttnMaxSplits;
    if (s_max < 1) s_max = 1;
    int best = 1;
    double best_score = -1.0;
    for (int s = 1; s <= s_max; ++s) {
        const long long ctas = (long long)heads * s;
        const long long rounds = (ctas + slots - 1) / slots;
        const double eff = (double)ctas / (double)(rounds * slots);
        const double score = eff - 0.002 * s;   // every further split adds a partial result to write and to combine
        if (score > best_score) { best_score = score; best = s; }
    }
    return best;
}

size_t attn_decode_scratch_floats(int batch, int nq, int n_splits) {
    return (size_t)batch * nq * n_splits * kPartStride;
}

cudaError_t launch_attn_decode(const LaunchCtx &lc, const float *q, int q_row_stride, bf16 *kcache, bf16 *vcache,
                               float *out_f32, bf16 *out_bf16, bf16 *out_bf16_lo, int out_row_stride, float *part,
                               uint32_t *tickets, const int32_t *d_len, int len_add, int batch, int nq, int nkv,
                               int max_seq, int n_splits, const AttnFused *fused) {
    const int G = nq / nkv;
    AttnParams p;
    p.q = q; p.q_row_stride = q_row_stride; p.kcache = kcache; p.vcache = vcache;
    p.out_f32 = out_f32; p.out_bf16 = out_bf16; p.out_bf16_lo = out_bf16_lo; p.out_row_stride = out_row_stride;
    p.part = part; p.part_floats = attn_decode_scratch_floats(batch, nq, n_splits);
    p.tickets = tickets; p.d_len = d_len; p.len_add = len_add;
    p.nkv = nkv; p.max_seq = max_seq; p.n_splits = n_splits;
    p.g_q = fused ? fused->g_q : nullptr; p.g_k = fused ? fused->g_k : nullptr;
    p.rope = fused ? fused->rope : nullptr; p.eps = fused ? fused->eps : 0.f;
    dim3 grid(n_splits, nkv, batch), block(kAttnWarps * 32);
#define NNC_ATTN_CASE(GG)                                                                  \
    case GG:                                                                               \
        return fused ? launch(lc, attn_decode_kernel<GG, true>, grid, block, p)           \
                     : launch(lc, attn_decode_kernel<GG, false>, grid, block, p);
    switch (G) {
        NNC_ATTN_CASE(1)
        NNC_ATTN_CASE(2)
        NNC_ATTN_CASE(4)
        NNC_ATTN_CASE(8)
    }
#undef NNC_ATTN_CASE
    return cudaErrorInvalidValue;
}

}  // namespace nnc
