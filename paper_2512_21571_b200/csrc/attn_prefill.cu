// Causal attention for a block of new tokens (the prompt phase): query at position p attends to cache
// positions 0..p of its sequence.  K and V are read from the bf16 cache, which already holds the new tokens.
//
// One warp per (token row, query head).  Keys are taken 32 at a time, one per lane for the score (the query
// sits in shared memory and is broadcast), then the 32 probabilities are shuffled around while every lane
// accumulates its 4 output elements.  Online softmax in fp32.
#include "common.cuh"
#include "nnc_internal.h"

namespace nnc {

namespace {

__global__ void __launch_bounds__(128)
attn_prefill_kernel(const float *__restrict__ qkv, int rows, int rows_per_seq, const bf16 *__restrict__ kcache,
                    const bf16 *__restrict__ vcache, bf16 *__restrict__ out, bf16 *__restrict__ out_lo, int nq, int nkv,
                    int max_seq, const int32_t *__restrict__ d_len) {
    __shared__ __align__(16) float qs[4][kHeadDim];
    pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long unit = (long)blockIdx.x * 4 + warp;
    if (unit >= (long)rows * nq) return;
    const int row = (int)(unit / nq), head = (int)(unit % nq);
    const int seq = row / rows_per_seq;
    const int pos = *d_len + row % rows_per_seq;
    const int G = nq / nkv, j = head / G;
    const int heads = nq + 2 * nkv;
    const float qscale = 1.4426950408889634f * rsqrtf((float)kHeadDim);
    {
        const float4 v = reinterpret_cast<const float4 *>(qkv + (size_t)row * heads * kHeadDim + (size_t)head * kHeadDim)[lane];
        reinterpret_cast<float4 *>(qs[warp])[lane] = make_float4(v.x * qscale, v.y * qscale, v.z * qscale, v.w * qscale);
    }
    __syncwarp();
    const size_t head_off = ((size_t)seq * nkv + j) * (size_t)max_seq * kHeadDim;
    const bf16 *kb = kcache + head_off, *vb = vcache + head_off;
    float m = -INFINITY, l = 0.f;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const int n_ctx = pos + 1;
    for (int t0 = 0; t0 < n_ctx; t0 += 32) {
        const int p = t0 + lane;
        float s = -INFINITY;
        if (p < n_ctx) {
            const uint4 *kr = reinterpret_cast<const uint4 *>(kb + (size_t)p * kHeadDim);
            float d = 0.f;
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const uint4 u = kr[c];
                const float4 a = reinterpret_cast<const float4 *>(qs[warp])[2 * c];
                const float4 b = reinterpret_cast<const float4 *>(qs[warp])[2 * c + 1];
                d = fmaf(bf16_lo(u.x), a.x, d); d = fmaf(bf16_hi(u.x), a.y, d);
                d = fmaf(bf16_lo(u.y), a.z, d); d = fmaf(bf16_hi(u.y), a.w, d);
                d = fmaf(bf16_lo(u.z), b.x, d); d = fmaf(bf16_hi(u.z), b.y, d);
                d = fmaf(bf16_lo(u.w), b.z, d); d = fmaf(bf16_hi(u.w), b.w, d);
            }
            s = d;
        }
        const float m_new = fmaxf(m, warp_max(s));
        const float pr = exp2f(s - m_new);
        const float alpha = exp2f(m - m_new);
        l = l * alpha + warp_sum(pr);
        m = m_new;
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] *= alpha;
        const int nv = min(32, n_ctx - t0);
        for (int t = 0; t < nv; ++t) {
            const float pt = __shfl_sync(0xffffffffu, pr, t);
            const uint2 u = reinterpret_cast<const uint2 *>(vb + (size_t)(t0 + t) * kHeadDim)[lane];
            acc[0] = fmaf(pt, bf16_lo(u.x), acc[0]);
            acc[1] = fmaf(pt, bf16_hi(u.x), acc[1]);
            acc[2] = fmaf(pt, bf16_lo(u.y), acc[2]);
            acc[3] = fmaf(pt, bf16_hi(u.y), acc[3]);
        }
    }
    const float inv = 1.f / l;
    uint2 o;
    o.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
    o.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
    const size_t oi = (size_t)row * nq * kHeadDim + (size_t)head * kHeadDim;
    reinterpret_cast<uint2 *>(out + oi)[lane] = o;
    if (out_lo) {  // rounding residual: out + out_lo carries 16 mantissa bits
        uint2 r;
        r.x = pack_bf16x2(acc[0] * inv - bf16_lo(o.x), acc[1] * inv - bf16_hi(o.x));
        r.y = pack_bf16x2(acc[2] * inv - bf16_lo(o.y), acc[3] * inv - bf16_hi(o.y));
        reinterpret_cast<uint2 *>(out_lo + oi)[lane] = r;
    }
}

}  // namespace

cudaError_t launch_attn_prefill(const LaunchCtx &lc, const float *qkv, int rows, int rows_per_seq, const bf16 *kcache,
                                const bf16 *vcache, bf16 *out, bf16 *out_lo, int nq, int nkv, int max_seq,
                                const int32_t *d_len) {
    const long units = (long)rows * nq;
    return launch(lc, attn_prefill_kernel, dim3((unsigned)((units + 3) / 4)), dim3(128), qkv, rows, rows_per_seq,
                  kcache, vcache, out, out_lo, nq, nkv, max_seq, d_len);
}

}  // namespace nnc
