// GQA split-K flash-decode: one query token per sequence against a contiguous bf16 KV cache.
//
// Grid (n_splits, n_kv_heads, batch), 128 threads.  A CTA owns one KV head and one contiguous range of
// positions; the G query heads that share the KV head ride along, so every K/V byte is loaded once and feeds
// G dot products.  Positions are walked in tiles of 128 with an online softmax; 16 lanes cover one position
// (16 bytes each), so a warp load is two fully used 256-byte cache rows.  Each CTA emits (m, l, o~) for its
// range; the CTA that finishes last for a (sequence, KV head) folds the partials in split order (a ticket
// counter, nobody waits), which keeps the result independent of arrival order.
//
// HBM-bound on K/V bytes; scores and probabilities never leave shared memory / registers.
#include "common.cuh"
#include "nnc_internal.h"

namespace nnc {

namespace {

constexpr int kTile = 128;
constexpr int kPartStride = kHeadDim + 2;  // o~[128], m, l

__device__ __forceinline__ void unpack8(const uint4 &u, float (&f)[8]) {
    f[0] = bf16_lo(u.x); f[1] = bf16_hi(u.x); f[2] = bf16_lo(u.y); f[3] = bf16_hi(u.y);
    f[4] = bf16_lo(u.z); f[5] = bf16_hi(u.z); f[6] = bf16_lo(u.w); f[7] = bf16_hi(u.w);
}

template <int G>
__global__ void __launch_bounds__(128)
attn_decode_kernel(const float *__restrict__ q, int q_row_stride, const bf16 *__restrict__ kcache,
                   const bf16 *__restrict__ vcache, float *__restrict__ out_f32, bf16 *__restrict__ out_bf16,
                   bf16 *__restrict__ out_bf16_lo, int out_row_stride, float *__restrict__ part, uint32_t *__restrict__ tickets,
                   const int32_t *__restrict__ d_len, int len_add, int nkv, int max_seq, int n_splits) {
    __shared__ float sc[G][kTile];       // scores, then probabilities, of the current tile
    __shared__ float red[4][G][kHeadDim];
    __shared__ float s_m[G], s_l[G], s_alpha[G];
    __shared__ bool is_last;

    pdl_wait();
    const int split = blockIdx.x, j = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = tid >> 4;   // 8 position slots
    const int dl = tid & 15;     // 16-byte slice of the head dimension
    const int n_ctx = (d_len ? *d_len : 0) + len_add;
    const int nq = nkv * G;
    int chunk = (n_ctx + n_splits - 1) / n_splits;
    chunk = (chunk + 15) & ~15;
    if (chunk < 16) chunk = 16;
    const int c0 = split * chunk;
    const int c1 = min(c0 + chunk, n_ctx);
    const int n_active = (n_ctx + chunk - 1) / chunk;
    if (c0 >= n_ctx) return;  // whole CTA; takes no ticket (n_active counts only non-empty ranges)

    // query slice in registers, pre-scaled so that exp2 can be used: s' = s * log2(e) / sqrt(d)
    const float qscale = 1.4426950408889634f * rsqrtf((float)kHeadDim);
    float qr[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const float *qp = q + (size_t)b * q_row_stride + (size_t)(j * G + g) * kHeadDim + dl * 8;
        const float4 a = reinterpret_cast<const float4 *>(qp)[0], c = reinterpret_cast<const float4 *>(qp)[1];
        qr[g][0] = a.x * qscale; qr[g][1] = a.y * qscale; qr[g][2] = a.z * qscale; qr[g][3] = a.w * qscale;
        qr[g][4] = c.x * qscale; qr[g][5] = c.y * qscale; qr[g][6] = c.z * qscale; qr[g][7] = c.w * qscale;
    }
    if (tid < G) { s_m[tid] = -INFINITY; s_l[tid] = 0.f; }

    const size_t head_off = ((size_t)b * nkv + j) * (size_t)max_seq * kHeadDim;
    const bf16 *kbase = kcache + head_off + dl * 8;
    const bf16 *vbase = vcache + head_off + dl * 8;

    float acc[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[g][i] = 0.f;

    for (int t0 = c0; t0 < c1; t0 += kTile) {
        // ---- scores of this tile ----
#pragma unroll 4
        for (int it = 0; it < kTile / 8; ++it) {
            const int p = t0 + it * 8 + slot;
            float s[G];
            if (p < c1) {
                float kf[8];
                unpack8(ldg_stream(kbase + (size_t)p * kHeadDim), kf);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float d = 0.f;
#pragma unroll
                    for (int i = 0; i < 8; ++i) d = fmaf(qr[g][i], kf[i], d);
                    s[g] = d;
                }
            } else {
#pragma unroll
                for (int g = 0; g < G; ++g) s[g] = 0.f;
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) s[g] += __shfl_xor_sync(0xffffffffu, s[g], o);
            }
            if (dl == 0) {
#pragma unroll
                for (int g = 0; g < G; ++g) sc[g][it * 8 + slot] = p < c1 ? s[g] : -INFINITY;
            }
        }
        __syncthreads();
        // ---- online softmax bookkeeping: warp w handles heads w, w+4 ----
        for (int g = warp; g < G; g += 4) {
            float mx = -INFINITY;
#pragma unroll
            for (int i = lane; i < kTile; i += 32) mx = fmaxf(mx, sc[g][i]);
            mx = warp_max(mx);
            const float m_old = s_m[g];
            const float m_new = fmaxf(m_old, mx);  // finite: the tile holds at least one valid position
            float sum = 0.f;
#pragma unroll
            for (int i = lane; i < kTile; i += 32) {
                const float pr = exp2f(sc[g][i] - m_new);
                sc[g][i] = pr;
                sum += pr;
            }
            sum = warp_sum(sum);
            if (lane == 0) {
                const float alpha = exp2f(m_old - m_new);  // 0 on the first tile
                s_alpha[g] = alpha;
                s_l[g] = s_l[g] * alpha + sum;
                s_m[g] = m_new;
            }
        }
        __syncthreads();
        // ---- o~ = o~ * alpha + P V ----
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float al = s_alpha[g];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[g][i] *= al;
        }
#pragma unroll 4
        for (int it = 0; it < kTile / 8; ++it) {
            const int p = t0 + it * 8 + slot;
            if (p < c1) {
                float vf[8];
                unpack8(ldg_stream(vbase + (size_t)p * kHeadDim), vf);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float pr = sc[g][it * 8 + slot];
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[g][i] = fmaf(pr, vf[i], acc[g][i]);
                }
            }
        }
        __syncthreads();
    }

    // ---- fold the 8 position slots: lanes 16 apart, then the 4 warps ----
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[g][i] += __shfl_xor_sync(0xffffffffu, acc[g][i], 16);
    if (lane < 16) {
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int i = 0; i < 8; ++i) red[warp][g][dl * 8 + i] = acc[g][i];
    }
    __syncthreads();
    pdl_launch_dependents();

    float *my_part = part + (((size_t)b * nq + (size_t)j * G) * n_splits + split) * kPartStride;
    // partial for head g lives at my_part + g * n_splits * kPartStride
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float *pp = my_part + (size_t)g * n_splits * kPartStride;
        pp[tid] = red[0][g][tid] + red[1][g][tid] + red[2][g][tid] + red[3][g][tid];
        if (tid == 0) { pp[kHeadDim] = s_m[g]; pp[kHeadDim + 1] = s_l[g]; }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned t = atomicAdd(&tickets[b * nkv + j], 1u);
        is_last = (t == (unsigned)n_active - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // ---- combine (last CTA of this sequence / KV head): o = sum_c 2^(m_c - M) o~_c / sum_c 2^(m_c - M) l_c ----
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const volatile float *pp = part + (((size_t)b * nq + (size_t)j * G + g) * n_splits) * kPartStride;
        float M = -INFINITY;
        for (int c = 0; c < n_active; ++c) M = fmaxf(M, pp[(size_t)c * kPartStride + kHeadDim]);
        float L = 0.f, o = 0.f;
        for (int c = 0; c < n_active; ++c) {
            const float w = exp2f(pp[(size_t)c * kPartStride + kHeadDim] - M);
            L = fmaf(w, pp[(size_t)c * kPartStride + kHeadDim + 1], L);
            o = fmaf(w, pp[(size_t)c * kPartStride + tid], o);
        }
        const float r = o / L;
        const size_t oi = (size_t)b * out_row_stride + (size_t)(j * G + g) * kHeadDim + tid;
        if (out_f32) out_f32[oi] = r;
        if (out_bf16) {
            const bf16 hi = __float2bfloat16_rn(r);
            out_bf16[oi] = hi;
            if (out_bf16_lo) out_bf16_lo[oi] = __float2bfloat16_rn(r - __bfloat162float(hi));
        }
    }
    if (tid == 0) tickets[b * nkv + j] = 0u;
}

}  // namespace

int attn_decode_splits(int sm_count, int batch, int nkv, int max_ctx) {
    // enough CTAs for about two per SM, but never ranges shorter than 64 positions
    int s = (2 * sm_count + batch * nkv - 1) / (batch * nkv);
    const int by_len = (max_ctx + 63) / 64;
    if (s > by_len) s = by_len;
    if (s > kAttnMaxSplits) s = kAttnMaxSplits;
    if (s < 1) s = 1;
    return s;
}

size_t attn_decode_scratch_floats(int batch, int nq, int n_splits) {
    return (size_t)batch * nq * n_splits * kPartStride;
}

cudaError_t launch_attn_decode(const LaunchCtx &lc, const float *q, int q_row_stride, const bf16 *kcache,
                               const bf16 *vcache, float *out_f32, bf16 *out_bf16, bf16 *out_bf16_lo, int out_row_stride,
                               float *part,
                               uint32_t *tickets, const int32_t *d_len, int len_add, int batch, int nq, int nkv,
                               int max_seq, int n_splits) {
    const int G = nq / nkv;
    dim3 grid(n_splits, nkv, batch), block(128);
#define NNC_ATTN_CASE(GG)                                                                                       \
    case GG:                                                                                                    \
        return launch(lc, attn_decode_kernel<GG>, grid, block, q, q_row_stride, kcache, vcache, out_f32,       \
                      out_bf16, out_bf16_lo, out_row_stride, part, tickets, d_len, len_add, nkv, max_seq, n_splits);
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
