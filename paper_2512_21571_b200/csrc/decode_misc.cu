// Small row-wise kernels of the forward pass: embedding gather, per-head QK-RMSNorm + RoPE + KV append,
// row-wise RMSNorm to a bf16 GEMM operand, and the device-side position counter.
#include "common.cuh"
#include "nnc_internal.h"

namespace nnc {

namespace {

// x[r][:] = float(E[token_r][:]); one block per row.  Out-of-range ids are clamped.
__global__ void embed_kernel(const bf16 *__restrict__ E, const int32_t *__restrict__ tokens, float *__restrict__ x,
                             int H, int vocab, float *__restrict__ tap) {
    NNC_TRACE_SCOPE(1);
    pdl_wait();
    const int r = blockIdx.x;
    int tok = tokens[r];
    tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);
    const uint2 *src = reinterpret_cast<const uint2 *>(E + (size_t)tok * H);
    float4 *dst = reinterpret_cast<float4 *>(x + (size_t)r * H);
    float4 *tp = tap ? reinterpret_cast<float4 *>(tap + (size_t)r * H) : nullptr;
    for (int i = threadIdx.x; i < H / 4; i += blockDim.x) {
        const uint2 u = src[i];
        const float4 v = make_float4(bf16_lo(u.x), bf16_hi(u.x), bf16_lo(u.y), bf16_hi(u.y));
        dst[i] = v;
        if (tp) tp[i] = v;
    }
    pdl_launch_dependents();
}

// One warp per (row, head) of the fused QKV activation [rows][(nq + 2 nkv) * 128] (fp32).
//   q heads: q <- RoPE_p(RMSNorm_128(q; g_q)) in place (left alone with skip_q: the attention kernel does it itself)
//   k heads: the same with g_k, then rounded to bf16 into the cache at position p
//   v heads: rounded to bf16 into the cache at position p
// p = *d_len + (row % rows_per_seq); sequence = row / rows_per_seq.  Lane l owns elements 2l, 2l+1 and their
// rotation partners 2l+64, 2l+65 (half-split pairing).
__global__ void __launch_bounds__(128)
qk_norm_rope_append_kernel(float *__restrict__ qkv, int rows, int rows_per_seq, const bf16 *__restrict__ g_q,
                           const bf16 *__restrict__ g_k, float eps, const float *__restrict__ rope,
                           bf16 *__restrict__ kcache, bf16 *__restrict__ vcache, int nq, int nkv, int max_seq,
                           const int32_t *__restrict__ d_len, int skip_q, uint16_t *__restrict__ k16,
                           uint16_t *__restrict__ v16) {
    NNC_TRACE_SCOPE(2);
    pdl_wait();
    const int heads = nq + 2 * nkv;
    const int per_row = skip_q ? 2 * nkv : heads;   // heads of a row this launch works on (the last ones)
    const int unit = blockIdx.x * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (unit < rows * per_row) {
        const int row = unit / per_row, head = heads - per_row + unit % per_row;
        const int seq = row / rows_per_seq;
        const int pos = *d_len + (row % rows_per_seq);
        float *p = qkv + (size_t)row * heads * kHeadDim + (size_t)head * kHeadDim;
        float2 a = reinterpret_cast<float2 *>(p)[lane];        // elements 2l, 2l+1
        float2 b = reinterpret_cast<float2 *>(p + 64)[lane];   // elements 2l+64, 2l+65
        (void)NNC_BC(pos >= 0 && pos < max_seq, 201);          // the host checks the capacity before it launches
        if (pos < max_seq) {
            if (head < nq + nkv) {
                const bf16 *g = head < nq ? g_q : g_k;
                const float ss = warp_sum(a.x * a.x + a.y * a.y + b.x * b.x + b.y * b.y);
                const float inv = rsqrtf(ss * (1.f / kHeadDim) + eps);
                const uint32_t ga = reinterpret_cast<const uint32_t *>(g)[lane];
                const uint32_t gb = reinterpret_cast<const uint32_t *>(g + 64)[lane];
                a.x *= inv * bf16_lo(ga); a.y *= inv * bf16_hi(ga);
                b.x *= inv * bf16_lo(gb); b.y *= inv * bf16_hi(gb);
                const float4 cs = reinterpret_cast<const float4 *>(rope + (size_t)pos * kHeadDim)[lane];  // c0 s0 c1 s1
                const float2 ra = make_float2(a.x * cs.x - b.x * cs.y, a.y * cs.z - b.y * cs.w);
                const float2 rb = make_float2(b.x * cs.x + a.x * cs.y, b.y * cs.z + a.y * cs.w);
                a = ra; b = rb;
            }
            if (head < nq) {
                reinterpret_cast<float2 *>(p)[lane] = a;
                reinterpret_cast<float2 *>(p + 64)[lane] = b;
            } else {
                const bool is_k = head < nq + nkv;
                const int j = is_k ? head - nq : head - nq - nkv;
                const size_t off = (((size_t)seq * nkv + j) * max_seq + pos) * kHeadDim;
                bf16 *dst = (is_k ? kcache : vcache) + off;
                const uint32_t pa = pack_bf16x2(a.x, a.y), pb = pack_bf16x2(b.x, b.y);
                reinterpret_cast<uint32_t *>(dst)[lane] = pa;
                reinterpret_cast<uint32_t *>(dst + 64)[lane] = pb;
                uint16_t *d16 = is_k ? k16 : v16;
                if (d16) {   // fp16 image of the bf16 row just written (the same values wherever fp16 can hold them)
                    reinterpret_cast<uint32_t *>(d16 + off)[lane] = pack_f16x2_sat(bf16_lo(pa), bf16_hi(pa));
                    reinterpret_cast<uint32_t *>(d16 + off + 64)[lane] = pack_f16x2_sat(bf16_lo(pb), bf16_hi(pb));
                }
            }
        }
    }
    pdl_launch_dependents();
}

// out[i][:] = bf16(RMSNorm(x[first + i*step][:]; gain)); one block per output row.  If out_lo is given it
// receives the bf16 rounding residual (value - float(out)), so that out + out_lo carries 16 mantissa bits.
// F16: out receives fp16 values instead (one term, saturating at +-65504).
template <bool F16>
__global__ void __launch_bounds__(256)
rmsnorm_rows_kernel(const float *__restrict__ x, const bf16 *__restrict__ gain, bf16 *__restrict__ out,
                    bf16 *__restrict__ out_lo, int H, float eps, int first, int step) {
    __shared__ float red[8];
    NNC_TRACE_SCOPE(4);
    pdl_launch_dependents();   // the next kernel may set itself up while this one runs
    // rows of up to 4096 elements stay in registers between the two passes (4 x 16 bytes per thread, all requested
    // at once); longer rows are read again
    constexpr int kKeep = 4;
    const int n4 = H / 4;
    // the gains are weights: they are requested before the wait for the kernel that produces x
    uint2 gk[kKeep];
#pragma unroll
    for (int u = 0; u < kKeep; ++u) {
        const int i = threadIdx.x + 256 * u;
        gk[u] = (i < n4) ? reinterpret_cast<const uint2 *>(gain)[i] : make_uint2(0u, 0u);
    }
    pdl_wait();
    const float4 *src = reinterpret_cast<const float4 *>(x + (size_t)(first + blockIdx.x * step) * H);
    uint2 *dst = reinterpret_cast<uint2 *>(out + (size_t)blockIdx.x * H);
    float4 keep[kKeep];
    float ss = 0.f;
#pragma unroll
    for (int u = 0; u < kKeep; ++u) {
        const int i = threadIdx.x + 256 * u;
        keep[u] = (i < n4) ? src[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < kKeep; ++u) ss += keep[u].x * keep[u].x + keep[u].y * keep[u].y + keep[u].z * keep[u].z + keep[u].w * keep[u].w;
    for (int i = threadIdx.x + 256 * kKeep; i < n4; i += 256) {
        const float4 v = src[i];
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    const float inv = rsqrtf(tot / (float)H + eps);
    auto emit = [&](int i, const float4 &v, const uint2 g) {
        const float y0 = v.x * inv * bf16_lo(g.x), y1 = v.y * inv * bf16_hi(g.x);
        const float y2 = v.z * inv * bf16_lo(g.y), y3 = v.w * inv * bf16_hi(g.y);
        uint2 o;
        if (F16) {
            o.x = pack_f16x2_sat(y0, y1);
            o.y = pack_f16x2_sat(y2, y3);
            dst[i] = o;
            return;
        }
        o.x = pack_bf16x2(y0, y1);
        o.y = pack_bf16x2(y2, y3);
        dst[i] = o;
        if (out_lo) {
            uint2 r;
            r.x = pack_bf16x2(y0 - bf16_lo(o.x), y1 - bf16_hi(o.x));
            r.y = pack_bf16x2(y2 - bf16_lo(o.y), y3 - bf16_hi(o.y));
            reinterpret_cast<uint2 *>(out_lo + (size_t)blockIdx.x * H)[i] = r;
        }
    };
#pragma unroll
    for (int u = 0; u < kKeep; ++u) {
        const int i = threadIdx.x + 256 * u;
        if (i < n4) emit(i, keep[u], gk[u]);
    }
    for (int i = threadIdx.x + 256 * kKeep; i < n4; i += 256) emit(i, src[i], reinterpret_cast<const uint2 *>(gain)[i]);
}

// dst[h][pos][:] = fp16(src[h][pos][:]) for pos < n_pos; 16 bytes (8 elements) per thread
__global__ void kv_rows_to_f16_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, int heads, int max_seq, int n_pos) {
    pdl_wait();
    const size_t per_head = (size_t)n_pos * (kHeadDim / 8), total = per_head * heads;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t h = i / per_head, r = i % per_head;
        const size_t at = h * (size_t)max_seq * (kHeadDim / 8) + r;
        const uint4 v = src[at];
        dst[at] = make_uint4(pack_f16x2_sat(bf16_lo(v.x), bf16_hi(v.x)), pack_f16x2_sat(bf16_lo(v.y), bf16_hi(v.y)),
                             pack_f16x2_sat(bf16_lo(v.z), bf16_hi(v.z)), pack_f16x2_sat(bf16_lo(v.w), bf16_hi(v.w)));
    }
    pdl_launch_dependents();
}

__global__ void copy_f32_kernel(const float *__restrict__ src, float *__restrict__ dst, size_t n) {
    pdl_wait();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = src[i];
    pdl_launch_dependents();
}

__global__ void add_len_kernel(int32_t *d_len, int delta) {
    NNC_TRACE_SCOPE(3);
    pdl_wait();
    if (threadIdx.x == 0) *d_len += delta;
}

}  // namespace

cudaError_t launch_embed(const LaunchCtx &lc, const bf16 *E, const int32_t *tokens, float *x, int rows, int H,
                         int vocab, float *tap) {
    return launch(lc, embed_kernel, dim3(rows), dim3(128), E, tokens, x, H, vocab, tap);
}

cudaError_t launch_qk_norm_rope_append(const LaunchCtx &lc, float *qkv, int rows, int rows_per_seq,
                                       const bf16 *g_q, const bf16 *g_k, float eps, const float *rope,
                                       bf16 *kcache_layer, bf16 *vcache_layer, int nq, int nkv, int max_seq,
                                       const int32_t *d_len, bool skip_q, void *k16, void *v16) {
    const long units = (long)rows * (skip_q ? 2 * nkv : nq + 2 * nkv);
    return launch(lc, qk_norm_rope_append_kernel, dim3((unsigned)((units + 3) / 4)), dim3(128), qkv, rows,
                  rows_per_seq, g_q, g_k, eps, rope, kcache_layer, vcache_layer, nq, nkv, max_seq, d_len, skip_q ? 1 : 0,
                  (uint16_t *)k16, (uint16_t *)v16);
}

cudaError_t launch_rmsnorm_rows(const LaunchCtx &lc, const float *x, const bf16 *gain, bf16 *out, bf16 *out_lo, int rows,
                                int H, float eps, int first, int step, bool out_f16) {
    if (out_f16) return launch(lc, rmsnorm_rows_kernel<true>, dim3(rows), dim3(256), x, gain, out, out_lo, H, eps, first, step);
    return launch(lc, rmsnorm_rows_kernel<false>, dim3(rows), dim3(256), x, gain, out, out_lo, H, eps, first, step);
}

cudaError_t launch_kv_rows_to_f16(const LaunchCtx &lc, const bf16 *src, void *dst, int heads, int max_seq, int n_pos) {
    if (n_pos <= 0) return cudaSuccess;
    size_t blocks = ((size_t)heads * n_pos * (kHeadDim / 8) + 255) / 256;
    if (blocks > 1184) blocks = 1184;
    return launch(lc, kv_rows_to_f16_kernel, dim3((unsigned)blocks), dim3(256), reinterpret_cast<const uint4 *>(src),
                  reinterpret_cast<uint4 *>(dst), heads, max_seq, n_pos);
}

cudaError_t launch_copy_f32(const LaunchCtx &lc, const float *src, float *dst, size_t n) {
    size_t blocks = (n + 255) / 256;
    if (blocks > 1184) blocks = 1184;
    return launch(lc, copy_f32_kernel, dim3((unsigned)blocks), dim3(256), src, dst, n);
}

cudaError_t launch_add_len(const LaunchCtx &lc, int32_t *d_len, int delta) {
    return launch(lc, add_len_kernel, dim3(1), dim3(32), d_len, delta);
}

}  // namespace nnc
