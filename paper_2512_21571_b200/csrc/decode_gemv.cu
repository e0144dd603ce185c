// Batch-1 decode GEMV family: y = W x for a bf16 matrix W[n_out][n_in] streamed once from HBM.
//
// HBM-bound (1 FLOP per weight byte): the kernel is organised around keeping many 16-byte loads in flight.
// One warp owns ROWS consecutive rows at a time and walks K in steps of 32 lanes x 16 bytes; U x ROWS = 8
// independent loads are issued per lane before any is consumed.  The activation vector (fp32) is staged once
// per CTA in shared memory, optionally RMS-normalised on the way (fused norm prologue: every CTA recomputes
// the sum of squares from the L2-resident vector, which costs n_in*4 bytes of L2 traffic per CTA).  Reduction
// is a warp-shuffle tree in fp32.  Epilogues: store, residual add, SwiGLU on interleaved gate/up rows, and
// logits + arg-max partials with a last-block-done final reduction (no spinning).
#include "common.cuh"
#include "nnc_internal.h"

namespace nnc {

namespace {

constexpr int kGemvThreads = 256;
constexpr int kGemvWarps = kGemvThreads / 32;

__device__ __forceinline__ float dot8(const uint4 &w, const float4 &a, const float4 &b, float acc) {
    acc = fmaf(bf16_lo(w.x), a.x, acc);
    acc = fmaf(bf16_hi(w.x), a.y, acc);
    acc = fmaf(bf16_lo(w.y), a.z, acc);
    acc = fmaf(bf16_hi(w.y), a.w, acc);
    acc = fmaf(bf16_lo(w.z), b.x, acc);
    acc = fmaf(bf16_hi(w.z), b.y, acc);
    acc = fmaf(bf16_lo(w.w), b.z, acc);
    acc = fmaf(bf16_hi(w.w), b.w, acc);
    return acc;
}

// is (v, i) a better arg-max candidate than (bv, bi)?  lowest index wins ties; NaN never wins
__device__ __forceinline__ bool better(float v, int i, float bv, int bi) {
    return v > bv || (v == bv && i < bi);
}

template <int ROWS, int MODE, bool NORM>
__global__ void __launch_bounds__(kGemvThreads)
gemv_kernel(const uint4 *__restrict__ W, const float *__restrict__ x, float *__restrict__ y, int n_out, int n_in,
            const bf16 *__restrict__ gain, float eps, ArgmaxScratch am) {
    NNC_TRACE_SCOPE(20 + MODE);
    extern __shared__ float4 xs[];  // two planes of n_in/8 float4: plane h holds elements 8c+4h .. 8c+4h+3 of chunk c
    __shared__ float red[kGemvWarps];
    __shared__ int red_i[kGemvWarps];
    __shared__ bool is_last;

    constexpr int U = 8 / ROWS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nchunk = n_in >> 3;
    const int n_groups = n_out / ROWS;
    const int gstride = gridDim.x * kGemvWarps;
    int group = blockIdx.x * kGemvWarps + warp;

    // Weights depend on no earlier kernel: pull the first lines of this warp's first rows toward L2 before
    // waiting on the producer of x.
    if (group < n_groups) {
        const uint4 *wrow = W + (size_t)group * ROWS * nchunk;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            int c = u * 32 + lane;
            if (c < nchunk && (lane & 7) == 0) {
#pragma unroll
                for (int r = 0; r < ROWS; ++r)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(wrow + (size_t)r * nchunk + c));
            }
        }
    }
    pdl_wait();

    // ---- stage x (optionally RMS-normalised) ----
    const int n4 = n_in >> 2;
    float ss = 0.f;
    for (int t = threadIdx.x; t < n4; t += kGemvThreads) {
        float4 v = reinterpret_cast<const float4 *>(x)[t];
        if (NORM) ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        xs[(t & 1) * nchunk + (t >> 1)] = v;
    }
    if (NORM) {
        ss = warp_sum(ss);
        if (lane == 0) red[warp] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < kGemvWarps; ++w) tot += red[w];
        const float inv = rsqrtf(tot / (float)n_in + eps);
        for (int t = threadIdx.x; t < n4; t += kGemvThreads) {
            float4 v = xs[(t & 1) * nchunk + (t >> 1)];
            uint2 g = reinterpret_cast<const uint2 *>(gain)[t];
            v.x *= inv * bf16_lo(g.x);
            v.y *= inv * bf16_hi(g.x);
            v.z *= inv * bf16_lo(g.y);
            v.w *= inv * bf16_hi(g.y);
            xs[(t & 1) * nchunk + (t >> 1)] = v;
        }
    }
    __syncthreads();

    float best_v = -INFINITY;
    int best_i = 0x7fffffff;

    for (; group < n_groups; group += gstride) {
        const uint4 *wrow = W + (size_t)group * ROWS * nchunk;
        float acc[ROWS];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) acc[r] = 0.f;

        for (int c0 = 0; c0 < nchunk; c0 += 32 * U) {
            uint4 w[U][ROWS];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int c = c0 + u * 32 + lane;
#pragma unroll
                for (int r = 0; r < ROWS; ++r)
                    w[u][r] = (c < nchunk) ? ldg_stream(wrow + (size_t)r * nchunk + c) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int c = c0 + u * 32 + lane;
                if (c < nchunk) {
                    const float4 a = xs[c], b = xs[nchunk + c];
#pragma unroll
                    for (int r = 0; r < ROWS; ++r) acc[r] = dot8(w[u][r], a, b, acc[r]);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) acc[r] = warp_sum(acc[r]);

        if (lane == 0) {
            const int row0 = group * ROWS;
            if (MODE == kGemvStore) {
#pragma unroll
                for (int r = 0; r < ROWS; ++r) y[row0 + r] = acc[r];
            } else if (MODE == kGemvResidual) {
#pragma unroll
                for (int r = 0; r < ROWS; ++r) y[row0 + r] += acc[r];
            } else if (MODE == kGemvSwiglu) {
#pragma unroll
                for (int r = 0; r < ROWS; r += 2) {
                    const float g = acc[r], u = acc[r + 1 < ROWS ? r + 1 : r];
                    y[(row0 + r) >> 1] = g / (1.f + __expf(-g)) * u;
                }
            } else {  // logits + running arg-max
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    y[row0 + r] = acc[r];
                    if (better(acc[r], row0 + r, best_v, best_i)) { best_v = acc[r]; best_i = row0 + r; }
                }
            }
        }
    }
    pdl_launch_dependents();

    if (MODE == kGemvLogits && am.out != nullptr) {
        if (lane == 0) { red[warp] = best_v; red_i[warp] = best_i; }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < kGemvWarps; ++w)
                if (better(red[w], red_i[w], best_v, best_i)) { best_v = red[w]; best_i = red_i[w]; }
            am.part_val[blockIdx.x] = best_v;
            am.part_idx[blockIdx.x] = best_i;
            __threadfence();
            const unsigned t = atomicAdd(am.ticket, 1u);
            is_last = (t == gridDim.x - 1);
        }
        __syncthreads();
        if (is_last) {  // the block that arrives last folds every block's candidate; nobody waits
            __threadfence();
            float bv = -INFINITY;
            int bi = 0x7fffffff;
            for (int b = threadIdx.x; b < (int)gridDim.x; b += kGemvThreads) {
                const float v = ((volatile float *)am.part_val)[b];
                const int i = ((volatile int *)am.part_idx)[b];
                if (better(v, i, bv, bi)) { bv = v; bi = i; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
            }
            __syncthreads();
            if (lane == 0) { red[warp] = bv; red_i[warp] = bi; }
            __syncthreads();
            if (threadIdx.x == 0) {
                for (int w = 1; w < kGemvWarps; ++w)
                    if (better(red[w], red_i[w], bv, bi)) { bv = red[w]; bi = red_i[w]; }
                *am.out = bi == 0x7fffffff ? 0 : bi;
                *am.ticket = 0u;
            }
        }
    }
}

template <int ROWS, int MODE, bool NORM>
cudaError_t launch_one(const LaunchCtx &lc, const bf16 *W, const float *x, float *y, int n_out, int n_in,
                       const bf16 *gain, float eps, const ArgmaxScratch &am, int ctas_per_sm) {
    auto kern = gemv_kernel<ROWS, MODE, NORM>;
    const size_t smem = (size_t)n_in * sizeof(float);
    static unsigned long long attr_done = 0;   // per instantiation, one bit per device
    if (cudaError_t e = ensure_dynamic_smem(kern, 200 * 1024, &attr_done); e != cudaSuccess) return e;
    const int n_groups = n_out / ROWS;
    const int cap = lc.sm_count * ctas_per_sm;
    int blocks = (n_groups + kGemvWarps - 1) / kGemvWarps;
    if (blocks > cap) {  // balance: every warp gets the same number of row groups (within one)
        const int iters = (n_groups + cap * kGemvWarps - 1) / (cap * kGemvWarps);
        blocks = (n_groups + iters * kGemvWarps - 1) / (iters * kGemvWarps);
    }
    if (MODE == kGemvLogits && blocks > kArgmaxMaxBlocks) blocks = kArgmaxMaxBlocks;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(kGemvThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = lc.stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = lc.pdl ? 1 : 0;
    if (lc.launches) ++*lc.launches;
    return cudaLaunchKernelEx(&cfg, kern, reinterpret_cast<const uint4 *>(W), x, y, n_out, n_in, gain, eps, am);
}

template <int MODE, bool NORM>
cudaError_t launch_rows(const LaunchCtx &lc, const bf16 *W, const float *x, float *y, int n_out, int n_in,
                        const bf16 *gain, float eps, const ArgmaxScratch &am) {
    // smem per CTA is n_in*4 bytes: bound the CTAs per SM by that as well as by threads
    int ctas = 4;
    while (ctas > 1 && (size_t)ctas * n_in * 4 > 200 * 1024) --ctas;
    const int slots = lc.sm_count * ctas * kGemvWarps;
    // more rows per warp amortise the shared-memory reads of x; fewer rows give more warps work
    if (n_out % 4 == 0 && n_out / 4 >= slots) return launch_one<4, MODE, NORM>(lc, W, x, y, n_out, n_in, gain, eps, am, ctas);
    if (n_out % 2 == 0 && (n_out / 2 >= slots / 2 || MODE == kGemvSwiglu))
        return launch_one<2, MODE, NORM>(lc, W, x, y, n_out, n_in, gain, eps, am, ctas);
    if (MODE == kGemvSwiglu) return cudaErrorInvalidValue;
    return launch_one<(MODE == kGemvSwiglu ? 2 : 1), MODE, NORM>(lc, W, x, y, n_out, n_in, gain, eps, am, ctas);
}

}  // namespace

cudaError_t launch_gemv(const LaunchCtx &lc, const void *Wv, const float *wscale, const float *x, float *y, int n_out, int n_in,
                        const bf16 *gain, float eps, int mode, const ArgmaxScratch *am, uint32_t *ctr) {
    if (wscale)   // FP8 codes: the streaming form only
        return launch_gemv_stream(lc, Wv, wscale, 1, x, y, n_out, n_in, gain, eps, mode, am, ctr);
    const bf16 *W = reinterpret_cast<const bf16 *>(Wv);
    if (gemv_stream_supported(n_out, n_in, mode)) return launch_gemv_stream(lc, W, nullptr, 2, x, y, n_out, n_in, gain, eps, mode, am, ctr);
    if (n_in % 8 != 0 || n_in <= 0 || n_out <= 0 || (size_t)n_in * 4 > 200 * 1024) return cudaErrorInvalidValue;
    ArgmaxScratch a = am ? *am : ArgmaxScratch{nullptr, nullptr, nullptr, nullptr};
    const bool norm = gain != nullptr;
    switch (mode) {
        case kGemvStore:
            return norm ? launch_rows<kGemvStore, true>(lc, W, x, y, n_out, n_in, gain, eps, a)
                        : launch_rows<kGemvStore, false>(lc, W, x, y, n_out, n_in, gain, eps, a);
        case kGemvResidual:
            return norm ? launch_rows<kGemvResidual, true>(lc, W, x, y, n_out, n_in, gain, eps, a)
                        : launch_rows<kGemvResidual, false>(lc, W, x, y, n_out, n_in, gain, eps, a);
        case kGemvSwiglu:
            if (n_out % 2) return cudaErrorInvalidValue;
            return norm ? launch_rows<kGemvSwiglu, true>(lc, W, x, y, n_out, n_in, gain, eps, a)
                        : launch_rows<kGemvSwiglu, false>(lc, W, x, y, n_out, n_in, gain, eps, a);
        case kGemvLogits:
            return norm ? launch_rows<kGemvLogits, true>(lc, W, x, y, n_out, n_in, gain, eps, a)
                        : launch_rows<kGemvLogits, false>(lc, W, x, y, n_out, n_in, gain, eps, a);
    }
    return cudaErrorInvalidValue;
}

}  // namespace nnc
