// Building blocks of the whole-step decode kernel (decode_step_mega.cu): ring primitives, the consumer side of one
// streaming GEMV phase, and the grid-wide barrier between phases.  The arithmetic of a GEMV phase is the one of
// gemv_stream_kernel (same slices, same fold order), so both paths give the same bits.
#pragma once
#include "common.cuh"
#include "nnc_internal.h"

namespace nnc {
namespace mega {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;   // + the producer warp
constexpr int kMaxStages = 4;
constexpr int kBlockRows = 64;
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 w;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w) : "r"(addr));
    return w;
}

template <int J>
__device__ __forceinline__ float dot_slice(const uint4 (&w)[J], const float (&xr)[J][8]) {
    float a[J][2];
#pragma unroll
    for (int i = 0; i < J; ++i) {
        a[i][0] = bf16_lo(w[i].x) * xr[i][0];
        a[i][1] = bf16_hi(w[i].x) * xr[i][1];
        a[i][0] = fmaf(bf16_lo(w[i].y), xr[i][2], a[i][0]);
        a[i][1] = fmaf(bf16_hi(w[i].y), xr[i][3], a[i][1]);
        a[i][0] = fmaf(bf16_lo(w[i].z), xr[i][4], a[i][0]);
        a[i][1] = fmaf(bf16_hi(w[i].z), xr[i][5], a[i][1]);
        a[i][0] = fmaf(bf16_lo(w[i].w), xr[i][6], a[i][0]);
        a[i][1] = fmaf(bf16_hi(w[i].w), xr[i][7], a[i][1]);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < J; ++i) s += a[i][0] + a[i][1];
    return s;
}

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }
__device__ __forceinline__ bool better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

using Geom = GemvGeom;   // one matrix of the step: shape and slicing (as chosen for gemv_stream_kernel)

// Shared-memory state of the ring and of the folds.
struct RingSmem {
    __align__(8) uint64_t full[kMaxStages], empty[kMaxStages];
    float part[2][kBlockRows][kConsumerWarps];
    float ssq[kConsumerWarps];
    float red[kConsumerWarps];
    int red_i[kConsumerWarps];
    bool is_last;
};

// Position in the ring; producer and consumers each keep their own copy and advance it identically.
struct RingPos {
    int stage;
    uint32_t phase;
    __device__ __forceinline__ void advance(int S) { if (++stage == S) { stage = 0; phase ^= 1u; } }
};

// This CTA's contiguous share of a matrix's stages.
__device__ __forceinline__ void stage_range(const Geom &g, int &st0, int &n_st) {
    const int per = g.n_stages / gridDim.x, rem = g.n_stages % gridDim.x;
    st0 = blockIdx.x * per + min((int)blockIdx.x, rem);
    n_st = per + ((int)blockIdx.x < rem ? 1 : 0);
}

// Grid-wide barrier k (k = 0, 1, 2, ... in launch order).  Called by the consumer threads only.  Returns false if the
// wait ran out or another CTA gave up (abort word set).
//   words[0 .. 15]  arrival counters of 16 groups of CTAs (group = blockIdx % 16), monotonic over the launch
//   words[16]       arrival counter of the groups, monotonic
//   words[17]       release word: number of barriers completed
//   words[18]       abort word
// Arrivals are spread over 16 + 1 addresses (148 atomics on one address serialise to microseconds) and everybody
// polls a word that is written once per barrier.  Barrier k + 1 cannot receive an arrival before barrier k has
// released, so the counters need no reset: the last arriver is the one that completes a multiple of the group size.
constexpr int kBarGroups = 16;
constexpr int kBarWords = 32;
__device__ __forceinline__ bool grid_barrier(uint32_t *words, int k, int *status) {
    consumer_sync();
    __shared__ int bar_ok;
    if (threadIdx.x == 0) {
        int ok = 1;
        const int grp = blockIdx.x % kBarGroups;
        const unsigned n_grp = gridDim.x < kBarGroups ? gridDim.x : kBarGroups;
        const unsigned size = gridDim.x / kBarGroups + ((unsigned)grp < gridDim.x % kBarGroups ? 1u : 0u);
        __threadfence();
        if ((atomicAdd(words + grp, 1u) + 1u) % size == 0u) {
            __threadfence();
            if ((atomicAdd(words + 16, 1u) + 1u) % n_grp == 0u) {
                __threadfence();
                asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(words + 17), "r"((uint32_t)k + 1u) : "memory");
            }
        }
        uint32_t seen = 0;
        for (uint32_t spin = 0;; ++spin) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(words + 17) : "memory");
            if (seen >= (uint32_t)k + 1u) break;
            if ((spin & 255u) == 255u) {
                uint32_t ab;
                asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(ab) : "l"(words + 18) : "memory");
                if (ab || spin > (1u << 25)) {
                    ok = 0;
                    atomicExch(words + 18, 1u);
                    if (status) atomicExch(status, 32);
                    break;
                }
            }
        }
        __threadfence();
        bar_ok = ok;
    }
    consumer_sync();
    return bar_ok != 0;
}

// Consumer side of one GEMV phase: y (op)= W x for this CTA's stages, which the producer streams in the same order.
//   x_embed != null: the activation is the bf16 embedding row (first layer); CTA 0 also stores it as fp32 to x_out.
//   NORM: x * gain goes to registers, 1/rms(x) is applied at the fold.  Activations are read with L2 loads: they
//   were written by other SMs earlier in this same kernel, so L1 may not be trusted.
template <int J, int MODE, bool NORM>
__device__ __forceinline__ void gemv_phase(const Geom &g, const float *x, const bf16 *x_embed, float *x_out, float *y,
                                           const bf16 *gain, float eps, RingSmem &rs, uint32_t ring_base,
                                           uint32_t slot_bytes, int S, RingPos &pos, float &best_v, int &best_i,
                                           bool &ok, int *status) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ksplit = g.ksplit, gpi = kConsumerWarps / ksplit;
    const int ks = warp % ksplit, gi = warp / ksplit;
    const int rw = g.rps / gpi;
    const uint32_t row_bytes = (uint32_t)g.K * 2u;
    int st0, n_st;
    stage_range(g, st0, n_st);

    float xr[J][8];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < J; ++i) {
        const int c = lane + 32 * i;
        if (c * 8 < g.kw) {
            const size_t e0 = (size_t)ks * g.kw + (size_t)c * 8;
            if (x_embed) {
                const uint4 u = __ldcg(reinterpret_cast<const uint4 *>(x_embed + e0));
                xr[i][0] = bf16_lo(u.x); xr[i][1] = bf16_hi(u.x); xr[i][2] = bf16_lo(u.y); xr[i][3] = bf16_hi(u.y);
                xr[i][4] = bf16_lo(u.z); xr[i][5] = bf16_hi(u.z); xr[i][6] = bf16_lo(u.w); xr[i][7] = bf16_hi(u.w);
                if (blockIdx.x == 0 && gi == 0) {
                    *reinterpret_cast<float4 *>(x_out + e0) = make_float4(xr[i][0], xr[i][1], xr[i][2], xr[i][3]);
                    *reinterpret_cast<float4 *>(x_out + e0 + 4) = make_float4(xr[i][4], xr[i][5], xr[i][6], xr[i][7]);
                }
            } else {
                const float4 a = __ldcg(reinterpret_cast<const float4 *>(x + e0));
                const float4 b = __ldcg(reinterpret_cast<const float4 *>(x + e0 + 4));
                xr[i][0] = a.x; xr[i][1] = a.y; xr[i][2] = a.z; xr[i][3] = a.w;
                xr[i][4] = b.x; xr[i][5] = b.y; xr[i][6] = b.z; xr[i][7] = b.w;
            }
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) xr[i][e] = 0.f;
        }
        if (NORM) {
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(xr[i][e], xr[i][e], ss);
            if (c * 8 < g.kw) {
                const uint4 gg = *reinterpret_cast<const uint4 *>(gain + (size_t)ks * g.kw + (size_t)c * 8);
                xr[i][0] *= bf16_lo(gg.x); xr[i][1] *= bf16_hi(gg.x); xr[i][2] *= bf16_lo(gg.y); xr[i][3] *= bf16_hi(gg.y);
                xr[i][4] *= bf16_lo(gg.z); xr[i][5] *= bf16_hi(gg.z); xr[i][6] *= bf16_lo(gg.w); xr[i][7] *= bf16_hi(gg.w);
            }
        }
    }
    if (NORM) {
        ss = warp_sum(ss);
        if (lane == 0) rs.ssq[warp] = ss;   // read after the first consumer_sync below
    }
    float inv = 1.f;
    const uint32_t slice_off = (uint32_t)ks * (uint32_t)g.kw * 2u;
    const int pb = max(1, kBlockRows / g.rps);
    const int t = threadIdx.x;

    for (int b0 = 0, blk = 0; b0 < n_st; b0 += pb, ++blk) {
        const int nb = min(pb, n_st - b0);
        const int buf = blk & 1;
        const int block_row0 = (st0 + b0) * g.rps;
        const int rows_here = min(nb * g.rps, g.n_out - block_row0);
        for (int j = 0; j < nb; ++j) {
            if (ok && !mbar_wait_bounded(smem_u32(&rs.full[pos.stage]), pos.phase)) {
                ok = false;
                if (lane == 0 && status) atomicExch(status, 33);
            }
            const uint32_t sbase = ring_base + (uint32_t)pos.stage * slot_bytes + slice_off;
            for (int m = 0; m < rw && ok; m += 2) {
                const int r_in_stage = gi + gpi * m;
                const int r_in_block = j * g.rps + r_in_stage;
                if (block_row0 + r_in_block >= g.n_out) break;   // ragged last stage (warp-uniform)
                const bool two = (m + 1 < rw) && (block_row0 + r_in_block + gpi < g.n_out);
                const uint32_t rbase0 = sbase + (uint32_t)r_in_stage * row_bytes;
                const uint32_t rbase1 = two ? rbase0 + (uint32_t)gpi * row_bytes : rbase0;
                uint4 w0[J], w1[J];
#pragma unroll
                for (int i = 0; i < J; ++i) {
                    const int c = lane + 32 * i;
                    w0[i] = make_uint4(0, 0, 0, 0);
                    w1[i] = make_uint4(0, 0, 0, 0);
                    if (c * 8 < g.kw) {
                        w0[i] = lds128(rbase0 + (uint32_t)c * 16u);
                        w1[i] = lds128(rbase1 + (uint32_t)c * 16u);
                    }
                }
                const float s0 = dot_slice<J>(w0, xr), s1 = dot_slice<J>(w1, xr);
                const bool upper = (lane & 16) != 0;
                float keep = upper ? s1 : s0;
                keep += __shfl_xor_sync(0xffffffffu, upper ? s0 : s1, 16);
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) keep += __shfl_xor_sync(0xffffffffu, keep, o);
                if (lane == 0) rs.part[buf][r_in_block][ks] = keep;
                if (lane == 16 && two) rs.part[buf][r_in_block + gpi][ks] = keep;
            }
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&rs.empty[pos.stage])) : "memory");
            pos.advance(S);
        }
        consumer_sync();
        if (NORM && blk == 0) {
            float tot = 0.f;
            for (int k = 0; k < ksplit; ++k) tot += rs.ssq[k];
            inv = rsqrtf(tot / (float)g.K + eps);
        }
        if (MODE == kGemvSwiglu) {
            if (2 * t + 1 < rows_here) {
                float gt = 0.f, up = 0.f;
                for (int k = 0; k < ksplit; ++k) { gt += rs.part[buf][2 * t][k]; up += rs.part[buf][2 * t + 1][k]; }
                gt *= inv; up *= inv;
                y[(block_row0 >> 1) + t] = gt / (1.f + __expf(-gt)) * up;
            }
        } else if (t < rows_here) {
            float v = 0.f;
            for (int k = 0; k < ksplit; ++k) v += rs.part[buf][t][k];
            v *= inv;
            const int row = block_row0 + t;
            if (MODE == kGemvResidual) atomicAdd(y + row, v);   // one writer per element: same sum as load-add-store
            else y[row] = v;
            if (MODE == kGemvLogits && better(v, row, best_v, best_i)) { best_v = v; best_i = row; }
        }
    }
}

}  // namespace mega
}  // namespace nnc
