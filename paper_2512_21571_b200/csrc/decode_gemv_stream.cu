// Batch-1 decode GEMV, streaming form: y = W x for a bf16 matrix W[n_out][K] read exactly once from HBM.
//
// HBM-bound (1 FLOP per weight byte), so the kernel is built around bytes in flight, not arithmetic:
//   - one persistent CTA per SM: a producer warp and 8 consumer warps around a shared-memory ring.  The producer
//     keeps the ring full with cp.async.bulk copies (the 1-D form of TMA) of 8-32 KB each -- whole consecutive
//     rows, which are contiguous in the row-major matrix -- so ~100 KB per SM are outstanding without holding
//     registers, and each copy is large enough that the copy engine's request rate is not the limit;
//   - the matrix is cut into stages of `rps` rows; CTAs claim short runs of consecutive stages from a global
//     counter (first run fixed, later runs by atomic, claimed one run ahead), so there is no wave quantisation
//     and SMs that stream faster take more of the matrix;
//   - inside a stage `ksplit` warps share a row, each taking a contiguous K slice whose activations it holds in
//     registers (times the norm gain when the RMSNorm prologue is fused; the scalar 1/rms is applied to the
//     finished sums), so shared memory carries weights only;
//   - per-row partial sums meet in a small double-buffered shared array and are folded in fixed order every
//     ~64 rows (deterministic: no float atomics), where the epilogue runs: store, residual add, SwiGLU on
//     interleaved gate/up rows, or logits + arg-max candidates (the last CTA folds those; nobody waits);
//   - launched with programmatic stream serialization: dependents are released at once and the producer never
//     waits on the previous kernel (weights depend on nothing), so a CTA starts streaming the moment its SM is
//     free.  The ring takes more than half of an SM's shared memory on purpose: two of these CTAs can never share
//     an SM, so each kernel's 148 CTAs land one per SM (with smaller rings the block scheduler was seen to stack
//     two CTAs of one kernel on some SMs and leave others idle whenever the previous kernel still held space).
// Second weight precision (the paper evaluates two, Section 4.1): the same kernel streams FP8 E4M3 codes with one
// power-of-two scale per output row (half the bytes per step).  A 16-byte chunk then carries 16 weights; codes are
// widened pairwise (cvt e4m3x2 -> f16x2 -> fp32) and multiplied in fp32; the row scale is applied to the finished
// sum together with 1/rms.
// Every mbarrier wait is bounded; on expiry the CTA raises the status word and drains.
#include <cuda_fp16.h>
#include <stdio.h>
#include <stdlib.h>

#include "common.cuh"
#include "nnc_internal.h"

namespace nnc {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;   // + the producer warp
constexpr int kMaxStages = 12;
constexpr int kRingBytes = 192 * 1024;          // the most a ring may take (geometry: a stage is at most a quarter of it)
// What a ring actually takes: as many stages as fit in 152 KB (three at the largest stage size).  Measured on the 8B
// decode step: 192 KB rings 2.887 ms, 168 KB 2.82, 160 KB 2.82, 152 KB 2.809, 144 KB 2.809, two 48 KB stages 2.98 --
// beyond three stages depth buys nothing, while a CTA under the 164 KB carve-out step leaves 92 instead of 28 KB of L1 to
// the kernel that follows it on the SM (the flash-decode reads K/V through L1) and room for that kernel's CTAs beside
// it.  Still more than half an SM, so exactly one of these CTAs fits per SM.
constexpr int kRingTarget = 152 * 1024;
constexpr int kBlockRows = 64;                    // rows between two folds of the partial sums
constexpr uint32_t kSpinLimit = 1u << 22;         // try_wait attempts before a wait gives up (each may block ~us)

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

// dot product of J 16-byte weight chunks with the matching activations: 2 J independent FMA chains
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

// two E4M3 codes (low 16 bits of `pair`) -> two floats
__device__ __forceinline__ float2 e4m3x2_to_float2(uint32_t pair) {
    uint32_t h2;
    asm("{\n.reg .b16 lo, hi;\nmov.b32 {lo, hi}, %1;\ncvt.rn.f16x2.e4m3x2 %0, lo;\n}" : "=r"(h2) : "r"(pair));
    return __half22float2(*reinterpret_cast<const __half2 *>(&h2));
}

// the same for 16-byte chunks of 16 E4M3 codes: xr holds the 16 matching activations
template <int J>
__device__ __forceinline__ float dot_slice_fp8(const uint4 (&w)[J], const float (&xr)[J][16]) {
    float a[J][2];
#pragma unroll
    for (int i = 0; i < J; ++i) {
        const uint32_t q[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
        a[i][0] = 0.f; a[i][1] = 0.f;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float2 lo = e4m3x2_to_float2(q[k]), hi = e4m3x2_to_float2(q[k] >> 16);
            a[i][0] = fmaf(lo.x, xr[i][4 * k], a[i][0]);
            a[i][1] = fmaf(lo.y, xr[i][4 * k + 1], a[i][1]);
            a[i][0] = fmaf(hi.x, xr[i][4 * k + 2], a[i][0]);
            a[i][1] = fmaf(hi.y, xr[i][4 * k + 3], a[i][1]);
        }
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < J; ++i) s += a[i][0] + a[i][1];
    return s;
}

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }

__device__ __forceinline__ bool better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

struct StreamParams {
    const uint8_t *W;
    const float *wscale;   // FP8 weights: one scale per output row (null for bf16 weights)
    const float *x;
    float *y;
    const bf16 *gain;
    float eps;
    int n_out, K;
    int ksplit;    // consumer warps per row (1, 2, 4, 8)
    int kw;        // columns of a warp's slice = K / ksplit (multiple of 8)
    int rps;       // rows per stage (a multiple of 8 / ksplit)
    int stages;    // ring depth
    int n_stages;  // stages in the whole matrix = ceil(n_out / rps)
    int pb;        // stages per fold block = kBlockRows / rps (at least 1)
    int claim;     // consecutive stages per work claim
    uint32_t *ctr; // {next run, CTAs done}: zero between launches; null = runs are dealt round-robin
    int *status;   // raised if a bounded wait runs out
    ArgmaxScratch am;
};

// J = 16-byte chunks per lane per row slice (kw <= J * 32 * CE elements).  WB = bytes per weight: 2 (bf16) or 1 (FP8
// E4M3 codes with a scale per row); CE = weights per 16-byte chunk.
template <int J, int MODE, bool NORM, int WB>
__global__ void __launch_bounds__(kThreads, 1) gemv_stream_kernel(const StreamParams p) {
    constexpr int CE = 16 / WB;
    NNC_TRACE_SCOPE(10 + MODE + 100 * (p.K / 1024));
    extern __shared__ __align__(128) uint8_t ring[];
    __shared__ __align__(8) uint64_t full[kMaxStages], empty[kMaxStages];
    __shared__ float part[2][kBlockRows][kConsumerWarps];
    __shared__ int slot_row[kMaxStages];        // first row of the stage held by each ring slot (-1: end of work)
    __shared__ int blk_row[2][kBlockRows];      // first row of each stage of the current fold block
    __shared__ float ssq[kConsumerWarps];       // sum of squares of each warp's activation slice
    __shared__ float red[kConsumerWarps];
    __shared__ int red_i[kConsumerWarps];
    __shared__ bool is_last;
    __shared__ int abort_s;                     // a consumer warp's wait ran out: every warp leaves at the next fold

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages;
    const uint32_t row_bytes = (uint32_t)p.K * (uint32_t)WB;
    const uint32_t stage_bytes = (uint32_t)p.rps * row_bytes;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < S; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&empty[s])), "r"(kConsumerWarps));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_launch_dependents();

    if (warp == kConsumerWarps) {
        // ---------------- producer: streams stages into the ring; never waits on the previous kernel ----------------
        // Work is claimed in runs of `claim` consecutive stages.  Each CTA starts with a fixed share that fills its ring
        // (runs i, i + grid, ...); later runs come from a global counter, so SMs that stream faster (they do differ
        // by ~15 %) simply take more.
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            const int n_runs = (p.n_stages + p.claim - 1) / p.claim;
            const int n_static = (S + p.claim - 1) / p.claim;
            const int grid = (int)gridDim.x;
            // run number of this CTA's k-th claim; claims are issued three runs ahead of the copies
            auto claim_id = [&](int k) {
                return (k < n_static || !p.ctr) ? (int)blockIdx.x + k * grid : grid * n_static + (int)atomicAdd(p.ctr, 1u);
            };
            int r0 = claim_id(0), r1 = claim_id(1), r2 = claim_id(2);
            for (int k = 3; r0 < n_runs && ok; ++k) {
                const int r3 = claim_id(k);
                const int s_end = min((r0 + 1) * p.claim, p.n_stages);
                for (int s = r0 * p.claim; s < s_end; ++s) {
                    if (!mbar_wait_bounded(smem_u32(&empty[stage]), phase ^ 1u)) { ok = false; break; }
                    const int row0 = s * p.rps;
                    const int rows = min(p.rps, p.n_out - row0);
                    slot_row[stage] = row0;
                    // a stage lies inside the matrix and inside its ring slot (checked build; a miss skips the copy and
                    // the consumers' bounded wait reports it)
                    if (NNC_BC(row0 >= 0 && rows > 0 && row0 + rows <= p.n_out && (uint32_t)rows * row_bytes <= stage_bytes &&
                               (uint32_t)(stage + 1) * stage_bytes <= (uint32_t)kRingBytes, 1001))
                        bulk_load(smem_u32(ring) + (uint32_t)stage * stage_bytes, p.W + (size_t)row0 * row_bytes,
                                  (uint32_t)rows * row_bytes, smem_u32(&full[stage]));
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                r0 = r1; r1 = r2; r2 = r3;
            }
            if (ok && mbar_wait_bounded(smem_u32(&empty[stage]), phase ^ 1u)) {
                slot_row[stage] = -1;   // end of work for this CTA
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&full[stage])) : "memory");
            } else if (p.status) {
                atomicExch(p.status, 17);
            }
            // the CTA that stops claiming last puts the counters back to zero for the next launch of this call site
            if (p.ctr && atomicAdd(p.ctr + 1, 1u) == gridDim.x - 1) { p.ctr[0] = 0u; p.ctr[1] = 0u; }
        }
        return;
    }

    // ---------------- consumers ----------------
    const int ksplit = p.ksplit, gpi = kConsumerWarps / ksplit;
    const int ks = warp % ksplit, gi = warp / ksplit;
    const int rw = p.rps / gpi;   // rows this warp owns in each stage: gi, gi + gpi, ...
    // gains are weights: fetch them before waiting on the kernel that produces x
    uint4 gr[NORM ? J : 1][CE / 8];
    if (NORM) {
#pragma unroll
        for (int i = 0; i < J; ++i) {
            const int c = lane + 32 * i;
#pragma unroll
            for (int h = 0; h < CE / 8; ++h)
                gr[i][h] = (c * CE < p.kw) ? *reinterpret_cast<const uint4 *>(p.gain + (size_t)ks * p.kw + (size_t)c * CE + 8 * h)
                                           : make_uint4(0, 0, 0, 0);
        }
    }
    pdl_wait();
    NNC_TRACE_MARK();

    // this warp's activation slice, in registers.  With the norm prologue it holds x * gain; the scalar
    // 1/rms(x) is applied to the finished row sums at the fold, so nothing waits for the sum of squares.
    float xr[J][CE];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < J; ++i) {
        const int c = lane + 32 * i;
        if (c * CE < p.kw) {
            const float4 *xp = reinterpret_cast<const float4 *>(p.x + (size_t)ks * p.kw + (size_t)c * CE);
#pragma unroll
            for (int q = 0; q < CE / 4; ++q) {
                const float4 a = xp[q];
                xr[i][4 * q] = a.x; xr[i][4 * q + 1] = a.y; xr[i][4 * q + 2] = a.z; xr[i][4 * q + 3] = a.w;
            }
        } else {
#pragma unroll
            for (int e = 0; e < CE; ++e) xr[i][e] = 0.f;
        }
        if (NORM) {
#pragma unroll
            for (int e = 0; e < CE; ++e) ss = fmaf(xr[i][e], xr[i][e], ss);
#pragma unroll
            for (int h = 0; h < CE / 8; ++h) {
                const uint4 g = gr[i][h];
                xr[i][8 * h + 0] *= bf16_lo(g.x); xr[i][8 * h + 1] *= bf16_hi(g.x);
                xr[i][8 * h + 2] *= bf16_lo(g.y); xr[i][8 * h + 3] *= bf16_hi(g.y);
                xr[i][8 * h + 4] *= bf16_lo(g.z); xr[i][8 * h + 5] *= bf16_hi(g.z);
                xr[i][8 * h + 6] *= bf16_lo(g.w); xr[i][8 * h + 7] *= bf16_hi(g.w);
            }
        }
    }
    if (NORM) {
        ss = warp_sum(ss);
        if (lane == 0) ssq[warp] = ss;   // read after the first consumer_sync below
    }

    float best_v = -INFINITY;
    int best_i = 0x7fffffff;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true, done = false;
    float inv = 1.f;
    const uint32_t slice_off = (uint32_t)ks * (uint32_t)p.kw * (uint32_t)WB;
    const int t = threadIdx.x;
    const int fold_unit = (MODE == kGemvSwiglu) ? (p.rps >> 1) : p.rps;   // outputs per stage
    const int tj = t / fold_unit, tr = t % fold_unit;                      // this thread's (stage in block, output in stage)

    for (int blk = 0; !done; ++blk) {
        const int buf = blk & 1;
        int nb = 0;
        for (int j = 0; j < p.pb; ++j) {
            if (!mbar_wait_bounded(smem_u32(&full[stage]), phase)) {
                // give up for the whole CTA: the flag is read by every warp after the barrier below, so all of them
                // leave the loop in the same iteration and no later barrier waits for a warp that has gone
                ok = false;
                *(volatile int *)&abort_s = 1;
                if (lane == 0 && p.status) atomicExch(p.status, 16);
                break;
            }
            const int row0 = slot_row[stage];
            if (row0 < 0) { done = true; break; }
            if (t == 0) blk_row[buf][j] = row0;
            const uint32_t sbase = smem_u32(ring) + (uint32_t)stage * stage_bytes + slice_off;
            // rows of this stage owned by the warp, two at a time (independent load / FMA streams, one joint reduction)
            for (int m = 0; m < rw; m += 2) {
                const int r_in_stage = gi + gpi * m;
                if (row0 + r_in_stage >= p.n_out) break;   // ragged last stage (warp-uniform)
                const bool two = (m + 1 < rw) && (row0 + r_in_stage + gpi < p.n_out);
                const uint32_t rbase0 = sbase + (uint32_t)r_in_stage * row_bytes;
                const uint32_t rbase1 = two ? rbase0 + (uint32_t)gpi * row_bytes : rbase0;
                uint4 w0[J], w1[J];
#pragma unroll
                for (int i = 0; i < J; ++i) {
                    const int c = lane + 32 * i;
                    w0[i] = make_uint4(0, 0, 0, 0);
                    w1[i] = make_uint4(0, 0, 0, 0);
                    if (c * CE < p.kw) {
                        w0[i] = lds128(rbase0 + (uint32_t)c * 16u);
                        w1[i] = lds128(rbase1 + (uint32_t)c * 16u);
                    }
                }
                float s0, s1;
                if constexpr (WB == 2) { s0 = dot_slice<J>(w0, xr); s1 = dot_slice<J>(w1, xr); }
                else { s0 = dot_slice_fp8<J>(w0, xr); s1 = dot_slice_fp8<J>(w1, xr); }
                // joint reduction: lanes 0-15 end up with row 0, lanes 16-31 with row 1
                const bool upper = (lane & 16) != 0;
                float keep = upper ? s1 : s0;
                keep += __shfl_xor_sync(0xffffffffu, upper ? s0 : s1, 16);
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) keep += __shfl_xor_sync(0xffffffffu, keep, o);
                const int r_in_block = j * p.rps + r_in_stage;
                if (lane == 0) part[buf][r_in_block][ks] = keep;
                if (lane == 16 && two) part[buf][r_in_block + gpi][ks] = keep;
            }
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&empty[stage])) : "memory");
            if (++stage == S) { stage = 0; phase ^= 1u; }
            ++nb;
        }
        consumer_sync();
        if (*(volatile int *)&abort_s) { ok = false; break; }
        if (NORM && blk == 0) {
            float tot = 0.f;
            for (int k = 0; k < ksplit; ++k) tot += ssq[k];   // warps 0 .. ksplit-1 hold the ksplit distinct slices
            inv = rsqrtf(tot / (float)p.K + p.eps);
        }
        // ---- fold the ksplit partial sums of each row in fixed order; epilogue ----
        if (tj < nb) {
            const int row0 = blk_row[buf][tj];
            if (MODE == kGemvSwiglu) {
                const int r = tj * p.rps + 2 * tr;
                if (row0 + 2 * tr + 1 < p.n_out) {
                    float g = 0.f, u = 0.f;
                    for (int k = 0; k < ksplit; ++k) { g += part[buf][r][k]; u += part[buf][r + 1][k]; }
                    g *= inv; u *= inv;
                    if (WB == 1) { g *= p.wscale[row0 + 2 * tr]; u *= p.wscale[row0 + 2 * tr + 1]; }
                    p.y[(row0 >> 1) + tr] = g / (1.f + __expf(-g)) * u;
                }
            } else if (row0 + tr < p.n_out) {
                float v = 0.f;
                for (int k = 0; k < ksplit; ++k) v += part[buf][tj * p.rps + tr][k];
                v *= inv;
                const int row = row0 + tr;
                if (WB == 1) v *= p.wscale[row];
                // residual: each element is touched by exactly one thread of one CTA per launch, so a reduction
                // without return value gives the same sum as load-add-store and exposes no load latency
                if (MODE == kGemvResidual) atomicAdd(p.y + row, v);
                else p.y[row] = v;
                if (MODE == kGemvLogits && better(v, row, best_v, best_i)) { best_v = v; best_i = row; }
            }
        }
    }

    if (MODE == kGemvLogits && p.am.out != nullptr) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best_v, o);
            const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
            if (better(ov, oi, best_v, best_i)) { best_v = ov; best_i = oi; }
        }
        if (lane == 0) { red[warp] = best_v; red_i[warp] = best_i; }
        consumer_sync();
        if (threadIdx.x == 0) {
            for (int w = 1; w < kConsumerWarps; ++w)
                if (better(red[w], red_i[w], best_v, best_i)) { best_v = red[w]; best_i = red_i[w]; }
            p.am.part_val[blockIdx.x] = best_v;
            p.am.part_idx[blockIdx.x] = best_i;
            __threadfence();
            const unsigned tk = atomicAdd(p.am.ticket, 1u);
            is_last = (tk == gridDim.x - 1);
        }
        consumer_sync();
        if (is_last) {  // the CTA that arrives last folds every CTA's candidate; nobody waits
            __threadfence();
            float bv = -INFINITY;
            int bi = 0x7fffffff;
            for (int b = threadIdx.x; b < (int)gridDim.x; b += kConsumerThreads) {
                const float v = ((volatile float *)p.am.part_val)[b];
                const int i = ((volatile int *)p.am.part_idx)[b];
                if (better(v, i, bv, bi)) { bv = v; bi = i; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
            }
            consumer_sync();
            if (lane == 0) { red[warp] = bv; red_i[warp] = bi; }
            consumer_sync();
            if (threadIdx.x == 0) {
                for (int w = 1; w < kConsumerWarps; ++w)
                    if (better(red[w], red_i[w], bv, bi)) { bv = red[w]; bi = red_i[w]; }
                *p.am.out = bi == 0x7fffffff ? 0 : bi;
                *p.am.ticket = 0u;
            }
        }
    }
    if (!ok) {
        // a copy never signalled: give whatever is still in flight time to land before shared memory is released
        for (int s = 0; s < 64; ++s) __nanosleep(1000);
    }
}

template <int J, int MODE, bool NORM, int WB>
cudaError_t launch_j(const LaunchCtx &lc, const StreamParams &p, int grid, size_t smem) {
    auto kern = gemv_stream_kernel<J, MODE, NORM, WB>;
    static unsigned long long attr_done = 0;   // per instantiation, one bit per device
    if (cudaError_t e = ensure_dynamic_smem(kern, kRingBytes, &attr_done); e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = lc.stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = lc.pdl ? 1 : 0;
    if (lc.launches) ++*lc.launches;
    return cudaLaunchKernelEx(&cfg, kern, p);
}

template <int MODE, bool NORM>
cudaError_t launch_mode(const LaunchCtx &lc, const StreamParams &p, int J, int grid, size_t smem, int wb) {
    if (wb == 1) {   // FP8: a chunk carries 16 weights, so half as many chunks cover a slice
        switch (J) {
            case 1: return launch_j<1, MODE, NORM, 1>(lc, p, grid, smem);
            case 2: return launch_j<2, MODE, NORM, 1>(lc, p, grid, smem);
            case 3: return launch_j<3, MODE, NORM, 1>(lc, p, grid, smem);
            case 4: return launch_j<4, MODE, NORM, 1>(lc, p, grid, smem);
        }
        return cudaErrorInvalidValue;
    }
    switch (J) {
        case 1: return launch_j<1, MODE, NORM, 2>(lc, p, grid, smem);
        case 2: return launch_j<2, MODE, NORM, 2>(lc, p, grid, smem);
        case 3: return launch_j<3, MODE, NORM, 2>(lc, p, grid, smem);
        case 4: return launch_j<4, MODE, NORM, 2>(lc, p, grid, smem);
        case 5: case 6: return launch_j<6, MODE, NORM, 2>(lc, p, grid, smem);
        case 7: case 8: return launch_j<8, MODE, NORM, 2>(lc, p, grid, smem);
    }
    return cudaErrorInvalidValue;
}

// Stage geometry for a shape: consumer warps per row, rows per stage.  Measured preferences: stages of 24-52 KB
// (each is one bulk copy; the per-stage handshake amortises and the copy engine's request rate never binds),
// an even number of rows per warp per stage (rows are processed in pairs), K slices of 2 KB or more, an even row
// count per stage when rows pair up as gate/up, and then the best balance over the SMs.
bool pick_geometry(int n_out, int K, int sm_count, bool pairs, int wb, int *ksplit_out, int *rps_out) {
    double best = -1.0;
#ifdef NNC_TUNING
    if (const char *g = getenv("NNC_GEMV_GEOM")) {   // "ksplit,rps": tuning builds only
        if (sscanf(g, "%d,%d", ksplit_out, rps_out) == 2) return true;
    }
#endif
    const int row_bytes = K * wb;
    const int ce = 16 / wb;                      // weights per 16-byte chunk
    const int max_chunks = wb == 2 ? 8 : 4;      // chunks per lane the kernel is instantiated for
    for (int ks = 8; ks >= 1; ks >>= 1) {
        if (K % (ce * ks)) continue;
        const int kw = K / ks;
        if ((kw + 32 * ce - 1) / (32 * ce) > max_chunks) continue;
        if (kw * wb < 512 && ks > 1) continue;
        const int gpi = kConsumerWarps / ks;
        for (int rps = gpi; rps <= kBlockRows; rps += gpi) {
            if (pairs && (rps & 1)) continue;
            const long bytes = (long)rps * row_bytes;
            if (bytes > kRingBytes / 4) break;
            const int rw = rps / gpi;
            if (rw > 8) break;
            const int n_stages = (n_out + rps - 1) / rps;
            const int grid = n_stages < sm_count ? n_stages : sm_count;
            const int per = (n_stages + grid - 1) / grid;
            double score = (double)n_stages / ((double)per * grid);
            if (rw & 1) score *= 0.85;
            if (bytes < 8192) score *= 0.80;
            else if (bytes < 16384) score *= 0.90;
            else if (bytes < 24576) score *= 0.95;
            if (kw * wb < 1024) score *= 0.90;
            else if (kw * wb < 2048) score *= 0.93;
            if (score > best) { best = score; *ksplit_out = ks; *rps_out = rps; }
        }
    }
    return best > 0.0;
}

}  // namespace

bool gemv_stream_supported(int n_out, int n_in, int mode, int wb) {
    int ks, rps;
    if (n_out < 1 || n_in % (16 / wb) || n_in < 64 || (mode == kGemvSwiglu && n_out % 2)) return false;
    return pick_geometry(n_out, n_in, 148, mode == kGemvSwiglu, wb, &ks, &rps);
}

cudaError_t launch_gemv_stream(const LaunchCtx &lc, const void *W, const float *wscale, int wb, const float *x, float *y,
                               int n_out, int n_in, const bf16 *gain, float eps, int mode, const ArgmaxScratch *am,
                               uint32_t *ctr) {
    if ((wb != 1 && wb != 2) || (wb == 1 && !wscale)) return cudaErrorInvalidValue;
    if (!gemv_stream_supported(n_out, n_in, mode, wb)) return cudaErrorInvalidValue;
    StreamParams p;
    if (!pick_geometry(n_out, n_in, lc.sm_count, mode == kGemvSwiglu, wb, &p.ksplit, &p.rps)) return cudaErrorInvalidValue;
    p.W = reinterpret_cast<const uint8_t *>(W);
    p.wscale = wscale;
    p.x = x; p.y = y; p.gain = gain; p.eps = eps; p.n_out = n_out; p.K = n_in;
    p.kw = n_in / p.ksplit;
    const int stage_bytes = p.rps * n_in * wb;
    int S = kRingTarget / stage_bytes;
    if (S > kMaxStages) S = kMaxStages;
    if (S < 2) return cudaErrorInvalidValue;
    p.stages = S;
    p.n_stages = (n_out + p.rps - 1) / p.rps;
    p.pb = kBlockRows / p.rps;
    if (p.pb < 1) p.pb = 1;
    p.status = lc.status;
    p.am = am ? *am : ArgmaxScratch{nullptr, nullptr, nullptr, nullptr};
    // claims of ~64 KB keep each CTA's reads in longer sequential pieces (measured: better on large matrices);
    // matrices with few stages per SM claim stage by stage so that the tail stays short
    p.claim = (stage_bytes >= 49152 || p.n_stages < 16 * lc.sm_count) ? 1 : (65536 + stage_bytes - 1) / stage_bytes;
    if (stage_bytes < 16384 && p.claim == 1) p.claim = (32768 + stage_bytes - 1) / stage_bytes;
    const int n_runs = (p.n_stages + p.claim - 1) / p.claim;
    int grid = n_runs < lc.sm_count ? n_runs : lc.sm_count;
    // With no more runs than CTAs every CTA takes exactly one run: dynamic claims buy nothing there, and leaving the
    // shared counters alone means many such small launches may be in flight at once without meeting on them.
    p.ctr = n_runs > lc.sm_count ? ctr : nullptr;
    if (mode == kGemvLogits && grid > kArgmaxMaxBlocks) grid = kArgmaxMaxBlocks;
    const size_t smem = (size_t)S * stage_bytes;
    const int ce32 = 32 * (16 / wb);
    const int J = (p.kw + ce32 - 1) / ce32;
    const bool norm = gain != nullptr;
    switch (mode) {
        case kGemvStore:
            return norm ? launch_mode<kGemvStore, true>(lc, p, J, grid, smem, wb) : launch_mode<kGemvStore, false>(lc, p, J, grid, smem, wb);
        case kGemvResidual:
            return norm ? launch_mode<kGemvResidual, true>(lc, p, J, grid, smem, wb) : launch_mode<kGemvResidual, false>(lc, p, J, grid, smem, wb);
        case kGemvSwiglu:
            return norm ? launch_mode<kGemvSwiglu, true>(lc, p, J, grid, smem, wb) : launch_mode<kGemvSwiglu, false>(lc, p, J, grid, smem, wb);
        case kGemvLogits:
            return norm ? launch_mode<kGemvLogits, true>(lc, p, J, grid, smem, wb) : launch_mode<kGemvLogits, false>(lc, p, J, grid, smem, wb);
    }
    return cudaErrorInvalidValue;
}

}  // namespace nnc
