// The whole batch-1 decode step as ONE persistent kernel (cooperative launch, one CTA per SM).
//
// A decode step is a chain of small HBM-bound phases (per layer: QKV GEMV, flash-decode, O GEMV, gate/up GEMV, down
// GEMV; then the lm_head).  As separate kernels every link of that chain costs ~2-3 us of completion, release and
// prologue during which no weight bytes move -- a third of the step for the 0.6B shape.  Here:
//   - each CTA's producer warp streams the CTA's share of EVERY matrix of the step, in order, through one
//     shared-memory ring (cp.async.bulk, 48 KB slots).  It never looks at the phase structure, so while the
//     consumers of all CTAs meet at the barrier between two phases the ring is already filling with the next matrix;
//   - the 8 consumer warps run the phases: the GEMV phases are the arithmetic of gemv_stream_kernel (same slices,
//     same fold order: identical bits), the attention phase runs the flash-decode body on two 4-warp groups per CTA;
//   - phases are separated by a grid-wide barrier (arrive counter in global memory, bounded spin with back-off,
//     abort word shared by all CTAs, status word for the host).  Activations written in one phase are read with L2
//     loads in the next: L1 is not coherent across SMs inside one kernel.
// The kernel needs every CTA resident at once, hence the cooperative launch; if that is refused the library falls
// back to the kernel-per-phase path.
#include <stdio.h>

#include "attn_decode_body.cuh"
#include "decode_mega_parts.cuh"

namespace nnc {

using namespace mega;

namespace {

template <int G>
struct MegaSmem {
    RingSmem ring;
    AttnSmem<G> attn[2];
};

// ---- producer: all stages of all matrices of the step, in phase order ----
__device__ __forceinline__ bool stream_matrix(const Geom &g, const uint8_t *W, RingSmem &rs, uint32_t ring_base,
                                              uint32_t slot_bytes, int S, RingPos &pos) {
    int st0, n_st;
    stage_range(g, st0, n_st);
    const uint32_t row_bytes = (uint32_t)g.K * 2u;
    for (int s = 0; s < n_st; ++s) {
        if (!mbar_wait_bounded(smem_u32(&rs.empty[pos.stage]), pos.phase ^ 1u)) return false;
        const int row0 = (st0 + s) * g.rps;
        const int rows = min(g.rps, g.n_out - row0);
        bulk_load(ring_base + (uint32_t)pos.stage * slot_bytes, W + (size_t)row0 * row_bytes, (uint32_t)rows * row_bytes,
                  smem_u32(&rs.full[pos.stage]));
        pos.advance(S);
    }
    return true;
}

// J dispatch for one GEMV phase (J = 16-byte chunks per lane per row slice)
template <int MODE, bool NORM>
__device__ __forceinline__ void run_gemv(const Geom &g, const float *x, const bf16 *x_embed, float *x_out, float *y,
                                         const bf16 *gain, float eps, RingSmem &rs, uint32_t ring_base, uint32_t slot_bytes,
                                         int S, RingPos &pos, float &bv, int &bi, bool &ok, int *status) {
    switch (g.J) {
        case 1: gemv_phase<1, MODE, NORM>(g, x, x_embed, x_out, y, gain, eps, rs, ring_base, slot_bytes, S, pos, bv, bi, ok, status); break;
        case 2: gemv_phase<2, MODE, NORM>(g, x, x_embed, x_out, y, gain, eps, rs, ring_base, slot_bytes, S, pos, bv, bi, ok, status); break;
        case 3: gemv_phase<3, MODE, NORM>(g, x, x_embed, x_out, y, gain, eps, rs, ring_base, slot_bytes, S, pos, bv, bi, ok, status); break;
        case 4: gemv_phase<4, MODE, NORM>(g, x, x_embed, x_out, y, gain, eps, rs, ring_base, slot_bytes, S, pos, bv, bi, ok, status); break;
        case 6: gemv_phase<6, MODE, NORM>(g, x, x_embed, x_out, y, gain, eps, rs, ring_base, slot_bytes, S, pos, bv, bi, ok, status); break;
        default: gemv_phase<8, MODE, NORM>(g, x, x_embed, x_out, y, gain, eps, rs, ring_base, slot_bytes, S, pos, bv, bi, ok, status); break;
    }
}

template <int G>
__global__ void __launch_bounds__(kThreads, 1) decode_step_mega_kernel(const MegaParams p) {
    NNC_TRACE_SCOPE(40);
    extern __shared__ __align__(128) uint8_t ring[];
    __shared__ MegaSmem<G> sm;
    RingSmem &rs = sm.ring;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages;
    const uint32_t ring_base = smem_u32(ring);
    uint32_t *abort_word = p.bars + 18;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&rs.full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&rs.empty[s])), "r"(kConsumerWarps));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    RingPos pos{0, 0u};

    if (warp == kConsumerWarps) {
        // ---------------- producer ----------------
        if (lane == 0) {
            bool ok = true;
            for (int l = 0; l < p.n_layers && ok; ++l) {
                const MegaLayer &w = p.layers[l];
                ok = stream_matrix(p.gq, reinterpret_cast<const uint8_t *>(w.wqkv), rs, ring_base, p.slot_bytes, S, pos);
                ok = ok && stream_matrix(p.go, reinterpret_cast<const uint8_t *>(w.wo), rs, ring_base, p.slot_bytes, S, pos);
                ok = ok && stream_matrix(p.gg, reinterpret_cast<const uint8_t *>(w.wgu), rs, ring_base, p.slot_bytes, S, pos);
                ok = ok && stream_matrix(p.gd, reinterpret_cast<const uint8_t *>(w.wd), rs, ring_base, p.slot_bytes, S, pos);
            }
            ok = ok && stream_matrix(p.gl, reinterpret_cast<const uint8_t *>(p.lm_head), rs, ring_base, p.slot_bytes, S, pos);
            if (!ok) { atomicExch(abort_word, 1u); if (p.status) atomicExch(p.status, 34); }
        }
        return;
    }

    // ---------------- consumers ----------------
    bool ok = true;
    float best_v = -INFINITY;
    int best_i = 0x7fffffff;
    int bar_k = 0;
    int tok = p.tokens[0];
    tok = tok < 0 ? 0 : (tok >= p.vocab ? p.vocab - 1 : tok);
    const bf16 *embed_row = p.embed + (size_t)tok * p.hidden;
    const int group = warp >> 2, gtid = threadIdx.x & 127;
    const int n_items = p.n_splits * p.nkv;

    AttnParams ap;
    ap.q = p.qkv; ap.q_row_stride = (p.nq + 2 * p.nkv) * kHeadDim;
    ap.out_f32 = p.attn_out; ap.out_bf16 = nullptr; ap.out_bf16_lo = nullptr; ap.out_row_stride = p.nq * kHeadDim;
    ap.part = p.part; ap.tickets = p.tickets; ap.d_len = p.d_len; ap.len_add = 1;
    ap.nkv = p.nkv; ap.max_seq = p.max_seq; ap.n_splits = p.n_splits;
    ap.rope = p.rope; ap.eps = p.eps;

    // tracing builds: CTAs 0 and 77 record, per phase, start / end of work / release from the barrier
#define NNC_PHASE_END(kid)                                                                          \
    {                                                                                               \
        const unsigned long long t_work__ = NNC_TRACE_NOW();                                        \
        (void)t_work__;                                                                             \
        if (!grid_barrier(p.bars, bar_k++, p.status)) return;                                       \
        const unsigned long long t_rel__ = NNC_TRACE_NOW();                                         \
        if (threadIdx.x == 0 && (blockIdx.x == 0 || blockIdx.x == 77)) NNC_TRACE_EVENT(kid, t_phase, t_work__, t_rel__); \
        t_phase = t_rel__;                                                                          \
    }
    unsigned long long t_phase = NNC_TRACE_NOW();
    (void)t_phase;
    for (int l = 0; l < p.n_layers; ++l) {
        const MegaLayer &w = p.layers[l];
        // QKV = Wqkv RMSNorm(x); the first layer reads the embedding row directly
        run_gemv<kGemvStore, true>(p.gq, p.x, l == 0 ? embed_row : nullptr, p.x, p.qkv, w.g_in, p.eps, rs, ring_base,
                                   p.slot_bytes, S, pos, best_v, best_i, ok, p.status);
        NNC_PHASE_END(101)
        // flash-decode (fused QK-norm, RoPE, KV append); two 4-warp groups per CTA, one work item at a time each
        ap.kcache = w.kc; ap.vcache = w.vc; ap.g_q = w.g_q; ap.g_k = w.g_k;
        for (int item = blockIdx.x * 2 + group; item < n_items; item += 2 * gridDim.x)
            attn_decode_body<G, true>(ap, item % p.n_splits, item / p.n_splits, 0, gtid, sm.attn[group], 2 + group);
        NNC_PHASE_END(102)
        run_gemv<kGemvResidual, false>(p.go, p.attn_out, nullptr, nullptr, p.x, nullptr, 0.f, rs, ring_base, p.slot_bytes, S,
                                       pos, best_v, best_i, ok, p.status);
        NNC_PHASE_END(103)
        run_gemv<kGemvSwiglu, true>(p.gg, p.x, nullptr, nullptr, p.act, w.g_post, p.eps, rs, ring_base, p.slot_bytes, S, pos,
                                    best_v, best_i, ok, p.status);
        NNC_PHASE_END(104)
        run_gemv<kGemvResidual, false>(p.gd, p.act, nullptr, nullptr, p.x, nullptr, 0.f, rs, ring_base, p.slot_bytes, S, pos,
                                       best_v, best_i, ok, p.status);
        NNC_PHASE_END(105)
    }
    run_gemv<kGemvLogits, true>(p.gl, p.x, nullptr, nullptr, p.logits, p.g_final, p.eps, rs, ring_base, p.slot_bytes, S, pos,
                                best_v, best_i, ok, p.status);

    if (p.am.out != nullptr) {   // arg-max: per-CTA candidate, the CTA that arrives last folds them (nobody waits)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best_v, o);
            const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
            if (better(ov, oi, best_v, best_i)) { best_v = ov; best_i = oi; }
        }
        if (lane == 0) { rs.red[warp] = best_v; rs.red_i[warp] = best_i; }
        consumer_sync();
        if (threadIdx.x == 0) {
            for (int wv = 1; wv < kConsumerWarps; ++wv)
                if (better(rs.red[wv], rs.red_i[wv], best_v, best_i)) { best_v = rs.red[wv]; best_i = rs.red_i[wv]; }
            p.am.part_val[blockIdx.x] = best_v;
            p.am.part_idx[blockIdx.x] = best_i;
            __threadfence();
            const unsigned tk = atomicAdd(p.am.ticket, 1u);
            rs.is_last = (tk == gridDim.x - 1);
        }
        consumer_sync();
        if (rs.is_last) {
            __threadfence();
            float bv = -INFINITY;
            int bi = 0x7fffffff;
            for (int b = threadIdx.x; b < (int)gridDim.x; b += kConsumerThreads) {
                const float v = __ldcg(p.am.part_val + b);
                const int i = __ldcg(p.am.part_idx + b);
                if (better(v, i, bv, bi)) { bv = v; bi = i; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
            }
            consumer_sync();
            if (lane == 0) { rs.red[warp] = bv; rs.red_i[warp] = bi; }
            consumer_sync();
            if (threadIdx.x == 0) {
                for (int wv = 1; wv < kConsumerWarps; ++wv)
                    if (better(rs.red[wv], rs.red_i[wv], bv, bi)) { bv = rs.red[wv]; bi = rs.red_i[wv]; }
                *p.am.out = bi == 0x7fffffff ? 0 : bi;
                *p.am.ticket = 0u;
            }
        }
    }
}

}  // namespace

namespace {

template <int G>
cudaError_t launch_g(const LaunchCtx &lc, MegaParams p) {
    auto kern = decode_step_mega_kernel<G>;
    static int static_smem = -1;   // per instantiation
    if (static_smem < 0) {
        cudaFuncAttributes fa;
        cudaError_t e = cudaFuncGetAttributes(&fa, kern);
        if (e != cudaSuccess) return e;
        static_smem = (int)fa.sharedSizeBytes;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - static_smem - 1024);
        if (e != cudaSuccess) return e;
    }
    const int budget = 227 * 1024 - static_smem - 1024;
    int S = budget / (int)p.slot_bytes;
    if (S > kMaxStages) S = kMaxStages;
    if (S < 2) return cudaErrorInvalidConfiguration;
    p.stages = S;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(lc.sm_count);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = (size_t)S * p.slot_bytes;
    cfg.stream = lc.stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;   // every CTA must be resident: the phases meet at grid barriers
    at[0].val.cooperative = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (lc.launches) ++*lc.launches;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, p);
    if (e == cudaErrorCooperativeLaunchTooLarge) {
        int occ = -1;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, kThreads, cfg.dynamicSmemBytes);
        cudaFuncAttributes fa;
        cudaFuncGetAttributes(&fa, kern);
        fprintf(stderr, "nnc: whole-step kernel: %d CTAs/SM fit (regs %d, static smem %zu, dynamic %zu, max threads %d)\n", occ,
                fa.numRegs, fa.sharedSizeBytes, cfg.dynamicSmemBytes, fa.maxThreadsPerBlock);
    }
    return e;
}

}  // namespace

bool decode_mega_supported(const MegaParams &p, int sm_count) {
    (void)sm_count;
    const int G = p.nkv > 0 ? p.nq / p.nkv : 0;
    if (!(G == 1 || G == 2 || G == 4 || G == 8)) return false;
    if (p.n_splits < 1 || p.n_splits > kAttnMaxSplits) return false;
    return p.slot_bytes > 0 && p.slot_bytes <= 64 * 1024;
}

cudaError_t launch_decode_mega(const LaunchCtx &lc, const MegaParams &p) {
    switch (p.nq / p.nkv) {
        case 1: return launch_g<1>(lc, p);
        case 2: return launch_g<2>(lc, p);
        case 4: return launch_g<4>(lc, p);
        case 8: return launch_g<8>(lc, p);
    }
    return cudaErrorInvalidValue;
}

}  // namespace nnc
