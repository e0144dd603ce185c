// Causal attention of the prompt phase, one-term fp16 form, TWO CTAs per SM.
//
// Same computation as attn_prefill_tc.cu (Section 3.1.2, Eq. 1: the score / probability tile stays on the SM between
// the two products), for the case where Q, P and the cache rows travel as one fp16 term each.  The organisation differs:
// a CTA is small enough (192 threads, 97 KB of shared memory, 256 tensor-memory columns) for two of them to share an SM,
// so that one CTA's set-up (query load, norm, rotation) and output pass hide behind the other's steady state, and the
// cache is walked in steps of 64 positions with TWO score buffers of 64 columns: while the softmax warps work on step j
// the tensor cores compute S_{j+1} = Q K_{j+1}^T and O += P_{j-1} V_{j-1}.
//
//   warp 0      TMA producer: K and V tiles of 64 cache positions (two 128B-swizzled boxes of 64 head-dimension
//               elements each), two stages.
//   warp 1      MMA issuer (one lane).  Q is a shared-memory operand here (tensor memory has no room for it beside
//               two S buffers and O in half an SM's columns).
//   warps 2-5   softmax, ONE thread per query row: no exchange between threads at all.  The thread loads its fp32
//               query row (optionally applying the per-head RMSNorm and RoPE), scales it to log2 units and writes it to
//               shared memory in the K-major swizzled operand layout; per step: 64 scores -> mask (diagonal tiles) ->
//               exp2 -> fp16 probabilities over the first 32 columns of the step's S buffer; finally O / l to the output.
// Online softmax with the lazy maximum of attn_prefill_tc.cu (threshold 2^8).  Every mbarrier wait is bounded; on
// expiry the CTA raises the status word, drains and frees its tensor memory.
#include "attn_prefill_common.cuh"

namespace nnc {

namespace {

constexpr int kFThreads = 192;
constexpr int kFSoftmax = 128;
constexpr int kStep = 64;                          // cache positions per step
constexpr int kHalfSlab = kStep * 128;             // bytes of a [64 positions][64 x 16 bit] swizzled slab
constexpr int kStepTile = 2 * kHalfSlab;           // [64][128] 16-bit tile
constexpr int kFSmem = kTile + 4 * kStepTile + 1024 /*align slack*/ + 128 /*barriers*/;   // Q, 2 x (K, V)
constexpr uint32_t kFColS = 0, kFColO = 128, kFTmemCols = 256;   // S buffers at columns 0 and 64

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Tracing builds: the roles keep per-step time stamps in shared memory (slot [step][what]; row 31 belongs to the CTA as a
// whole) and thread 0 turns them into records when the CTA is done, so that recording is not on the path it measures.
#ifdef NNC_TRACE
#define NNC_TS(j, k, t) do { if (traced && (j) < 32) trace_ts[(j)][(k)] = (t); } while (0)
#else
#define NNC_TS(j, k, t) do { } while (0)
#endif

template <bool OUT_FP16>
__global__ void __launch_bounds__(kFThreads, 2)
attn_prefill_f16_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const PfParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t q_tile = base;
    auto k_tile = [&](int st) { return base + (uint32_t)kTile + (uint32_t)st * 2u * kStepTile; };
    auto v_tile = [&](int st) { return k_tile(st) + (uint32_t)kStepTile; };
    const uint32_t bars = base + (uint32_t)kTile + 4u * kStepTile;
    const uint32_t q_ready = bars;
    auto k_full = [&](int st) { return bars + 8u * (1 + st); };
    auto v_full = [&](int st) { return bars + 8u * (3 + st); };
    auto s_full = [&](int st) { return bars + 8u * (5 + st); };
    auto p_full = [&](int st) { return bars + 8u * (7 + st); };
    auto pv_done = [&](int st) { return bars + 8u * (9 + st); };
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &abort_s;
        const unsigned long long tr_cta = NNC_TRACE_NOW();
    (void)tr_cta;
#ifdef NNC_TRACE
    __shared__ unsigned long long trace_ts[32][8];
#endif
    // The grid is one-dimensional and ordered by decreasing length: all (head, sequence) pairs of the last query tile
    // (the most cache tiles) first, the first query tile last, so that the long CTAs never start late.  Neighbouring
    // CTAs are query heads of the same KV head: they stream the same cache tiles at the same time.
    const int per_qt = p.nq * p.batch;
    const int qt = p.n_qt - 1 - (int)blockIdx.x / per_qt;
    const int h = ((int)blockIdx.x % per_qt) % p.nq, seq = ((int)blockIdx.x % per_qt) / p.nq;
    const int G = p.nq / p.nkv, jkv = h / G;
    const int q0 = qt * kQM;
    const int n_valid = p.n_past + p.T;
    const int n_keys = min(p.n_past + q0 + kQM, n_valid);   // cache positions the last row of this tile may see
    const int n_tiles = (n_keys + kStep - 1) / kStep;   // steps of 64 cache positions
    const bool traced = NNC_TRACE_ALL_CTAS || (h == p.nq / 2 && seq == 0);   // tracing builds only
    (void)traced;

    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(q_ready, kFSoftmax);
        for (int st = 0; st < 2; ++st) {
            mbar_init(k_full(st), 1); mbar_init(v_full(st), 1); mbar_init(s_full(st), 1);
            mbar_init(p_full(st), kFSoftmax); mbar_init(pv_done(st), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        // with two CTAs of 256 columns per SM the allocation always finds room once an earlier kernel's CTAs have left
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(kFTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    pdl_launch_dependents();

    if (warp == 0) {
        if (lane == 0) {   // ---------------- TMA producer ----------------
            pdl_wait();    // the cache rows of the new tokens come from the preceding kernel
            const int z = seq * p.nkv + jkv;
            auto load_k = [&](int j) {
                const int st = j & 1;
                mbar_expect_tx(k_full(st), kStepTile);
                tma_load_3d(k_tile(st), &map_k, k_full(st), 0, j * kStep, z);
                tma_load_3d(k_tile(st) + kHalfSlab, &map_k, k_full(st), 64, j * kStep, z);
            };
            auto load_v = [&](int j) {
                const int st = j & 1;
                mbar_expect_tx(v_full(st), kStepTile);
                tma_load_3d(v_tile(st), &map_v, v_full(st), 0, j * kStep, z);
                tma_load_3d(v_tile(st) + kHalfSlab, &map_v, v_full(st), 64, j * kStep, z);
            };
            // A stage's K tile is free as soon as the S of the step that read it is complete -- a whole softmax pass before
            // that step's second product -- so K runs one step ahead of V here: K_{j+1} is requested when S_{j-1} is
            // complete, V_j when O += P_{j-2} V_{j-2} is.  The events come in exactly this order, and each load has more
            // than a softmax pass before it is needed.
            load_k(0);
            if (n_tiles > 1) load_k(1);
            load_v(0);
            for (int j = 1; j < n_tiles; ++j) {
                if (j + 1 < n_tiles) {
                    if (!mbar_wait(s_full((j - 1) & 1), (uint32_t)(((j - 1) >> 1) & 1), abort_flag, p.status, 31)) break;
                    load_k(j + 1);
                }
                if (j >= 2 && !mbar_wait(pv_done(j & 1), (uint32_t)(((j - 2) >> 1) & 1), abort_flag, p.status, 32)) break;
                load_v(j);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {   // ---------------- MMA issuer ----------------
            constexpr uint32_t idesc_qk = make_idesc(kStep, true, false);
            constexpr uint32_t idesc_pv = make_idesc(kHeadDim, true, true);
            bool ok = mbar_wait(q_ready, 0u, abort_flag, p.status, 33);
            const uint64_t dq = make_smem_desc(q_tile);
            const uint64_t dk[2] = {make_smem_desc(k_tile(0)), make_smem_desc(k_tile(1))};
            const uint64_t dv[2] = {make_smem_desc_mn(v_tile(0), kHalfSlab), make_smem_desc_mn(v_tile(1), kHalfSlab)};
            const uint32_t to = tmem_base + kFColO;
            auto issue_qk = [&](int j) -> bool {
                const int st = j & 1, u = j >> 1;
                if (!mbar_wait(k_full(st), (uint32_t)(u & 1), abort_flag, p.status, 34)) return false;
                // the score buffer holds P_{j-2} until O += P_{j-2} V_{j-2} has completed
                if (j >= 2 && !mbar_wait(pv_done(st), (uint32_t)((u - 1) & 1), abort_flag, p.status, 35)) return false;
                tc_fence_after();
                const uint32_t d = tmem_base + kFColS + (uint32_t)st * kStep;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)     // 16 head-dimension elements per instruction
                    umma_bf16(d, dq + (uint64_t)(((ks >> 2) * kSlab + (ks & 3) * 32) >> 4),
                              dk[st] + (uint64_t)(((ks >> 2) * kHalfSlab + (ks & 3) * 32) >> 4), idesc_qk, ks != 0);
                umma_commit(s_full(st));
                return true;
            };
            if (ok) ok = issue_qk(0);
            for (int j = 0; ok && j < n_tiles; ++j) {
                const unsigned long long tr0 = NNC_TRACE_NOW();
                (void)tr0;
                if (j + 1 < n_tiles && !issue_qk(j + 1)) break;
                const int st = j & 1, u = j >> 1;
                const unsigned long long tr1 = NNC_TRACE_NOW();
                (void)tr1;
                if (!mbar_wait(p_full(st), (uint32_t)(u & 1), abort_flag, p.status, 36)) break;
                if (!mbar_wait(v_full(st), (uint32_t)(u & 1), abort_flag, p.status, 37)) break;
                tc_fence_after();
                if (j < 31) { NNC_TS(j, 0, tr0); NNC_TS(j, 1, tr1); NNC_TS(j, 2, NNC_TRACE_NOW()); }
                const uint32_t pa = tmem_base + kFColS + (uint32_t)st * kStep;   // P: two positions per column
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)     // 16 cache positions per instruction
                    umma_bf16_ts(to, pa + (uint32_t)ks * 8u, dv[st] + (uint64_t)(ks * (2048 >> 4)), idesc_pv, (j != 0) || (ks != 0));
                umma_commit(pv_done(st));
            }
        }
    } else {   // ---------------- softmax warps 2..5: one thread per query row ----------------
        const int quarter = warp & 3;                    // the TMEM lane quarter this warp may touch
        const int r = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int tok = q0 + r;
        const bool valid = tok < p.T;
        const int pos = p.n_past + tok;                  // absolute position of this row's query
        pdl_wait();
        {   // Q -> shared memory, K-major under the 128-byte swizzle (16-byte chunk index XOR row % 8)
            const float qscale = 1.4426950408889634f * rsqrtf((float)kHeadDim);
            const float *src = p.qkv + ((size_t)seq * p.T + (size_t)min(tok, p.T - 1)) * p.row_stride + (size_t)h * kHeadDim;
            float q[128];
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                const float4 a = reinterpret_cast<const float4 *>(src)[c];
                q[4 * c] = a.x; q[4 * c + 1] = a.y; q[4 * c + 2] = a.z; q[4 * c + 3] = a.w;
            }
            if (p.g_q) {
                float ss = 0.f;
#pragma unroll
                for (int e = 0; e < 128; ++e) ss = fmaf(q[e], q[e], ss);
                const float inv = rsqrtf(ss * (1.f / kHeadDim) + p.eps);
                const float *cs = p.rope + (size_t)min(pos, p.n_past + p.T - 1) * kHeadDim;   // (cos, sin) of pair i at 2i
#pragma unroll
                for (int i = 0; i < 64; i += 2) {
                    const float4 t = *reinterpret_cast<const float4 *>(cs + 2 * i);         // c_i s_i c_{i+1} s_{i+1}
                    const uint32_t ga = *reinterpret_cast<const uint32_t *>(p.g_q + i), gb = *reinterpret_cast<const uint32_t *>(p.g_q + 64 + i);
                    const float a0 = q[i] * inv * bf16_lo(ga), a1 = q[i + 1] * inv * bf16_hi(ga);
                    const float b0 = q[64 + i] * inv * bf16_lo(gb), b1 = q[65 + i] * inv * bf16_hi(gb);
                    q[i] = a0 * t.x - b0 * t.y;      q[i + 1] = a1 * t.z - b1 * t.w;
                    q[64 + i] = b0 * t.x + a0 * t.y; q[65 + i] = b1 * t.z + a1 * t.w;
                }
            }
            const float sc = valid ? qscale : 0.f;
#pragma unroll
            for (int cc = 0; cc < 16; ++cc) {   // 16-byte chunk cc of the row: head-dimension elements 8 cc .. 8 cc + 7
                uint4 v;
                v.x = pack_f16x2_sat(q[8 * cc] * sc, q[8 * cc + 1] * sc);
                v.y = pack_f16x2_sat(q[8 * cc + 2] * sc, q[8 * cc + 3] * sc);
                v.z = pack_f16x2_sat(q[8 * cc + 4] * sc, q[8 * cc + 5] * sc);
                v.w = pack_f16x2_sat(q[8 * cc + 6] * sc, q[8 * cc + 7] * sc);
                sts128(q_tile + (uint32_t)(cc >> 3) * kSlab + (uint32_t)r * 128u + (uint32_t)(((cc & 7) ^ (r & 7)) << 4), v);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes, async-proxy (MMA) reads
            mbar_arrive(q_ready);
        }
        float m_used = -INFINITY, l = 0.f;
        const uint32_t to = tmem_base + lane_addr + kFColO;
        bool ok = true;
        const unsigned long long tr_q = NNC_TRACE_NOW();
        (void)tr_q;
        for (int j = 0; j < n_tiles; ++j) {
            const int st = j & 1, u = j >> 1;
            const unsigned long long ts0 = NNC_TRACE_NOW();
            (void)ts0;
            ok = __all_sync(0xffffffffu, mbar_wait(s_full(st), (uint32_t)(u & 1), abort_flag, p.status, 38));
            if (!ok) break;
            const unsigned long long ts1 = NNC_TRACE_NOW();
            (void)ts1;
            tc_fence_after();
            const uint32_t ts = tmem_base + lane_addr + kFColS + (uint32_t)st * kStep;
            uint32_t sv[2][32];
            tmem_ld32_nowait(ts, sv[0]);
            tmem_ld32_nowait(ts + 32u, sv[1]);
            tmem_wait_ld();
            const unsigned long long ts2 = NNC_TRACE_NOW();
            (void)ts2;
            if (j * kStep + kStep - 1 > p.n_past + q0) {   // the step reaches past the first row's position: causal mask
                const int k0 = j * kStep;
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (k0 + 32 * c + e > pos) sv[c][e] = 0xff800000u;   // -inf
            }
            // three-input maxima, four independent chains
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) mx[q] = max3(mx[q], __uint_as_float(sv[c][e + 2 * q]), __uint_as_float(sv[c][e + 2 * q + 1]));
                }
            const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
            if (j == 0) {
                m_used = m_tile;   // finite: position 0 is visible to every row
            } else {
                // a row whose step is masked out entirely (the second half of a diagonal tile) has m_tile = -inf: no move
                const bool need = m_tile > m_used + kLazyMax;
                if (__any_sync(0xffffffffu, need)) {
                    // O is rescaled in tensor memory, 32 columns at a time; rows that keep their maximum multiply by 1.
                    // The product of the previous step must have landed first.
                    ok = __all_sync(0xffffffffu, mbar_wait(pv_done((j - 1) & 1), (uint32_t)(((j - 1) >> 1) & 1), abort_flag, p.status, 40));
                    if (!ok) break;
                    tc_fence_after();
                    const float m_new = need ? m_tile : m_used;
                    const float alpha = ex2_approx(m_used - m_new);
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t t[32];
                        tmem_ld32(to + 32u * c, t);
#pragma unroll
                        for (int e = 0; e < 32; ++e) t[e] = __float_as_uint(__uint_as_float(t[e]) * alpha);
                        tmem_st32(to + 32u * c, t);
                    }
                    tmem_wait_st();
                    l *= alpha;
                    m_used = m_new;
                }
            }
            // exponents are <= 2^8 by the lazy maximum; results below 2^-126 flush to zero, which a row sum >= 1 cannot see.
            // P over S: fp16 pairs, two positions per column, so chunk c (positions 32 c .. 32 c + 31) lands in columns
            // 16 c .. 16 c + 15 of the step's buffer -- columns whose scores this thread already holds in registers.
            // the subtraction and the row sum run as packed two-lane fp32 operations: half the instructions
            float2 sum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            const float2 neg_m = make_float2(-m_used, -m_used);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t ph[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const float2 x = __fadd2_rn(make_float2(__uint_as_float(sv[c][2 * e]), __uint_as_float(sv[c][2 * e + 1])), neg_m);
                    const float2 pr = make_float2(ex2_approx(x.x), ex2_approx(x.y));
                    sum[e & 1] = __fadd2_rn(sum[e & 1], pr);
                    ph[e] = pack_f16x2_sat(pr.x, pr.y);   // probabilities are at most 2^8: inside the fp16 range
                }
                tmem_st16(ts + 16u * c, ph);
            }
            l += (sum[0].x + sum[0].y) + (sum[1].x + sum[1].y);
            const unsigned long long ts3 = NNC_TRACE_NOW();
            (void)ts3;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(p_full(st));
            if (warp == 2 && lane == 0 && j < 31) { NNC_TS(j, 3, ts0); NNC_TS(j, 4, ts1); NNC_TS(j, 5, ts2); NNC_TS(j, 6, ts3); NNC_TS(j, 7, NNC_TRACE_NOW()); }
        }
        // ---- O / l -> output ----
        const unsigned long long tr_e = NNC_TRACE_NOW();
        (void)tr_e;
        if (warp == 2 && lane == 0) { NNC_TS(31, 0, tr_q); NNC_TS(31, 1, tr_e); }
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(pv_done((n_tiles - 1) & 1), (uint32_t)(((n_tiles - 1) >> 1) & 1), abort_flag, p.status, 39));
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / l;
            const size_t oi = ((size_t)seq * p.T + (size_t)tok) * p.nq * kHeadDim + (size_t)h * kHeadDim;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t t[32];
                tmem_ld32(to + 32u * c, t);
                if (!valid) continue;
                if (OUT_FP16) {
                    uint32_t o[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        o[e] = pack_f16x2_sat(__uint_as_float(t[2 * e]) * inv, __uint_as_float(t[2 * e + 1]) * inv);
                    uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<__half *>(p.out) + oi + 32 * c);
#pragma unroll
                    for (int e = 0; e < 4; ++e) dst[e] = make_uint4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
                } else {
                    uint32_t o[16], ol[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const float a = __uint_as_float(t[2 * e]) * inv, b = __uint_as_float(t[2 * e + 1]) * inv;
                        o[e] = pack_bf16x2(a, b);
                        ol[e] = pack_bf16x2(a - bf16_lo(o[e]), b - bf16_hi(o[e]));
                    }
                    uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<bf16 *>(p.out) + oi + 32 * c);
#pragma unroll
                    for (int e = 0; e < 4; ++e) dst[e] = make_uint4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
                    if (p.out_lo) {
                        uint4 *dl = reinterpret_cast<uint4 *>(reinterpret_cast<bf16 *>(p.out_lo) + oi + 32 * c);
#pragma unroll
                        for (int e = 0; e < 4; ++e) dl[e] = make_uint4(ol[4 * e], ol[4 * e + 1], ol[4 * e + 2], ol[4 * e + 3]);
                    }
                }
            }
        }
    }

    // ---- teardown ----
    __syncwarp();
    if (*abort_flag && threadIdx.x == 0) {
        // let copies that are still in flight land before the shared memory is released
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kFTmemCols) : "memory");
    }
#ifdef NNC_TRACE
    // tracing builds: the roles kept their per-tile time stamps in shared memory; they leave as records only now, so that
    // recording does not sit on the path it measures
    if (traced && threadIdx.x == 0) {
        const unsigned long long t_end = NNC_TRACE_NOW();
        NNC_TRACE_EVENT(315, tr_cta, trace_ts[31][0], t_end);
        NNC_TRACE_EVENT(314, tr_cta, trace_ts[31][1], t_end);
        for (int j = 0; j < n_tiles && j < 31; ++j) {
            NNC_TRACE_EVENT(311, trace_ts[j][0], trace_ts[j][1], trace_ts[j][2]);
            NNC_TRACE_EVENT(312, trace_ts[j][3], trace_ts[j][4], trace_ts[j][5]);
            NNC_TRACE_EVENT(313, trace_ts[j][5], trace_ts[j][6], trace_ts[j][7]);
        }
    }
#endif
}

template <bool OUT_FP16>
cudaError_t launch_pf16(const LaunchCtx &lc, const CUtensorMap &mk, const CUtensorMap &mv, const PfParams &p, dim3 grid) {
    auto kern = attn_prefill_f16_kernel<OUT_FP16>;
    static unsigned long long attr_done = 0;   // per instantiation, one bit per device
    if (cudaError_t e = ensure_dynamic_smem(kern, kFSmem, &attr_done); e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kFThreads);
    cfg.dynamicSmemBytes = kFSmem;
    cfg.stream = lc.stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = lc.pdl ? 1 : 0;
    if (lc.launches) ++*lc.launches;
    return cudaLaunchKernelEx(&cfg, kern, mk, mv, p);
}

}  // namespace

// The one-term fp16 form of launch_attn_prefill: the tensor maps cover the fp16 image of the cache rows.
cudaError_t launch_attn_prefill_f16(const LaunchCtx &lc, const CUtensorMap &mk, const CUtensorMap &mv, const PfParams &p, dim3 grid,
                                    bool out_fp16) {
    return out_fp16 ? launch_pf16<true>(lc, mk, mv, p, grid) : launch_pf16<false>(lc, mk, mv, p, grid);
}

}  // namespace nnc
