// Causal attention of the prompt phase, one-term fp16 form, TWO CTAs per SM.
//
// Same computation as attn_prefill_tc.cu (Section 3.1.2, Eq. 1: the score / probability tile stays on the SM between
// the two products), for the case where Q, P and the cache rows travel as one fp16 term each.  The organisation differs:
// a CTA is small enough (192 threads, 97 KB of shared memory, 256 tensor-memory columns) for two of them to share an SM,
// and each one runs its chain  S = Q K_j^T  ->  softmax  ->  O += P_j V_j  strictly in order on ONE score buffer.  The
// overlap of tensor-core work with softmax work comes from the other CTA of the SM, which also hides a CTA's set-up
// (query load, norm, rotation) and its output pass behind the partner's steady state.
//
//   warp 0      TMA producer: K tile and V tile of 128 cache positions each (two 128B-swizzled boxes of 64
//               head-dimension elements), single-buffered: K_{j+1} is requested when S_j is complete, V_{j+1} when
//               O += P_j V_j is complete; both have a softmax pass of slack before they are needed.
//   warp 1      MMA issuer (one lane).  Q is a shared-memory operand here (tensor memory has no room for it beside
//               S and O in half an SM's columns).
//   warps 2-5   softmax, ONE thread per query row: no exchange between threads at all.  The thread loads its fp32
//               query row (optionally applying the per-head RMSNorm and RoPE), scales it to log2 units and writes it to
//               shared memory in the K-major swizzled operand layout; per tile: 128 scores -> mask (diagonal tiles) ->
//               exp2 -> fp16 probabilities over the first 64 columns of S; finally O / l to the output.
// Online softmax with the lazy maximum of attn_prefill_tc.cu (threshold 2^8).  Every mbarrier wait is bounded; on
// expiry the CTA raises the status word, drains and frees its tensor memory.
#include "attn_prefill_common.cuh"

namespace nnc {

namespace {

constexpr int kFThreads = 192;
constexpr int kFSoftmax = 128;
constexpr int kFSmem = 3 * kTile + 1024 /*align slack*/ + 128 /*barriers*/;   // Q, K, V
constexpr uint32_t kFColS = 0, kFColO = 128, kFTmemCols = 256;

__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <bool OUT_FP16>
__global__ void __launch_bounds__(kFThreads, 2)
attn_prefill_f16_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const PfParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t q_tile = base, k_tile = base + (uint32_t)kTile, v_tile = base + 2u * kTile;
    const uint32_t bars = base + 3u * kTile;
    const uint32_t q_ready = bars, k_full = bars + 8u, v_full = bars + 16u, s_full = bars + 24u, p_full = bars + 32u,
                   pv_done = bars + 40u;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &abort_s;
        const unsigned long long tr_cta = NNC_TRACE_NOW();
    (void)tr_cta;
#ifdef NNC_TRACE
    __shared__ unsigned long long trace_ts[32][8];
#define NNC_TS(j, k, t) do { if (traced && (j) < 32) trace_ts[(j)][(k)] = (t); } while (0)
#else
#define NNC_TS(j, k, t) do { } while (0)
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
    const int n_tiles = (n_keys + kKN - 1) / kKN;
    const bool traced = NNC_TRACE_ALL_CTAS || (h == p.nq / 2 && seq == 0);   // tracing builds only
    (void)traced;

    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(q_ready, kFSoftmax);
        mbar_init(k_full, 1); mbar_init(v_full, 1); mbar_init(s_full, 1);
        mbar_init(p_full, kFSoftmax); mbar_init(pv_done, 1);
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
            for (int j = 0; j < n_tiles; ++j) {
                const uint32_t prev = (uint32_t)((j - 1) & 1);
                if (j > 0 && !mbar_wait(s_full, prev, abort_flag, p.status, 31)) break;    // K_{j-1} has been read
                mbar_expect_tx(k_full, kTile);
                tma_load_3d(k_tile, &map_k, k_full, 0, j * kKN, z);
                tma_load_3d(k_tile + kSlab, &map_k, k_full, 64, j * kKN, z);
                if (j > 0 && !mbar_wait(pv_done, prev, abort_flag, p.status, 32)) break;   // V_{j-1} has been read
                mbar_expect_tx(v_full, kTile);
                tma_load_3d(v_tile, &map_v, v_full, 0, j * kKN, z);
                tma_load_3d(v_tile + kSlab, &map_v, v_full, 64, j * kKN, z);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {   // ---------------- MMA issuer ----------------
            constexpr uint32_t idesc_qk = make_idesc(kKN, true, false);
            constexpr uint32_t idesc_pv = make_idesc(kHeadDim, true, true);
            bool ok = mbar_wait(q_ready, 0u, abort_flag, p.status, 33);
            const uint64_t dq = make_smem_desc(q_tile), dk = make_smem_desc(k_tile);
            const uint64_t dv = make_smem_desc_mn(v_tile, kSlab);
            const uint32_t ts = tmem_base + kFColS, to = tmem_base + kFColO;
            for (int j = 0; ok && j < n_tiles; ++j) {
                const uint32_t par = (uint32_t)(j & 1);
                const unsigned long long tr0 = NNC_TRACE_NOW();
                (void)tr0;
                if (!mbar_wait(k_full, par, abort_flag, p.status, 34)) break;
                // the score buffer holds P_{j-1} until O += P_{j-1} V_{j-1} has completed
                if (j > 0 && !mbar_wait(pv_done, par ^ 1u, abort_flag, p.status, 35)) break;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // 16 head-dimension elements per instruction
                    const uint64_t off = (uint64_t)(((ks >> 2) * kSlab + (ks & 3) * 32) >> 4);
                    umma_bf16(ts, dq + off, dk + off, idesc_qk, ks != 0);
                }
                umma_commit(s_full);
                const unsigned long long tr1 = NNC_TRACE_NOW();
                (void)tr1;
                if (!mbar_wait(p_full, par, abort_flag, p.status, 36)) break;
                if (!mbar_wait(v_full, par, abort_flag, p.status, 37)) break;
                tc_fence_after();
                NNC_TS(j, 0, tr0); NNC_TS(j, 1, tr1); NNC_TS(j, 2, NNC_TRACE_NOW());
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)     // 16 cache positions per instruction; P: two positions per column
                    umma_bf16_ts(to, ts + (uint32_t)ks * 8u, dv + (uint64_t)(ks * (2048 >> 4)), idesc_pv, (j != 0) || (ks != 0));
                umma_commit(pv_done);
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
        const uint32_t ts = tmem_base + lane_addr + kFColS, to = tmem_base + lane_addr + kFColO;
        bool ok = true;
        const unsigned long long tr_q = NNC_TRACE_NOW();
        (void)tr_q;
        for (int j = 0; j < n_tiles; ++j) {
            const unsigned long long ts0 = NNC_TRACE_NOW();
            (void)ts0;
            ok = __all_sync(0xffffffffu, mbar_wait(s_full, (uint32_t)(j & 1), abort_flag, p.status, 38));
            if (!ok) break;
            const unsigned long long ts1 = NNC_TRACE_NOW();
            (void)ts1;
            tc_fence_after();
            // S_j complete also means O += P_{j-1} V_{j-1} is complete: the issuer waited for it before this product
            uint32_t sv[4][32];
            tmem_ld32_nowait(ts, sv[0]);
            tmem_ld32_nowait(ts + 32u, sv[1]);
            tmem_ld32_nowait(ts + 64u, sv[2]);
            tmem_ld32_nowait(ts + 96u, sv[3]);
            tmem_wait_ld();
            const unsigned long long ts2 = NNC_TRACE_NOW();
            (void)ts2;
            if (j * kKN + kKN - 1 > p.n_past + q0) {   // the tile reaches past the first row's position: causal mask
                const int k0 = j * kKN;
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (k0 + 32 * c + e > pos) sv[c][e] = 0xff800000u;   // -inf
            }
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    mx[0] = fmaxf(mx[0], __uint_as_float(sv[c][e]));     mx[1] = fmaxf(mx[1], __uint_as_float(sv[c][e + 1]));
                    mx[2] = fmaxf(mx[2], __uint_as_float(sv[c][e + 2])); mx[3] = fmaxf(mx[3], __uint_as_float(sv[c][e + 3]));
                }
            const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
            if (j == 0) {
                m_used = m_tile;   // finite: position 0 is visible to every row
            } else {
                const bool need = m_tile > m_used + kLazyMax;
                if (__any_sync(0xffffffffu, need)) {
                    // O is rescaled in tensor memory, 32 columns at a time; rows that keep their maximum multiply by 1
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
            // 16 c .. 16 c + 15 -- columns whose scores this thread already holds in registers.
            float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t ph[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const float a = ex2_approx(__uint_as_float(sv[c][2 * e]) - m_used);
                    const float b = ex2_approx(__uint_as_float(sv[c][2 * e + 1]) - m_used);
                    sum[(2 * e) & 3] += a;
                    sum[(2 * e + 1) & 3] += b;
                    ph[e] = pack_f16x2_sat(a, b);   // probabilities are at most 2^8: inside the fp16 range
                }
                tmem_st16(ts + 16u * c, ph);
            }
            l += (sum[0] + sum[1]) + (sum[2] + sum[3]);
            const unsigned long long ts3 = NNC_TRACE_NOW();
            (void)ts3;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(p_full);
            if (warp == 2 && lane == 0) { NNC_TS(j, 3, ts0); NNC_TS(j, 4, ts1); NNC_TS(j, 5, ts2); NNC_TS(j, 6, ts3); NNC_TS(j, 7, NNC_TRACE_NOW()); }
        }
        // ---- O / l -> output ----
        const unsigned long long tr_e = NNC_TRACE_NOW();
        (void)tr_e;
        if (warp == 2 && lane == 0) { NNC_TS(31, 0, tr_q); NNC_TS(31, 1, tr_e); }
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(pv_done, (uint32_t)((n_tiles - 1) & 1), abort_flag, p.status, 39));
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
