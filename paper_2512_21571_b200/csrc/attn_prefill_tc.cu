// Causal attention of the prompt phase on the 5th-generation tensor cores: the query at position p attends to
// cache positions 0..p of its sequence.  K and V are read from the bf16 cache, which already holds the new tokens.
//
// The score / probability tile never leaves the SM between the two products -- the form the paper's
// "MatMul -> Exp -> MatMul" pass-through layout takes here (Section 3.1.2, Eq. 1): S = Q K^T is accumulated in
// tensor memory, the softmax warps read it with tcgen05.ld, and write the probabilities back over it as the bf16
// A operand of O += P V, which tcgen05.mma reads straight from tensor memory.
//
// One CTA per (128 query rows, query head, sequence), 320 threads:
//   warp 0      TMA producer: K and V tiles of 128 cache positions (two 128B-swizzled boxes of 64 head-dimension
//               elements each) into a two-stage shared-memory ring.  The tensor map's position extent is the number
//               of valid cache rows, so rows past the end arrive as zeros (0 * stale bits would not be 0).
//   warp 1      MMA issuer (one lane): S[j&1] = Q K_j^T into one of two score buffers, so the product of tile j+1
//               runs while the softmax warps work on tile j; then O += P_j V_j with V as an MN-major operand (the
//               cache row is [position][head dim], contraction over positions).  Q, like P, is an A operand in
//               TENSOR memory, which leaves the shared memory to K and V (a 128 x 128 x 16 instruction issues every
//               ~65 cycles with A in either place).
//   warps 2-9   softmax: two threads per query row (warps w and w + 4 share a tensor-memory lane quarter and split
//               the 128 columns of a row between them; the row maximum crosses through shared memory).  They load Q
//               (fp32; optionally applying the per-head RMSNorm and RoPE on the way: a thread holds the whole head, so
//               the norm and the rotation pairs (i, i + 64) are thread-local), scale it to log2 units and write it to
//               tensor memory as value + residual bf16 pairs; per tile: scores -> mask (diagonal tiles) -> exp2 ->
//               probabilities; finally O / l to the output.
// Q and P are fed as two bf16 terms (value + residual) multiplied into the same accumulator: a single bf16 term
// costs 2^-9 per operand, which the parity tolerance of deep models does not allow.  Q is split by rounding; P, which
// is produced 128 x 128 values at a time on the critical path, by truncating the fp32 bit pattern twice.
// Online softmax with a lazy maximum: the running maximum m only moves (and O is rescaled in tensor memory) when a
// tile's maximum exceeds it by more than 2^8; probabilities then stay below 256, which fp32 sums and the bf16
// pair hold without loss.  The result is the exact softmax whatever m is.
// Every mbarrier wait is bounded; on expiry the CTA raises the status word, drains and frees its tensor memory.
#include "attn_prefill_common.cuh"

namespace nnc {

namespace {

constexpr int kPfThreads = 320;
constexpr int kSoftmaxThreads = 256;
constexpr int kPfSmem = 4 * kTile + 1024 /*align slack*/ + 256 /*barriers*/;   // 2 x (K, V)
// tensor-memory columns: two score / probability buffers, the output accumulator, the queries (value pairs in the
// first 64 columns, residual pairs in the next 64; two head-dimension elements per column)
constexpr uint32_t kColS = 0, kColO = 256, kColQ = 384, kTmemCols = 512;

// OUT_FP16: the output is one fp16 matrix (saturating) instead of a bf16 value + residual pair.
// (The one-term fp16 form of the same computation is a kernel of its own, attn_prefill_f16.cu.)
template <bool OUT_FP16>
__global__ void __launch_bounds__(kPfThreads, 1)
attn_prefill_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const PfParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    auto k_tile = [&](int s) { return base + (uint32_t)s * 2u * kTile; };
    auto v_tile = [&](int s) { return k_tile(s) + (uint32_t)kTile; };
    const uint32_t bars = base + 4u * kTile;
    const uint32_t q_ready = bars;
    auto k_full = [&](int s) { return bars + 8u * (1 + s); };
    auto v_full = [&](int s) { return bars + 8u * (3 + s); };
    auto s_full = [&](int s) { return bars + 8u * (5 + s); };
    auto p_full = [&](int s) { return bars + 8u * (7 + s); };
    auto pv_done = [&](int s) { return bars + 8u * (9 + s); };
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ float xch[2][2][kQM];   // [tile parity][column half][row]: the pair's half-row maxima (and, at the end, sums)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &abort_s;
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

    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(q_ready, kSoftmaxThreads);
        for (int s = 0; s < 2; ++s) {
            mbar_init(k_full(s), 1); mbar_init(v_full(s), 1); mbar_init(s_full(s), 1);
            mbar_init(p_full(s), kSoftmaxThreads); mbar_init(pv_done(s), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(kTmemCols)
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
                const int s = j & 1, u = j >> 1;
                if (j >= 2 && !mbar_wait(pv_done(s), (uint32_t)((u - 1) & 1), abort_flag, p.status, 21)) break;
                mbar_expect_tx(k_full(s), kTile);
                tma_load_3d(k_tile(s), &map_k, k_full(s), 0, j * kKN, z);
                tma_load_3d(k_tile(s) + kSlab, &map_k, k_full(s), 64, j * kKN, z);
                mbar_expect_tx(v_full(s), kTile);
                tma_load_3d(v_tile(s), &map_v, v_full(s), 0, j * kKN, z);
                tma_load_3d(v_tile(s) + kSlab, &map_v, v_full(s), 64, j * kKN, z);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {   // ---------------- MMA issuer ----------------
            constexpr uint32_t idesc_qk = make_idesc(kKN, false, false);
            constexpr uint32_t idesc_pv = make_idesc(kHeadDim, false, true);
            bool ok = mbar_wait(q_ready, 0u, abort_flag, p.status, 22);
            tc_fence_after();
            // Descriptors differ only in their 14-bit start-address field (bytes >> 4), so every operand descriptor of
            // the kernel is a base computed once plus a compile-time constant: the issuing thread spends a handful of
            // instructions per tcgen05.mma, less than the ~65 cycles one 128 x 128 x 16 instruction executes for.
            const uint32_t tq = tmem_base + kColQ;
            const uint64_t dk[2] = {make_smem_desc(k_tile(0)), make_smem_desc(k_tile(1))};
            const uint64_t dv[2] = {make_smem_desc_mn(v_tile(0), kSlab), make_smem_desc_mn(v_tile(1), kSlab)};
            auto issue_qk = [&](int j) -> bool {
                const int s = j & 1, u = j >> 1;
                if (!mbar_wait(k_full(s), (uint32_t)(u & 1), abort_flag, p.status, 23)) return false;
                if (j >= 2 && !mbar_wait(pv_done(s), (uint32_t)((u - 1) & 1), abort_flag, p.status, 24)) return false;
                tc_fence_after();
                const uint32_t d = tmem_base + kColS + (uint32_t)s * kKN;
                const uint64_t b0 = dk[s];
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // 16 head-dimension elements per instruction
                    const uint64_t off = (uint64_t)(((ks >> 2) * kSlab + (ks & 3) * 32) >> 4);
                    umma_bf16_ts(d, tq + (uint32_t)ks * 8u, b0 + off, idesc_qk, ks != 0);
                    umma_bf16_ts(d, tq + 64u + (uint32_t)ks * 8u, b0 + off, idesc_qk, 1u);
                }
                umma_commit(s_full(s));
                return true;
            };
            if (ok) ok = issue_qk(0);
            for (int j = 0; ok && j < n_tiles; ++j) {
                if (j + 1 < n_tiles && !issue_qk(j + 1)) break;
                const int s = j & 1, u = j >> 1;
                const unsigned long long tr0 = NNC_TRACE_NOW();
                (void)tr0;
                if (!mbar_wait(p_full(s), (uint32_t)(u & 1), abort_flag, p.status, 25)) break;
                const unsigned long long tr1 = NNC_TRACE_NOW();
                (void)tr1;
                if (!mbar_wait(v_full(s), (uint32_t)(u & 1), abort_flag, p.status, 26)) break;
                tc_fence_after();
                const uint32_t d = tmem_base + kColO;
                const uint32_t pa = tmem_base + kColS + (uint32_t)s * kKN;   // P value in columns 0..63, residual in 64..127
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // 16 cache positions per instruction
                    const uint64_t b = dv[s] + (uint64_t)(ks * (2048 >> 4));
                    umma_bf16_ts(d, pa + (uint32_t)ks * 8u, b, idesc_pv, (j != 0) || (ks != 0));
                    umma_bf16_ts(d, pa + 64u + (uint32_t)ks * 8u, b, idesc_pv, 1u);
                }
                umma_commit(pv_done(s));
                if (blockIdx.x == 0) NNC_TRACE_EVENT(302, tr0, tr1, NNC_TRACE_NOW());
            }
        }
    } else {   // ---------------- softmax warps 2..9: two threads per query row ----------------
        const int quarter = warp & 3;                    // the TMEM lane quarter this warp may touch
        const int half = (warp - 2) >> 2;                // which 64 of a row's 128 columns this thread owns
        const int r = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int tok = q0 + r;
        const bool valid = tok < p.T;
        const int pos = p.n_past + tok;                  // absolute position of this row's query
        // the two warps of a quarter meet on their own named barrier (ids 2..5)
        auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(2 + quarter) : "memory"); };
        pdl_wait();
        {   // Q -> tensor memory, value + residual.  Both threads of a row read the whole head (the norm and the rotation
            // need all of it) and each writes its own half.
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
            // this thread's 64 elements: value pairs to columns 32 * half .. + 31 of the first block, residual pairs to
            // the same columns of the second
            const uint32_t tqw = tmem_base + lane_addr + kColQ + 32u * half;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                uint32_t qh[16], ql[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {   // compile-time indices on both sides keep q[] in registers; half is warp-uniform
                    const float a = valid ? (half ? q[64 + 32 * i + 2 * e] : q[32 * i + 2 * e]) * qscale : 0.f;
                    const float b = valid ? (half ? q[64 + 32 * i + 2 * e + 1] : q[32 * i + 2 * e + 1]) * qscale : 0.f;
                    qh[e] = pack_bf16x2(a, b);
                    ql[e] = pack_bf16x2(a - bf16_lo(qh[e]), b - bf16_hi(qh[e]));
                }
                tmem_st16(tqw + 16u * i, qh);
                tmem_st16(tqw + 64u + 16u * i, ql);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(q_ready);
        }
        float m_used = -INFINITY, l = 0.f;   // l: this thread's share of the row sum
        // A warp whose wait ran out goes `dead`: it touches nothing any more but keeps meeting its partner at every
        // pair barrier (one per tile and one at the end), so the partner can never be left waiting at one.
        bool dead = false;
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j & 1, u = j >> 1;
            const unsigned long long ts0 = NNC_TRACE_NOW();
            (void)ts0;
            if (!dead) dead = !__all_sync(0xffffffffu, mbar_wait(s_full(s), (uint32_t)(u & 1), abort_flag, p.status, 27));
            const unsigned long long ts1 = NNC_TRACE_NOW();
            (void)ts1;
            const uint32_t ts = tmem_base + lane_addr + kColS + (uint32_t)s * kKN;
            float sv[64];
            float m_tile = -INFINITY;
            if (!dead) {
                tc_fence_after();
                uint32_t t0[32], t1[32];
                tmem_ld32_nowait(ts + 64u * half, t0);
                tmem_ld32_nowait(ts + 64u * half + 32u, t1);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) { sv[e] = __uint_as_float(t0[e]); sv[32 + e] = __uint_as_float(t1[e]); }
                const int k0 = j * kKN + 64 * half;   // cache position of this thread's first column
                if (j * kKN + kKN - 1 > p.n_past + q0) {   // the tile reaches past the first row's position: causal mask
#pragma unroll
                    for (int e = 0; e < 64; ++e)
                        if (k0 + e > pos) sv[e] = -INFINITY;
                }
                // four independent chains: with two softmax warps per scheduler a 64-long dependent chain is not hidden
                float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int e = 0; e < 64; e += 4) {
                    mx[0] = fmaxf(mx[0], sv[e]); mx[1] = fmaxf(mx[1], sv[e + 1]);
                    mx[2] = fmaxf(mx[2], sv[e + 2]); mx[3] = fmaxf(mx[3], sv[e + 3]);
                }
                m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                xch[s][half][r] = m_tile;
            }
            // After this barrier both threads of a row hold their scores in registers, so the probability columns may
            // be written over the partner's score columns (value pairs of positions 64..127 land in columns 32..63,
            // residual pairs of positions 0..63 in columns 64..95).
            pair_sync();
            if (dead) continue;
            m_tile = fmaxf(m_tile, xch[s][half ^ 1][r]);
            if (j == 0) {
                m_used = m_tile;   // finite: position 0 is visible to every row
            } else {
                const bool need = m_tile > m_used + kLazyMax;   // the same verdict in both threads of the row
                if (__any_sync(0xffffffffu, need)) {
                    // O is rescaled in tensor memory (each thread its 64 columns); the product of the previous tile
                    // must have landed first
                    dead = !__all_sync(0xffffffffu, mbar_wait(pv_done((j - 1) & 1), (uint32_t)(((j - 1) >> 1) & 1), abort_flag, p.status, 28));
                    if (dead) continue;
                    tc_fence_after();
                    const float m_new = need ? m_tile : m_used;
                    const float alpha = exp2f(m_used - m_new);   // 1 for the rows that keep their maximum
                    const uint32_t to = tmem_base + lane_addr + kColO + 64u * half;
                    uint32_t t0[32], t1[32];
                    tmem_ld32_nowait(to, t0);
                    tmem_ld32_nowait(to + 32u, t1);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        t0[e] = __float_as_uint(__uint_as_float(t0[e]) * alpha);
                        t1[e] = __float_as_uint(__uint_as_float(t1[e]) * alpha);
                    }
                    tmem_st32(to, t0);
                    tmem_st32(to + 32u, t1);
                    tmem_wait_st();
                    l *= alpha;
                    m_used = m_new;
                }
            }
            // exponents are <= 2^8 by the lazy maximum; results below 2^-126 flush to zero, which a row sum >= 1 cannot see
            float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int e = 0; e < 64; e += 4) {
#pragma unroll
                for (int c = 0; c < 4; ++c) { sv[e + c] = ex2_approx(sv[e + c] - m_used); sum[c] += sv[e + c]; }
            }
            l += (sum[0] + sum[1]) + (sum[2] + sum[3]);
            // P over S: value pairs in columns 0..63, residual pairs in columns 64..127 (two positions per column);
            // this thread's 64 positions are columns 32 * half .. + 31 of each
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                uint32_t ph[16], pl[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    // value = the upper 16 bits of the fp32 pattern (truncation), residual = the upper 16 bits of
                    // what is left: byte permutes and two subtractions, nothing on the conversion pipe, which the
                    // exponentials keep busy.  value + residual still carries 15-16 bits of the probability.
                    const uint32_t a = __float_as_uint(sv[32 * i + 2 * e]), b = __float_as_uint(sv[32 * i + 2 * e + 1]);
                    ph[e] = __byte_perm(a, b, 0x7632);
                    const float ra = __uint_as_float(a) - __uint_as_float(a & 0xffff0000u);
                    const float rb = __uint_as_float(b) - __uint_as_float(b & 0xffff0000u);
                    pl[e] = __byte_perm(__float_as_uint(ra), __float_as_uint(rb), 0x7632);
                }
                tmem_st16(ts + 32u * half + 16u * i, ph);
                tmem_st16(ts + 64u + 32u * half + 16u * i, pl);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(p_full(s));
            if (blockIdx.x == 0 && warp == 2 && lane == 0) NNC_TRACE_EVENT(303, ts0, ts1, NNC_TRACE_NOW());
        }
        bool ok = !dead;
        // ---- O / l -> output: the pair adds its partial row sums, each thread writes its 64 columns ----
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(pv_done((n_tiles - 1) & 1), (uint32_t)(((n_tiles - 1) >> 1) & 1), abort_flag, p.status, 29));
        xch[n_tiles & 1][half][r] = l;   // the parity the last tile did not use
        pair_sync();
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / (l + xch[n_tiles & 1][half ^ 1][r]);
            const uint32_t to = tmem_base + lane_addr + kColO + 64u * half;
            const size_t oi = ((size_t)seq * p.T + (size_t)tok) * p.nq * kHeadDim + (size_t)h * kHeadDim + 64 * half;
#pragma unroll 1
            for (int i = 0; i < 2; ++i) {
                uint32_t t[32];
                tmem_ld32(to + 32u * i, t);
                if (!valid) continue;
                if (OUT_FP16) {
                    uint32_t o[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        o[e] = pack_f16x2_sat(__uint_as_float(t[2 * e]) * inv, __uint_as_float(t[2 * e + 1]) * inv);
                    uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<__half *>(p.out) + oi + 32 * i);
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
                    uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<bf16 *>(p.out) + oi + 32 * i);
#pragma unroll
                    for (int e = 0; e < 4; ++e) dst[e] = make_uint4(o[4 * e], o[4 * e + 1], o[4 * e + 2], o[4 * e + 3]);
                    if (p.out_lo) {
                        uint4 *dl = reinterpret_cast<uint4 *>(reinterpret_cast<bf16 *>(p.out_lo) + oi + 32 * i);
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
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

template <bool OUT_FP16>
cudaError_t launch_pf(const LaunchCtx &lc, const CUtensorMap &mk, const CUtensorMap &mv, const PfParams &p, dim3 grid) {
    auto kern = attn_prefill_tc_kernel<OUT_FP16>;
    static unsigned long long attr_done = 0;   // per instantiation, one bit per device
    if (cudaError_t e = ensure_dynamic_smem(kern, kPfSmem, &attr_done); e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kPfThreads);
    cfg.dynamicSmemBytes = kPfSmem;
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

// rows = batch * rows_per_seq new tokens, the token of row s * rows_per_seq + i sitting at position n_past + i of
// sequence s; the cache must already hold their K/V.  n_past is a host value: it sizes the tensor maps.
// kv_f16: kcache / vcache point at an fp16 image of the cache rows (same layout) and the kernel runs its one-term form.
cudaError_t launch_attn_prefill(const LaunchCtx &lc, const float *qkv, int rows, int rows_per_seq, const void *kcache,
                                const void *vcache, bool kv_f16, void *out, void *out_lo, bool out_fp16, int nq, int nkv,
                                int max_seq, int n_past, const AttnFused *fused) {
    const int batch = rows / rows_per_seq, T = rows_per_seq;
    if (T <= 0 || batch <= 0 || n_past < 0 || n_past + T > max_seq || nq % nkv) return cudaErrorInvalidValue;
    if (((uintptr_t)qkv | (uintptr_t)kcache | (uintptr_t)vcache | (uintptr_t)out | (uintptr_t)out_lo) & 15) return cudaErrorInvalidValue;
    CUtensorMap mk, mv;
    const int box_rows = kv_f16 ? 64 : kKN;   // the fp16 form walks the cache in steps of 64 positions
    if (!make_cache_map(&mk, kcache, batch * nkv, n_past + T, max_seq, kv_f16, box_rows) ||
        !make_cache_map(&mv, vcache, batch * nkv, n_past + T, max_seq, kv_f16, box_rows))
        return cudaErrorInvalidValue;
    PfParams p;
    p.qkv = qkv; p.row_stride = (nq + 2 * nkv) * kHeadDim; p.out = out; p.out_lo = out_lo;
    p.T = T; p.n_past = n_past; p.nq = nq; p.nkv = nkv; p.status = lc.status;
    p.g_q = fused ? fused->g_q : nullptr; p.rope = fused ? fused->rope : nullptr; p.eps = fused ? fused->eps : 0.f;
    p.batch = batch; p.n_qt = (T + kQM - 1) / kQM;
    const dim3 grid((unsigned)(p.n_qt * nq * batch));
    if (kv_f16) return launch_attn_prefill_f16(lc, mk, mv, p, grid, out_fp16);
    return out_fp16 ? launch_pf<true>(lc, mk, mv, p, grid) : launch_pf<false>(lc, mk, mv, p, grid);
}

}  // namespace nnc
