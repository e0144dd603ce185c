// Body of the GQA split-K flash-decode (see attn_decode.cu for the design): one 4-warp group handles one
// (sequence, KV head, position range) and synchronises on a named barrier of its own, so the body can be placed
// in kernels that hold other warps besides the group.
#pragma once
#include "common.cuh"
#include "nnc_internal.h"

namespace nnc {

constexpr int kPartStride = kHeadDim + 4;  // o~[128], m, l, 2 pad words (rows stay 16-byte aligned)
constexpr int kAttnWarps = 4;
constexpr int kSingleRange = 128;    // contexts up to this length are handled by one CTA per KV head
constexpr int kPrefetchAhead = 3;   // blocks of 16 positions, per warp: far enough to cover DRAM latency; much further and a
                                    // batch of long contexts keeps more prefetched lines in flight than L2 holds on to

__device__ __forceinline__ uint4 ldg_cg(const void *p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void mma_bf16_full(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                              uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// transposes an 8x8 matrix of 16-bit elements held one row per 4 lanes (lane l: row l / 4, columns 2 (l % 4), + 1)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t r;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(x));
    return r;
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

// value + residual bf16 pairs of two floats: hi holds bf16(x), lo holds bf16(x - hi)
__device__ __forceinline__ void split2(float x, float y, uint32_t &hi, uint32_t &lo) {
    hi = pack_bf16x2(x, y);
    lo = pack_bf16x2(x - bf16_lo(hi), y - bf16_hi(hi));
}

struct AttnParams {
    const float *q;          // [batch][q_row_stride]: query heads first; FUSED: then key heads, then value heads (raw)
    int q_row_stride;
    bf16 *kcache, *vcache;   // this layer: [batch][nkv][max_seq][128]
    float *out_f32;          // [batch][out_row_stride] or null
    bf16 *out_bf16, *out_bf16_lo;
    int out_row_stride;
    float *part;
    size_t part_floats;      // floats behind `part` (what the checked build compares the partial slots with)
    uint32_t *tickets;
    const int32_t *d_len;    // cached positions before this call (null = 0)
    int len_add;             // positions attended = *d_len + len_add
    int nkv, max_seq, n_splits;
    const bf16 *g_q, *g_k;   // FUSED: per-head RMSNorm gains
    const float *rope;       // FUSED: [max_seq][64][2]
    float eps;
};

// RMSNorm over the 128 elements of one head + rotation by the table row; lane l owns elements 2l, 2l+1 and their
// rotation partners 2l+64, 2l+65 (half-split pairing).
__device__ __forceinline__ void norm_rope(float2 &a, float2 &b, const bf16 *gain, const float *rope_row, float eps, int lane) {
    const float ss = warp_sum(a.x * a.x + a.y * a.y + b.x * b.x + b.y * b.y);
    const float inv = rsqrtf(ss * (1.f / kHeadDim) + eps);
    const uint32_t ga = reinterpret_cast<const uint32_t *>(gain)[lane];
    const uint32_t gb = reinterpret_cast<const uint32_t *>(gain + 64)[lane];
    a.x *= inv * bf16_lo(ga); a.y *= inv * bf16_hi(ga);
    b.x *= inv * bf16_lo(gb); b.y *= inv * bf16_hi(gb);
    const float4 cs = reinterpret_cast<const float4 *>(rope_row)[lane];  // c0 s0 c1 s1
    const float2 ra = make_float2(a.x * cs.x - b.x * cs.y, a.y * cs.z - b.y * cs.w);
    const float2 rb = make_float2(b.x * cs.x + a.x * cs.y, b.y * cs.z + a.y * cs.w);
    a = ra; b = rb;
}


template <int G>
struct AttnSmem {
    __align__(16) float qs[G][kHeadDim];             // processed queries, pre-scaled for exp2
    float comb[kAttnWarps][G][kPartStride];          // per-warp (o~, m, l); reused for the combine weights
    bool is_last;
};

__device__ __forceinline__ void attn_group_sync(int bar_id) {
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(kAttnWarps * 32) : "memory");
}

// tid = thread index inside the group (0..127).  Everything that reads the new token's projections or the cache
// length must come after the caller has waited on their producer.
template <int G, bool FUSED>
__device__ __forceinline__ void attn_decode_body(const AttnParams &p, int split, int j, int b, int tid, AttnSmem<G> &sm,
                                                 int bar_id) {
    constexpr int kWarps = kAttnWarps;
    const int warp = tid >> 5, lane = tid & 31;
    const int g8 = lane >> 2, t4 = lane & 3;   // fragment coordinates: row / column group, and position inside it
    const int nq = p.nkv * G;
    const size_t head_off = ((size_t)b * p.nkv + j) * (size_t)p.max_seq * kHeadDim;
    bf16 *kbase = p.kcache + head_off;
    bf16 *vbase = p.vcache + head_off;
    const int n_ctx = (p.d_len ? *p.d_len : 0) + p.len_add;
    int chunk = (n_ctx + p.n_splits - 1) / p.n_splits;
    chunk = (chunk + 15) & ~15;
    if (chunk < 16) chunk = 16;
    if (n_ctx <= kSingleRange) chunk = kSingleRange;   // short context: one CTA per KV head, no partials
    const int c0 = split * chunk;
    const int c1 = min(c0 + chunk, n_ctx);
    const int n_active = (n_ctx + chunk - 1) / chunk;
    if (c0 >= n_ctx) return;  // whole CTA; takes no ticket (n_active counts only non-empty ranges)
    if (!NNC_BC(n_ctx >= 1 && n_ctx <= p.max_seq, 3001)) return;   // the host checks the capacity before it launches

    // ---- K/V fragment loads of one block of 16 positions: K rows p0 + 8h + g8 (h = 0, 1), V rows
    //      p0 + {2 t4, 2 t4 + 1, 2 t4 + 8, 2 t4 + 9}; rows past the range are clamped here and masked later ----
    // two register buffers: the warp's next block is in flight while it works on the current one
    uint4 kfa[2][4], vfa[4][2], kfb[2][4], vfb[4][2];
    auto load_block = [&](uint4 (&kf)[2][4], uint4 (&vf)[4][2], int p0) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int pos = min(p0 + 8 * h + g8, c1 - 1);
            const bf16 *kr = kbase + (size_t)pos * kHeadDim + 8 * t4;
#pragma unroll
            for (int c = 0; c < 4; ++c) kf[h][c] = ldg_cg(kr + 32 * c);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int pos = min(p0 + 2 * t4 + (r & 1) + 8 * (r >> 1), c1 - 1);
            const bf16 *vr = vbase + (size_t)pos * kHeadDim + 8 * g8;
            vf[r][0] = ldg_cg(vr);
            vf[r][1] = ldg_cg(vr + 64);
        }
    };
    const int n_blocks = (c1 - c0 + 15) >> 4;
    // the warp's first block is requested now and lands while the queries are prepared -- unless it holds the row
    // that is appended below
    const bool early = warp < n_blocks && !(FUSED && c0 + warp * 16 + 16 >= n_ctx);
    if (early) load_block(kfa, vfa, c0 + warp * 16);
    // ... and so is its second block, into the other register buffer
    const bool early2 = warp + kWarps < n_blocks && !(FUSED && c0 + (warp + kWarps) * 16 + 16 >= n_ctx);
    if (early2) load_block(kfb, vfb, c0 + (warp + kWarps) * 16);

    // ---- queries (and, fused, the new token's K/V row) ----
    const float qscale = 1.4426950408889634f * rsqrtf((float)kHeadDim);   // scores in log2 units
    const float *qrow = p.q + (size_t)b * p.q_row_stride;
    for (int g = warp; g < G; g += kWarps) {
        const float *src = qrow + (size_t)(j * G + g) * kHeadDim;
        float2 a = __ldcg(reinterpret_cast<const float2 *>(src) + lane);   // L2: written earlier by other SMs
        float2 c = __ldcg(reinterpret_cast<const float2 *>(src + 64) + lane);
        if (FUSED) norm_rope(a, c, p.g_q, p.rope + (size_t)(n_ctx - 1) * kHeadDim, p.eps, lane);
        reinterpret_cast<float2 *>(&sm.qs[g][0])[lane] = make_float2(a.x * qscale, a.y * qscale);
        reinterpret_cast<float2 *>(&sm.qs[g][64])[lane] = make_float2(c.x * qscale, c.y * qscale);
    }
    if (FUSED && split == n_active - 1) {
        // this CTA's range ends with the new position: normalise + rotate its key, round both rows to bf16, append
        const int pos = n_ctx - 1;
        if (warp == (G % kWarps)) {
            const float *src = qrow + (size_t)(nq + j) * kHeadDim;
            float2 a = __ldcg(reinterpret_cast<const float2 *>(src) + lane);   // L2: written earlier by other SMs
            float2 c = __ldcg(reinterpret_cast<const float2 *>(src + 64) + lane);
            norm_rope(a, c, p.g_k, p.rope + (size_t)pos * kHeadDim, p.eps, lane);
            bf16 *dst = kbase + (size_t)pos * kHeadDim;
            reinterpret_cast<uint32_t *>(dst)[lane] = pack_bf16x2(a.x, a.y);
            reinterpret_cast<uint32_t *>(dst + 64)[lane] = pack_bf16x2(c.x, c.y);
        }
        if (warp == ((G + 1) % kWarps)) {
            const float *src = qrow + (size_t)(nq + p.nkv + j) * kHeadDim;
            const float4 v = __ldcg(reinterpret_cast<const float4 *>(src) + lane);
            bf16 *dst = vbase + (size_t)pos * kHeadDim;
            reinterpret_cast<uint2 *>(dst)[lane] = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
        }
        __threadfence_block();
    }
    attn_group_sync(bar_id);

    // ---- Q^T fragments (the 8-column operand): column g8 is a query head (zero beyond G); contraction step
    //      s = 2c + e covers the head-dimension elements 8 (4c + t4) + 4e + {0,1} (first half of the step) and
    //      + {2,3} (second half), the same elements the K chunk c of this lane holds ----
    uint32_t qh[8][2], ql[8][2];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        float4 lo4 = make_float4(0.f, 0.f, 0.f, 0.f), hi4 = lo4;
        if (g8 < G) {
            lo4 = *reinterpret_cast<const float4 *>(&sm.qs[g8 < G ? g8 : 0][8 * (4 * c + t4)]);
            hi4 = *reinterpret_cast<const float4 *>(&sm.qs[g8 < G ? g8 : 0][8 * (4 * c + t4) + 4]);
        }
        split2(lo4.x, lo4.y, qh[2 * c][0], ql[2 * c][0]);
        split2(lo4.z, lo4.w, qh[2 * c][1], ql[2 * c][1]);
        split2(hi4.x, hi4.y, qh[2 * c + 1][0], ql[2 * c + 1][0]);
        split2(hi4.z, hi4.w, qh[2 * c + 1][1], ql[2 * c + 1][1]);
    }

    // O^T tile i: rows are head-dimension elements 8 g8 + i ([0], [1]) and 64 + 8 g8 + i ([2], [3]); columns are the
    // query heads 2 t4 ([0], [2]) and 2 t4 + 1 ([1], [3])
    float o[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    // per head 2 t4 + e: running maximum (identical across the 8 lanes that share t4) and this lane's partial sum
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

    auto process_block = [&](const uint4 (&kf)[2][4], const uint4 (&vf)[4][2], int p0) {
        // long ranges: ask L2 for the block this warp will reach kPrefetchAhead iterations from now (16 rows of K and
        // of V, 4 KB each, contiguous), so that the fragment loads above find their rows in L2
        {
            const int pf = p0 + kPrefetchAhead * kWarps * 16;
            if (lane < 2 && pf + 16 <= c1) {
                const bf16 *src = (lane ? vbase : kbase) + (size_t)pf * kHeadDim;
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(16u * kHeadDim * 2u) : "memory");
            }
        }
        // ---- scores, transposed: S^T = K Q^T; s[0], s[1] = position p0 + g8, heads 2 t4, 2 t4 + 1;
        //      s[2], s[3] = position p0 + 8 + g8 ----
        float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            mma_bf16_full(s, kf[0][c].x, kf[1][c].x, kf[0][c].y, kf[1][c].y, qh[2 * c][0], qh[2 * c][1]);
            mma_bf16_full(s, kf[0][c].x, kf[1][c].x, kf[0][c].y, kf[1][c].y, ql[2 * c][0], ql[2 * c][1]);
            mma_bf16_full(s, kf[0][c].z, kf[1][c].z, kf[0][c].w, kf[1][c].w, qh[2 * c + 1][0], qh[2 * c + 1][1]);
            mma_bf16_full(s, kf[0][c].z, kf[1][c].z, kf[0][c].w, kf[1][c].w, ql[2 * c + 1][0], ql[2 * c + 1][1]);
        }
        if (p0 + g8 >= c1) s[0] = s[1] = -INFINITY;
        if (p0 + 8 + g8 >= c1) s[2] = s[3] = -INFINITY;
        float pr[4], alpha[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            float mx = fmaxf(s[e], s[e + 2]);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
            const float m_new = fmaxf(m_run[e], mx);        // finite: the block holds at least one valid position
            alpha[e] = exp2f(m_run[e] - m_new);             // 0 on the first block
            pr[e] = exp2f(s[e] - m_new);
            pr[e + 2] = exp2f(s[e + 2] - m_new);
            l_run[e] = l_run[e] * alpha[e] + (pr[e] + pr[e + 2]);
            m_run[e] = m_new;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) { o[i][0] *= alpha[0]; o[i][1] *= alpha[1]; o[i][2] *= alpha[0]; o[i][3] *= alpha[1]; }
        // ---- P^T fragments (contraction index = position inside the block), as value + residual: the 8x8 blocks
        //      (position, head) this lane holds a row of are transposed across the warp, after which this lane holds
        //      head g8, positions 2 t4, 2 t4 + 1 (first block) and 2 t4 + 8, 2 t4 + 9 (second block) ----
        uint32_t ph0, pl0, ph1, pl1;
        split2(pr[0], pr[1], ph0, pl0);
        split2(pr[2], pr[3], ph1, pl1);
        ph0 = movmatrix_trans(ph0); pl0 = movmatrix_trans(pl0);
        ph1 = movmatrix_trans(ph1); pl1 = movmatrix_trans(pl1);
        // ---- O^T += V^T P^T ----
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t sel = (i & 1) ? 0x7632u : 0x5410u;
            const uint32_t a0 = prmt((&vf[0][0].x)[i >> 1], (&vf[1][0].x)[i >> 1], sel);
            const uint32_t a1 = prmt((&vf[0][1].x)[i >> 1], (&vf[1][1].x)[i >> 1], sel);
            const uint32_t a2 = prmt((&vf[2][0].x)[i >> 1], (&vf[3][0].x)[i >> 1], sel);
            const uint32_t a3 = prmt((&vf[2][1].x)[i >> 1], (&vf[3][1].x)[i >> 1], sel);
            mma_bf16_full(o[i], a0, a1, a2, a3, ph0, ph1);
            mma_bf16_full(o[i], a0, a1, a2, a3, pl0, pl1);
        }
    };
    {
        int blk = warp;
        if (blk < n_blocks && !early) load_block(kfa, vfa, c0 + blk * 16);
        bool have_b = early2;   // the second buffer already holds (or is receiving) the block after this one
        while (blk < n_blocks) {
            if (blk + kWarps < n_blocks && !have_b) load_block(kfb, vfb, c0 + (blk + kWarps) * 16);
            have_b = false;
            process_block(kfa, vfa, c0 + blk * 16);
            blk += kWarps;
            if (blk >= n_blocks) break;
            if (blk + kWarps < n_blocks) load_block(kfa, vfa, c0 + (blk + kWarps) * 16);
            process_block(kfb, vfb, c0 + blk * 16);
            blk += kWarps;
        }
    }

    // ---- merge the warps: (o~, m, l) per query head into shared memory, then one partial per CTA ----
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 4);
        l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 8);
        l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 16);
    }
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int head = 2 * t4 + e;
        if (head < G) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                sm.comb[warp][head][8 * g8 + i] = o[i][e];
                sm.comb[warp][head][64 + 8 * g8 + i] = o[i][2 + e];
            }
            if (g8 == 0) { sm.comb[warp][head][kHeadDim] = m_run[e]; sm.comb[warp][head][kHeadDim + 1] = l_run[e]; }
        }
    }
    attn_group_sync(bar_id);

    float *my_part = p.part + (((size_t)b * nq + (size_t)j * G) * p.n_splits + split) * kPartStride;
    if (n_active > 1 &&
        !NNC_BC((((size_t)b * nq + (size_t)j * G + (G - 1)) * p.n_splits + split + 1) * kPartStride <= p.part_floats, 3002))
        return;
    // partial for head g lives at my_part + g * n_splits * kPartStride
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm.comb[w][g][kHeadDim]);
        float L = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float sc = exp2f(sm.comb[w][g][kHeadDim] - M);   // 0 for a warp that had no block
            L = fmaf(sc, sm.comb[w][g][kHeadDim + 1], L);
            acc = fmaf(sc, sm.comb[w][g][tid], acc);
        }
        if (n_active == 1) {
            // the only range of this head: no partial, no ticket -- the same arithmetic the combine would do
            const float r = acc * (1.f / L);
            const size_t oi = (size_t)b * p.out_row_stride + (size_t)(j * G + g) * kHeadDim + tid;
            if (p.out_f32) p.out_f32[oi] = r;
            if (p.out_bf16) {
                const bf16 hi = __float2bfloat16_rn(r);
                p.out_bf16[oi] = hi;
                if (p.out_bf16_lo) p.out_bf16_lo[oi] = __float2bfloat16_rn(r - __bfloat162float(hi));
            }
            continue;
        }
        float *pp = my_part + (size_t)g * p.n_splits * kPartStride;
        pp[tid] = acc;
        if (tid == 0) { pp[kHeadDim] = M; pp[kHeadDim + 1] = L; }
    }
    if (n_active == 1) return;
    __threadfence();
    attn_group_sync(bar_id);
    if (tid == 0) {
        const unsigned tk = atomicAdd(&p.tickets[b * p.nkv + j], 1u);
        sm.is_last = (tk == (unsigned)n_active - 1);
    }
    attn_group_sync(bar_id);
    if (!sm.is_last) return;
    __threadfence();
    // ---- combine (last CTA of this sequence / KV head): o = sum_c 2^(m_c - M) o~_c / sum_c 2^(m_c - M) l_c.
    //      The splits are folded in split order, whichever CTA arrived last. ----
    float (*wgt)[kAttnMaxSplits] = reinterpret_cast<float (*)[kAttnMaxSplits]>(&sm.comb[0][0][0]);   // [G][kAttnMaxSplits], reuses comb
    const float *pbase = p.part + (((size_t)b * nq + (size_t)j * G) * p.n_splits) * kPartStride;
    // One warp per head, 4 output elements per lane.  The (m, l) words and the first batch of partial rows are all
    // requested before anything is waited for, so the whole combine costs one memory round trip; the weights of a
    // head are produced and consumed by the same warp (a warp barrier suffices).
    constexpr int kBatch = 40;
    for (int g = warp; g < G; g += kWarps) {
        const float *pp = pbase + (size_t)g * p.n_splits * kPartStride;
        const float *pv = pp + 4 * lane;
        float mv[2], lv[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int c = lane + 32 * u;
            mv[u] = c < n_active ? __ldcg(pp + (size_t)c * kPartStride + kHeadDim) : -INFINITY;
            lv[u] = c < n_active ? __ldcg(pp + (size_t)c * kPartStride + kHeadDim + 1) : 0.f;
        }
        float4 v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
            v[u] = (u < n_active) ? __ldcg(reinterpret_cast<const float4 *>(pv + (size_t)u * kPartStride)) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float M = warp_max(fmaxf(mv[0], mv[1]));
        const float w0 = exp2f(mv[0] - M), w1 = exp2f(mv[1] - M);
        wgt[g][lane] = w0;
        wgt[g][lane + 32] = w1;
        // fixed summation order over the splits: lane partials, then the shuffle tree
        const float il = 1.f / warp_sum(fmaf(w0, lv[0], w1 * lv[1]));
        __syncwarp();
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const float w = (u < n_active) ? wgt[g][u] : 0.f;
            acc.x = fmaf(w, v[u].x, acc.x); acc.y = fmaf(w, v[u].y, acc.y);
            acc.z = fmaf(w, v[u].z, acc.z); acc.w = fmaf(w, v[u].w, acc.w);
        }
        for (int c = kBatch; c < n_active; ++c) {   // split counts beyond one batch (up to kAttnMaxSplits)
            const float4 x = __ldcg(reinterpret_cast<const float4 *>(pv + (size_t)c * kPartStride));
            const float w = wgt[g][c];
            acc.x = fmaf(w, x.x, acc.x); acc.y = fmaf(w, x.y, acc.y); acc.z = fmaf(w, x.z, acc.z); acc.w = fmaf(w, x.w, acc.w);
        }
        const float4 r = make_float4(acc.x * il, acc.y * il, acc.z * il, acc.w * il);
        const size_t oi = (size_t)b * p.out_row_stride + (size_t)(j * G + g) * kHeadDim + 4 * lane;
        if (p.out_f32) *reinterpret_cast<float4 *>(p.out_f32 + oi) = r;
        if (p.out_bf16) {
            const uint2 hi = make_uint2(pack_bf16x2(r.x, r.y), pack_bf16x2(r.z, r.w));
            *reinterpret_cast<uint2 *>(p.out_bf16 + oi) = hi;
            if (p.out_bf16_lo)
                *reinterpret_cast<uint2 *>(p.out_bf16_lo + oi) =
                    make_uint2(pack_bf16x2(r.x - bf16_lo(hi.x), r.y - bf16_hi(hi.x)), pack_bf16x2(r.z - bf16_lo(hi.y), r.w - bf16_hi(hi.y)));
        }
    }
    if (tid == 0) p.tickets[b * p.nkv + j] = 0u;
}

}  // namespace nnc
