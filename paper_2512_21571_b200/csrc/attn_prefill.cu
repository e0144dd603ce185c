// Causal attention for a block of new tokens (the prompt phase): the query at position p attends to cache
// positions 0..p of its sequence.  K and V are read from the bf16 cache, which already holds the new tokens.
//
// Flash-attention on the warp-level tensor-core path (mma.sync m16n8k16, bf16 in, fp32 accumulate):
//   - grid (query tiles of 128 positions, query heads, sequences), 8 warps; a warp owns 16 query rows and keeps
//     its Q fragments, the running (m, l) and the 16 x 128 output accumulator in registers;
//   - K/V tiles of 64 cache positions are staged in shared memory with cp.async (16 bytes per thread, XOR-swizzled
//     chunks so that ldmatrix is conflict-free), double-buffered: the next tile streams in while the current one
//     is multiplied.  The G query heads that share a KV head run in different CTAs and meet in L2;
//   - Q and the probabilities are fed as two bf16 terms each (value + rounding residual), so the products keep
//     fp32-level accuracy (a single bf16 term costs ~2^-9 per operand, which the parity bar does not allow);
//   - only the tiles on the diagonal apply the causal mask; query tiles are issued longest first.
#include "common.cuh"
#include "nnc_internal.h"

namespace nnc {

namespace {

constexpr int kBM = 128;   // query rows per CTA
constexpr int kBN = 64;    // cache positions per tile
constexpr int kPfWarps = 8;
constexpr int kTileBytes = kBN * kHeadDim * 2;   // 16 KB

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// value + residual bf16 pairs of two floats
__device__ __forceinline__ void split_pair(float x, float y, uint32_t &hi, uint32_t &lo) {
    hi = pack_bf16x2(x, y);
    lo = pack_bf16x2(x - bf16_lo(hi), y - bf16_hi(hi));
}

// byte offset of 16-byte chunk `chunk` (0..15) of row `row` inside a [kBN][128] bf16 tile, XOR-swizzled
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
    return (uint32_t)(row * 256 + ((chunk ^ (row & 7)) << 4));
}

// cp.async of one K and one V tile (cache positions k0 .. k0 + 63, clamped to the last valid row) into a stage
__device__ __forceinline__ void load_tile(uint32_t stage_base, const bf16 *kbase, const bf16 *vbase, int k0, int last_row,
                                          int tid) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int idx = tid + 256 * i;          // 1024 chunks of 16 bytes per tile
        const int row = idx >> 4, chunk = idx & 15;
        const size_t src = (size_t)min(k0 + row, last_row) * kHeadDim + chunk * 8;
        cp_async16(stage_base + tile_off(row, chunk), kbase + src);
        cp_async16(stage_base + kTileBytes + tile_off(row, chunk), vbase + src);
    }
}

__global__ void __launch_bounds__(kPfWarps * 32, 1)
attn_prefill_kernel(const float *__restrict__ qkv, int rows_per_seq, const bf16 *__restrict__ kcache,
                    const bf16 *__restrict__ vcache, bf16 *__restrict__ out, bf16 *__restrict__ out_lo, int nq, int nkv,
                    int max_seq, const int32_t *__restrict__ d_len) {
    extern __shared__ __align__(128) uint8_t pf_smem[];   // 2 stages x (K tile, V tile)
    pdl_wait();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int qt = gridDim.x - 1 - blockIdx.x;   // longest rows first
    const int h = blockIdx.y, seq = blockIdx.z;
    const int T = rows_per_seq, P0 = *d_len;
    const int G = nq / nkv, j = h / G, heads = nq + 2 * nkv;
    const int q0 = qt * kBM;
    const int r0 = q0 + warp * 16 + g, r1 = r0 + 8;   // this thread's two query rows (token index inside the call)

    // ---- Q fragments (pre-scaled so that exp2 can be used), as value + residual ----
    const float qscale = 1.4426950408889634f * rsqrtf((float)kHeadDim);
    uint32_t qh[8][4], ql[8][4];
    {
        const float *qa = qkv + ((size_t)seq * T + min(r0, T - 1)) * heads * kHeadDim + (size_t)h * kHeadDim;
        const float *qb = qkv + ((size_t)seq * T + min(r1, T - 1)) * heads * kHeadDim + (size_t)h * kHeadDim;
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const float2 a0 = *reinterpret_cast<const float2 *>(qa + 16 * s + 2 * t);
            const float2 a2 = *reinterpret_cast<const float2 *>(qa + 16 * s + 2 * t + 8);
            const float2 a1 = *reinterpret_cast<const float2 *>(qb + 16 * s + 2 * t);
            const float2 a3 = *reinterpret_cast<const float2 *>(qb + 16 * s + 2 * t + 8);
            split_pair(a0.x * qscale, a0.y * qscale, qh[s][0], ql[s][0]);
            split_pair(a1.x * qscale, a1.y * qscale, qh[s][1], ql[s][1]);
            split_pair(a2.x * qscale, a2.y * qscale, qh[s][2], ql[s][2]);
            split_pair(a3.x * qscale, a3.y * qscale, qh[s][3], ql[s][3]);
        }
    }

    // cache positions the last row of this tile may see; never past the head's slab, whatever the caller put in *d_len
    const int n_keys = min(min(P0 + q0 + kBM, P0 + T), max_seq);
    const int n_tiles = (n_keys + kBN - 1) / kBN;
    const size_t head_off = ((size_t)seq * nkv + j) * (size_t)max_seq * kHeadDim;
    const bf16 *kbase = kcache + head_off, *vbase = vcache + head_off;
    const uint32_t smem0 = smem_addr(pf_smem);

    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // rows r0, r1; l is a per-lane partial

    load_tile(smem0, kbase, vbase, 0, n_keys - 1, tid);
    cp_async_commit();

    for (int kt = 0; kt < n_tiles; ++kt) {
        const uint32_t st = smem0 + (uint32_t)(kt & 1) * 2u * kTileBytes;
        if (kt + 1 < n_tiles) {
            load_tile(smem0 + (uint32_t)((kt + 1) & 1) * 2u * kTileBytes, kbase, vbase, (kt + 1) * kBN, n_keys - 1, tid);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const int k0 = kt * kBN;
        const int row_lo = P0 + q0 + warp * 16;           // absolute position of this warp's first query row
        if (k0 <= row_lo + 15) {                          // warp-uniform: the tile holds something this warp may see
            // ---- S = Q K^T over the 64 positions of the tile ----
            float sacc[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
#pragma unroll
            for (int s = 0; s < 8; ++s) {
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    uint32_t kb[4];
                    const int mi = lane >> 3;
                    ldsm_x4(kb, st + tile_off(16 * np + (mi >> 1) * 8 + (lane & 7), 2 * s + (mi & 1)));
                    mma16816(sacc[2 * np], qh[s], kb[0], kb[1]);
                    mma16816(sacc[2 * np], ql[s], kb[0], kb[1]);
                    mma16816(sacc[2 * np + 1], qh[s], kb[2], kb[3]);
                    mma16816(sacc[2 * np + 1], ql[s], kb[2], kb[3]);
                }
            }
            // ---- causal mask (diagonal tiles only), online softmax ----
            if (k0 + kBN - 1 > row_lo) {
#pragma unroll
                for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int kabs = k0 + nt * 8 + 2 * t + e;
                        if (kabs > P0 + r0) sacc[nt][e] = -INFINITY;
                        if (kabs > P0 + r1) sacc[nt][2 + e] = -INFINITY;
                    }
            }
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                mx0 = fmaxf(mx0, fmaxf(sacc[nt][0], sacc[nt][1]));
                mx1 = fmaxf(mx1, fmaxf(sacc[nt][2], sacc[nt][3]));
            }
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);   // finite from the first tile on (key 0 is visible)
            const float al0 = exp2f(m0 - mn0), al1 = exp2f(m1 - mn1);
            m0 = mn0; m1 = mn1;
            float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                sacc[nt][0] = exp2f(sacc[nt][0] - mn0); sacc[nt][1] = exp2f(sacc[nt][1] - mn0);
                sacc[nt][2] = exp2f(sacc[nt][2] - mn1); sacc[nt][3] = exp2f(sacc[nt][3] - mn1);
                sum0 += sacc[nt][0] + sacc[nt][1];
                sum1 += sacc[nt][2] + sacc[nt][3];
            }
            l0 = l0 * al0 + sum0; l1 = l1 * al1 + sum1;
#pragma unroll
            for (int i = 0; i < 16; ++i) { o[i][0] *= al0; o[i][1] *= al0; o[i][2] *= al1; o[i][3] *= al1; }
            // ---- O += P V ----
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                uint32_t ph[4], pl[4];
                split_pair(sacc[2 * kk][0], sacc[2 * kk][1], ph[0], pl[0]);
                split_pair(sacc[2 * kk][2], sacc[2 * kk][3], ph[1], pl[1]);
                split_pair(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1], ph[2], pl[2]);
                split_pair(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3], ph[3], pl[3]);
#pragma unroll
                for (int dp = 0; dp < 8; ++dp) {
                    uint32_t vb[4];
                    const int mi = lane >> 3;
                    ldsm_x4_trans(vb, st + kTileBytes + tile_off(16 * kk + (mi & 1) * 8 + (lane & 7), 2 * dp + (mi >> 1)));
                    mma16816(o[2 * dp], ph, vb[0], vb[1]);
                    mma16816(o[2 * dp], pl, vb[0], vb[1]);
                    mma16816(o[2 * dp + 1], ph, vb[2], vb[3]);
                    mma16816(o[2 * dp + 1], pl, vb[2], vb[3]);
                }
            }
        }
        __syncthreads();   // the other stage is refilled at the top of the next iteration
    }

    // ---- normalise and store as value + residual bf16 ----
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float i0 = 1.f / l0, i1 = 1.f / l1;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int r = half ? r1 : r0;
        if (r >= T) continue;
        const float inv = half ? i1 : i0;
        const size_t base = ((size_t)seq * T + r) * nq * kHeadDim + (size_t)h * kHeadDim + 2 * t;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            uint32_t hi, lo;
            split_pair(o[nt][2 * half] * inv, o[nt][2 * half + 1] * inv, hi, lo);
            *reinterpret_cast<uint32_t *>(out + base + nt * 8) = hi;
            if (out_lo) *reinterpret_cast<uint32_t *>(out_lo + base + nt * 8) = lo;
        }
    }
}

}  // namespace

cudaError_t launch_attn_prefill(const LaunchCtx &lc, const float *qkv, int rows, int rows_per_seq, const bf16 *kcache,
                                const bf16 *vcache, bf16 *out, bf16 *out_lo, int nq, int nkv, int max_seq,
                                const int32_t *d_len) {
    static unsigned long long attr_done = 0;   // one bit per device
    const int smem = 4 * kTileBytes;
    if (cudaError_t e = ensure_dynamic_smem(attn_prefill_kernel, smem, &attr_done); e != cudaSuccess) return e;
    const int batch = rows / rows_per_seq;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((rows_per_seq + kBM - 1) / kBM, nq, batch);
    cfg.blockDim = dim3(kPfWarps * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = lc.stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = lc.pdl ? 1 : 0;
    if (lc.launches) ++*lc.launches;
    return cudaLaunchKernelEx(&cfg, attn_prefill_kernel, qkv, rows_per_seq, kcache, vcache, out, out_lo, nq, nkv, max_seq, d_len);
}

}  // namespace nnc
