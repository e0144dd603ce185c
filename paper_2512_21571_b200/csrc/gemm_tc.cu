// Tensor-core GEMM for the prompt phase and batched decode:  Y[T][N] = X[T][K] * W[N][K]^T, bf16 operands,
// fp32 accumulation in tensor memory (tcgen05 / TMEM), hand-written PTX.
//
// Structure (one persistent CTA per SM, 192 threads):
//   warp 0      TMA producer: streams 128-row x 64-column (128-byte, 128B-swizzled) operand tiles into a
//               shared-memory ring, one mbarrier per stage
//   warp 1      MMA issuer: one elected lane issues tcgen05.mma (M=128, N=BN, K=16) four times per stage and
//               commits the stage back to the producer; accumulators alternate between two TMEM buffers
//   warps 2-5   epilogue: tcgen05.ld 32 columns at a time, apply the epilogue, store; runs concurrently with
//               the main loop of the next tile thanks to the second accumulator
// Two operand assignments share the code: tokens on the M side (prefill; weights are the N operand, BN=256)
// or weights on the M side ("swap", used when there are few tokens, e.g. a decode batch of 32: weights fill
// the 128 TMEM lanes and the tokens are the narrow N operand, so no tensor-core work is wasted on padding).
// Operand types: bf16 (activations optionally as value + rounding residual, two MMAs per weight tile) or fp16 (one
// term; the weights are then an fp16 copy scaled by a power of two, undone by `out_scale` in the epilogue).  A and B
// of one tcgen05.mma always have the same type.
// Every mbarrier wait is bounded by a wall-clock limit; on expiry the CTA raises an abort flag, records a
// status word for the host, drains and frees its TMEM.
#include "tc_common.cuh"

namespace nnc {

namespace {

constexpr int kBM = 128;
constexpr int kBK = 64;
constexpr int kGemmThreads = 192;

struct GemmParams {
    void *Y;          // output
    void *Y_lo;       // SwiGLU epilogue only: bf16 rounding residual of Y (nullable)
    int T, N, K;      // tokens, weight rows, reduction
    int ldy;          // output row stride in elements
    int m_tiles, n_tiles;
    int stream;          // 1: the (tile, K stage) space is cut into one contiguous range per CTA (SWAP only)
    float *part;         // stream: fp32 partial tiles [CTA][first / last segment][BN / 32][8][128 rows][4]
    uint32_t *tickets;   // stream: one "piece parked" flag per partial-tile slot, zero at rest
    size_t part_bytes;   // stream: bytes behind `part`
    const float *out_scale;   // DEVICE scalar multiplied into every accumulator before the epilogue (nullable = 1)
    int *status;
};

// One piece of work: K stages [kb_lo, kb_hi) of output tile tile_id.  n_pieces > 1: the tile's K range is shared by
// n_pieces consecutive CTAs, this one holding piece number `piece` (pieces are numbered in K order).
struct Segment {
    int tile_id, kb_lo, kb_hi, piece, n_pieces, first_cta;
};

// Enumerates a CTA's segments; every role of the CTA walks the same list.
//   classic: whole tiles, strided over the grid.
//   stream:  the tile-major list of all (tile, K stage) pairs is cut into gridDim.x equal contiguous ranges, so every
//            CTA streams the same number of weight bytes whatever the tile count; a tile whose stages fall into
//            several ranges is finished by the CTA that holds its first K piece (see the epilogue).
struct WorkIter {
    int kb_count, tiles, stream;
    long long total;   // stream: tiles * kb_count
    long long s, s_begin, s_end;
    __device__ long long range_lo(int cta) const { return (long long)cta * total / (long long)gridDim.x; }
    __device__ int cta_of(long long stage) const { return (int)(((stage + 1) * (long long)gridDim.x - 1) / total); }
    __device__ WorkIter(int tiles_, int kb_count_, int stream_) : kb_count(kb_count_), tiles(tiles_), stream(stream_) {
        total = (long long)tiles * kb_count;
        if (stream) { s_begin = range_lo(blockIdx.x); s_end = range_lo(blockIdx.x + 1); }
        else { s_begin = blockIdx.x; s_end = tiles; }
        s = s_begin;
    }
    __device__ bool next(Segment &g) {
        if (s >= s_end) return false;
        if (!stream) {
            g = Segment{(int)s, 0, kb_count, 0, 1, (int)blockIdx.x};
            s += gridDim.x;
            return true;
        }
        const int tile = (int)(s / kb_count);
        const long long t0 = (long long)tile * kb_count;
        const int kb_lo = (int)(s - t0);
        const long long left = s_end - s;
        const int len = (kb_count - kb_lo < left) ? kb_count - kb_lo : (int)left;
        const int c_first = cta_of(t0), c_last = cta_of(t0 + kb_count - 1);
        g = Segment{tile, kb_lo, kb_lo + len, (int)blockIdx.x - c_first, c_last - c_first + 1, c_first};
        s += len;
        return true;
    }
    // partial-tile slot of the piece CTA `cta` holds of tile `tile`: a CTA has at most two partial segments, the
    // first of its range (slot 0) and the last (slot 1)
    __device__ int slot_of(int cta, int tile) const {
        const long long lo = range_lo(cta), t0 = (long long)tile * kb_count;
        return 2 * cta + ((lo >= t0) ? 0 : 1);
    }
};

// Shared-memory stage: [weight tile][activation tile][activation residual tile (SPLIT)].
// SWAP puts the weights on the M side (128 rows) and BN tokens on the N side; otherwise 128 tokens x BN weights.
template <int BN, bool SWAP, bool SPLIT, int KA>
struct SmemLayout {
    static constexpr int kW = (SWAP ? kBM : BN) * kBK * 2;
    static constexpr int kX = (SWAP ? BN : kBM) * kBK * 2;
    static constexpr int kAtom = kW + kX * (SPLIT ? 2 : 1);   // one 64-wide K slab of every operand
    static constexpr int kStage = KA * kAtom;                 // KA slabs per pipeline stage
    // <= 32 tokens: the ring stays under 160 KB (three stages of 48 KB).  Measured on the batch-32 decode step: 11.17 ms
    // with a 192 KB ring (4 x 48 KB; 7 x 24 KB = 168 KB: 10.8), 10.63 ms with 144 KB, 10.78 ms even with 96 KB (4 x 24 KB)
    // -- ring depth hardly matters, a CTA that leaves a quarter of the SM's shared memory free does.
    static constexpr int kStagesFit = ((SWAP && BN == 32 ? 160 : 192) * 1024) / kStage;
    static constexpr int kStages = kStagesFit > 8 ? 8 : kStagesFit;
    static constexpr int kBytes = kStages * kStage + 1024 /*align slack*/ + 256 /*barriers*/;
    static constexpr int kTmemCols = (2 * BN < 32) ? 32 : 2 * BN;
};

__device__ __forceinline__ float silu_mul(float g, float u) { return g / (1.f + __expf(-g)) * u; }

// EPI: 0 fp32 store, 1 bf16 store, 2 fp32 accumulate (Y += D), 3 SwiGLU on interleaved gate/up weight rows -> bf16
// SPLIT: the activations come as two bf16 matrices (value and rounding residual); both are multiplied with the
// same weight tile into the same accumulator, which restores ~16 mantissa bits on the activation side.
// F16: operands are fp16 (single term) and the SwiGLU epilogue writes one fp16 matrix (saturating at +-65504).
template <int BN, bool SWAP, int EPI, bool SPLIT, int KA, bool F16>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
               const __grid_constant__ CUtensorMap map_x_lo, GemmParams p) {
    using L = SmemLayout<BN, SWAP, SPLIT, KA>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = base + L::kStages * L::kStage;      // full[S][KA], empty[S], tfull[2], tempty[2], 8 B each
    // full: one barrier per K slab of a stage, so that the MMAs of a stage start when its FIRST slab has landed (a stage of
    // four slabs is 96 KB; waiting for all of it would cost the start of every product a microsecond or two)
    static_assert((L::kStages * (KA + 1) + 4) * 8 <= 256, "barrier block");
    auto full_bar = [&](int s, int a) { return bars + 8u * (s * KA + a); };
    auto empty_bar = [&](int s) { return bars + 8u * (L::kStages * KA + s); };
    auto tfull_bar = [&](int a) { return bars + 8u * (L::kStages * (KA + 1) + a); };
    auto tempty_bar = [&](int a) { return bars + 8u * (L::kStages * (KA + 1) + 2 + a); };
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ bool split_last;
    __shared__ __align__(16) uint8_t swiglu_stage[(SWAP && EPI == 3) ? 8192 : 16];   // per epilogue warp: two [32][16] bf16 tiles

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &abort_s;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < L::kStages; ++s) {
            for (int a = 0; a < KA; ++a) mbar_init(full_bar(s, a), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)),
                     "r"((uint32_t)L::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    // launched with programmatic stream serialization: the set-up above overlaps the previous kernel's tail, and the
    // next kernel may start its own set-up now; everything that touches that kernel's data waits below
    pdl_launch_dependents();

    const int kb_count = p.K / (kBK * KA);   // pipeline stages along K
    const int total_tiles = p.m_tiles * p.n_tiles;   // output tile id: m fastest
    const int stream = SWAP ? p.stream : 0;

    if (warp == 0) {
        if (lane == 0) {  // ---------------- TMA producer ----------------
            pdl_wait();
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            WorkIter it(total_tiles, kb_count, stream);
            Segment g;
            while (ok && it.next(g)) {
                const int mt = g.tile_id % p.m_tiles, nt = g.tile_id / p.m_tiles;
                const int kb_lo = g.kb_lo, kb_hi = g.kb_hi;
                const int w_row = SWAP ? mt * kBM : nt * BN;
                const int x_row = SWAP ? nt * BN : mt * kBM;
                const unsigned long long tr0 = NNC_TRACE_NOW();
                (void)tr0;
                for (int kb = kb_lo; kb < kb_hi; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 1)) { ok = false; break; }
                    const uint32_t sw = base + stage * L::kStage;
#pragma unroll
                    for (int a = 0; a < KA; ++a) {   // KA consecutive slabs: KA * 128 contiguous bytes of every weight row
                        const uint32_t sa = sw + a * L::kAtom;
                        const int kx = (kb * KA + a) * kBK;
                        mbar_expect_tx(full_bar(stage, a), L::kAtom);
                        tma_load_2d(sa, &map_w, full_bar(stage, a), kx, w_row);
                        tma_load_2d(sa + L::kW, &map_x, full_bar(stage, a), kx, x_row);
                        if (SPLIT) tma_load_2d(sa + L::kW + L::kX, &map_x_lo, full_bar(stage, a), kx, x_row);
                    }
                    if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
                }
                if (NNC_TRACE_ALL_CTAS || blockIdx.x == 0) NNC_TRACE_EVENT(201, tr0, tr0, NNC_TRACE_NOW());
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {  // ---------------- MMA issuer ----------------
            constexpr uint32_t idesc = make_idesc(BN, F16);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            WorkIter it(total_tiles, kb_count, stream);
            Segment g;
            while (ok && it.next(g)) {
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, 2)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                const unsigned long long tr0 = NNC_TRACE_NOW();
                unsigned long long tr_first = tr0;
                (void)tr0; (void)tr_first;
                const int kb_lo = g.kb_lo, kb_hi = g.kb_hi;
                for (int kb = kb_lo; kb < kb_hi; ++kb) {
                    const uint32_t sw = base + stage * L::kStage;
#pragma unroll
                    for (int a = 0; a < KA; ++a) {
                        if (!mbar_wait(full_bar(stage, a), phase, abort_flag, p.status, 3)) { ok = false; break; }
                        if (kb == kb_lo && a == 0) tr_first = NNC_TRACE_NOW();
                        tc_fence_after();
                        const uint32_t sa = sw + a * L::kAtom;
                        const uint64_t dw = make_smem_desc(sa), dx = make_smem_desc(sa + L::kW),
                                       dxl = make_smem_desc(sa + L::kW + L::kX);
#pragma unroll
                        for (int k = 0; k < kBK / 16; ++k) {
                            const uint64_t off = (uint64_t)(k * 2);  // 32 bytes, in 16-byte units
                            const uint32_t accum = (kb != kb_lo) || (a != 0) || (k != 0);
                            if (SWAP) {
                                umma_bf16(d_tmem, dw + off, dx + off, idesc, accum);
                                if (SPLIT) umma_bf16(d_tmem, dw + off, dxl + off, idesc, 1u);
                            } else {
                                umma_bf16(d_tmem, dx + off, dw + off, idesc, accum);
                                if (SPLIT) umma_bf16(d_tmem, dxl + off, dw + off, idesc, 1u);
                            }
                        }
                    }
                    if (!ok) break;
                    umma_commit(empty_bar(stage));
                    if (++stage == L::kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit(tfull_bar(acc));
                if (NNC_TRACE_ALL_CTAS || blockIdx.x == 0) NNC_TRACE_EVENT(202, tr0, tr_first, NNC_TRACE_NOW());
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {  // ---------------- epilogue warps 2..5 ----------------
        const int quarter = warp & 3;  // TMEM lane quarter this warp may read
        const unsigned long long trk0 = NNC_TRACE_NOW();
        (void)trk0;
        pdl_wait();
        const float osc = p.out_scale ? __ldg(p.out_scale) : 1.f;
        int acc = 0;
        uint32_t acc_phase = 0;
        // SWAP stores: row m = weight row, columns = tokens n0 .. n0 + 31; a warp stores 32 consecutive weight rows per token
        auto store_swap = [&](const uint32_t (&r)[32], int m, int n0) {
            if (EPI == 3) {
                // Gate rows sit in even lanes, up rows in odd lanes.  The two lanes of a pair swap half of their
                // values so that each computes 16 of the pair's 32 tokens; the results are staged in this warp's
                // shared-memory tile [token][16 outputs] and leave as two 16-byte stores per token.
                const int par = lane & 1, col = lane >> 1;
                bf16 (*st_hi)[16] = reinterpret_cast<bf16 (*)[16]>(swiglu_stage + (size_t)(quarter * 2) * 1024);
                bf16 (*st_lo)[16] = reinterpret_cast<bf16 (*)[16]>(swiglu_stage + (size_t)(quarter * 2 + 1) * 1024);
                float a[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float send = __uint_as_float(par ? r[2 * i] : r[2 * i + 1]);
                    const float recv = __shfl_xor_sync(0xffffffffu, send, 1);
                    const float gate = par ? recv : __uint_as_float(r[2 * i]);
                    const float up = par ? __uint_as_float(r[2 * i + 1]) : recv;
                    a[i] = silu_mul(gate, up);   // token n0 + 2 i + par
                }
                __syncwarp();   // the previous call's readers are done with the tile
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const bf16 hi = __float2bfloat16_rn(a[i]);
                    st_hi[2 * i + par][col] = hi;
                    st_lo[2 * i + par][col] = __float2bfloat16_rn(a[i] - __bfloat162float(hi));
                }
                __syncwarp();
                const int t = n0 + lane;                       // this lane stores token t
                const int m0 = m - lane;                       // first weight row of this warp (even)
                if (t < p.T) {
                    const size_t yo = (size_t)t * p.ldy + (m0 >> 1);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (m0 + 16 * h + 15 < p.N) {          // N is a multiple of 16: a chunk of 8 outputs is whole or absent
                            *reinterpret_cast<uint4 *>(reinterpret_cast<bf16 *>(p.Y) + yo + 8 * h) =
                                *reinterpret_cast<const uint4 *>(&st_hi[lane][8 * h]);
                            if (p.Y_lo)
                                *reinterpret_cast<uint4 *>(reinterpret_cast<bf16 *>(p.Y_lo) + yo + 8 * h) =
                                    *reinterpret_cast<const uint4 *>(&st_lo[lane][8 * h]);
                        }
                    }
                }
            } else if (EPI == 2) {
                // all 32 old values are requested before the first store: a load-add-store chain per token would pay
                // one memory round trip per token
                float *y = reinterpret_cast<float *>(p.Y) + m;
                float old[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) old[i] = (m < p.N && n0 + i < p.T) ? __ldcg(y + (size_t)(n0 + i) * p.ldy) : 0.f;
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (m < p.N && n0 + i < p.T) y[(size_t)(n0 + i) * p.ldy] = old[i] + __uint_as_float(r[i]);
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int t = n0 + i;
                    if (m < p.N && t < p.T) {
                        const float v = __uint_as_float(r[i]);
                        if (EPI == 1) reinterpret_cast<bf16 *>(p.Y)[(size_t)t * p.ldy + m] = __float2bfloat16_rn(v);
                        else reinterpret_cast<float *>(p.Y)[(size_t)t * p.ldy + m] = v;
                    }
                }
            }
        };
        WorkIter it(total_tiles, kb_count, stream);
        Segment g;
        bool dead = false;   // this warp has seen the abort; in stream mode it keeps walking (the group barriers below
                             // need all four warps) but touches nothing any more
        while (it.next(g)) {
            const int tile_id = g.tile_id;
            const int mt = tile_id % p.m_tiles, nt = tile_id / p.m_tiles;
            const bool shared_tile = SWAP && g.n_pieces > 1;
            const bool got = !dead && mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, 4);
            if (!got) {
                dead = true;
                if (!stream) break;
                if (!shared_tile) continue;
            }
            tc_fence_after();
            const int m = mt * kBM + quarter * 32 + lane;  // D row held by this thread
            const unsigned long long tr0 = NNC_TRACE_NOW();
            unsigned long long tr1 = tr0;
            (void)tr0; (void)tr1;
            if (shared_tile) {
                // ---- the tile's K range is shared with other CTAs.  Every piece but the first parks its fp32 tile in
                //      scratch and raises its flag.  The first piece is the last segment of its CTA's range, so it is
                //      the one that finishes last by schedule: it keeps its tile in tensor memory, waits (bounded) for
                //      the other flags, adds the pieces in K order and runs the epilogue. ----
                const int row = quarter * 32 + lane;
                constexpr size_t kSlotFloats = (size_t)BN * kBM;
                if (g.piece != 0) {
                    const int my_slot = it.slot_of(blockIdx.x, tile_id);
                    float *slot = p.part + (size_t)my_slot * kSlotFloats;
                    if (got && NNC_BC(((size_t)my_slot + 1) * kSlotFloats * sizeof(float) <= p.part_bytes, 4001)) {
#pragma unroll 1
                        for (int c0 = 0; c0 < BN; c0 += 32) {
                            uint32_t r[32];
                            tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + c0), r);
                            // slot layout [32-column chunk][4-column group][row][4]: a warp's store covers 512 contiguous bytes
                            uint4 *dst = reinterpret_cast<uint4 *>(slot) + (size_t)(c0 >> 5) * 8 * kBM + row;
#pragma unroll
                            for (int i = 0; i < 8; ++i) dst[i * kBM] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(tempty_bar(acc));
                    }
                    tr1 = NNC_TRACE_NOW();
                    asm volatile("bar.sync 2, 128;" ::: "memory");   // all four warps' stores are issued
                    if (warp == 2 && lane == 0 && !*abort_flag) {
                        __threadfence();
                        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.tickets + my_slot), "r"(1u) : "memory");
                    }
                    if ((NNC_TRACE_ALL_CTAS || blockIdx.x == 0) && warp == 2 && lane == 0) NNC_TRACE_EVENT(203, tr0, tr1, NNC_TRACE_NOW());
                } else {
                    // Accumulating epilogue of a 32-token tile: the old output values do not depend on the other pieces, so
                    // they are requested now and arrive while this CTA waits for the flags and reads the pieces.
                    constexpr bool kOldEarly = EPI == 2 && BN == 32;
                    float old_y[kOldEarly ? 32 : 1];
                    if (kOldEarly && got) {
                        const float *y = reinterpret_cast<const float *>(p.Y) + m;
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            old_y[i] = (m < p.N && nt * BN + i < p.T) ? __ldcg(y + (size_t)(nt * BN + i) * p.ldy) : 0.f;
                    }
                    if (warp == 2) {
                        // bounded wait for the other pieces (they never wait for anything of this CTA's); one flag per
                        // lane, so that all of them are polled in one memory round trip
                        bool ok = got;
                        unsigned long long t_first = 0;
                        for (int q0 = 1; q0 < g.n_pieces && ok; q0 += 32) {
                            const int q = q0 + lane;
                            const uint32_t *flag = (q < g.n_pieces) ? p.tickets + it.slot_of(g.first_cta + q, tile_id) : nullptr;
                            for (uint32_t spin = 0;; ++spin) {
                                uint32_t v = 1u;
                                if (flag) asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
                                if (__all_sync(0xffffffffu, v != 0u)) break;
                                if ((spin & 255u) == 255u) {
                                    int give_up = 0;
                                    if (lane == 0) {
                                        const unsigned long long now = global_ns();
                                        if (t_first == 0) t_first = now;
                                        if (*abort_flag || now - t_first > kWaitLimitNs) {
                                            if (!*abort_flag) { *abort_flag = 1; atomicExch(p.status, 5); }
                                            give_up = 1;
                                        }
                                    }
                                    if (__shfl_sync(0xffffffffu, give_up, 0)) { ok = false; break; }
                                }
                            }
                        }
                        if (lane == 0) split_last = ok;
                    }
                    asm volatile("bar.sync 2, 128;" ::: "memory");
                    tr1 = NNC_TRACE_NOW();
                    if (split_last && got) {
#pragma unroll 1
                        for (int c0 = 0; c0 < BN; c0 += 32) {
                            uint32_t r[32];
                            tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + c0), r);
                            float sum[32];
#pragma unroll
                            for (int i = 0; i < 32; ++i) sum[i] = __uint_as_float(r[i]);
                            // the parked pieces are added in K order; up to kU pieces' loads are in flight at a time
                            constexpr int kU = kOldEarly ? 3 : 4;   // the early old values take a piece's worth of registers
                            const size_t in_slot = ((size_t)(c0 >> 5) * 8 * kBM + row) * 4;
                            for (int q0 = 1; q0 < g.n_pieces; q0 += kU) {
                                float4 v[kU][8];
#pragma unroll
                                for (int u = 0; u < kU; ++u) {
                                    if (q0 + u < g.n_pieces) {
                                        const float4 *src = reinterpret_cast<const float4 *>(
                                            p.part + (size_t)it.slot_of(g.first_cta + q0 + u, tile_id) * kSlotFloats + in_slot);
#pragma unroll
                                        for (int i = 0; i < 8; ++i) v[u][i] = __ldcg(src + i * kBM);
                                    }
                                }
#pragma unroll
                                for (int u = 0; u < kU; ++u) {
                                    if (q0 + u < g.n_pieces) {
#pragma unroll
                                        for (int i = 0; i < 8; ++i) {
                                            sum[4 * i] += v[u][i].x; sum[4 * i + 1] += v[u][i].y;
                                            sum[4 * i + 2] += v[u][i].z; sum[4 * i + 3] += v[u][i].w;
                                        }
                                    }
                                }
                            }
#pragma unroll
                            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(sum[i] * osc);
                            const unsigned long long tr2 = NNC_TRACE_NOW();
                            (void)tr2;
                            if (kOldEarly) {
                                float *y = reinterpret_cast<float *>(p.Y) + m;
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (m < p.N && nt * BN + i < p.T) y[(size_t)(nt * BN + i) * p.ldy] = old_y[i] + __uint_as_float(r[i]);
                            } else {
                                store_swap(r, m, nt * BN + c0);
                            }
                            if ((NNC_TRACE_ALL_CTAS || blockIdx.x == 0) && warp == 2 && lane == 0) NNC_TRACE_EVENT(206, tr1, tr2, NNC_TRACE_NOW());
                        }
                    }
                    if (got) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(tempty_bar(acc));
                    }
                    asm volatile("bar.sync 2, 128;" ::: "memory");   // every warp has read the parked pieces
                    if (warp == 2 && lane == 0 && split_last) {
                        // flags back to rest for the next launch that uses this scratch
                        for (int q = 1; q < g.n_pieces; ++q) p.tickets[it.slot_of(g.first_cta + q, tile_id)] = 0u;
                    }
                    if ((NNC_TRACE_ALL_CTAS || blockIdx.x == 0) && warp == 2 && lane == 0) NNC_TRACE_EVENT(205, tr0, tr1, NNC_TRACE_NOW());
                }
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
                continue;
            }
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + c0), r);
                if (p.out_scale) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * osc);
                }
                const int n0 = nt * BN + c0;
                if (!SWAP) {
                    // row m = token, columns n0.. = weight rows: contiguous per thread
                    if (m < p.T) {
                        if (EPI == 3) {
                            const size_t yo = (size_t)m * p.ldy + (n0 >> 1);
                            bf16 *y = reinterpret_cast<bf16 *>(p.Y) + yo;
                            bf16 *yl = p.Y_lo ? reinterpret_cast<bf16 *>(p.Y_lo) + yo : nullptr;
                            if (n0 + 32 <= p.N) {
                                uint32_t o[8], ol[8];
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const float a0 = silu_mul(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]));
                                    const float a1 = silu_mul(__uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
                                    if (F16) {
                                        o[i] = pack_f16x2_sat(a0, a1);
                                        ol[i] = 0u;
                                    } else {
                                        o[i] = pack_bf16x2(a0, a1);
                                        ol[i] = pack_bf16x2(a0 - bf16_lo(o[i]), a1 - bf16_hi(o[i]));
                                    }
                                }
                                reinterpret_cast<uint4 *>(y)[0] = make_uint4(o[0], o[1], o[2], o[3]);
                                reinterpret_cast<uint4 *>(y)[1] = make_uint4(o[4], o[5], o[6], o[7]);
                                if (yl) {
                                    reinterpret_cast<uint4 *>(yl)[0] = make_uint4(ol[0], ol[1], ol[2], ol[3]);
                                    reinterpret_cast<uint4 *>(yl)[1] = make_uint4(ol[4], ol[5], ol[6], ol[7]);
                                }
                            } else {
                                for (int i = 0; i < 16; ++i)
                                    if (n0 + 2 * i + 1 < p.N) {
                                        const float a = silu_mul(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                                        if (F16) {
                                            reinterpret_cast<uint16_t *>(y)[i] = (uint16_t)(pack_f16x2_sat(a, 0.f) & 0xffffu);
                                        } else {
                                            const bf16 hi = __float2bfloat16_rn(a);
                                            y[i] = hi;
                                            if (yl) yl[i] = __float2bfloat16_rn(a - __bfloat162float(hi));
                                        }
                                    }
                            }
                        } else if (EPI == 1) {
                            bf16 *y = reinterpret_cast<bf16 *>(p.Y) + (size_t)m * p.ldy + n0;
                            if (n0 + 32 <= p.N) {
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    uint4 o;
                                    o.x = pack_bf16x2(__uint_as_float(r[8 * i]), __uint_as_float(r[8 * i + 1]));
                                    o.y = pack_bf16x2(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3]));
                                    o.z = pack_bf16x2(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5]));
                                    o.w = pack_bf16x2(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7]));
                                    reinterpret_cast<uint4 *>(y)[i] = o;
                                }
                            } else {
                                for (int i = 0; i < 32; ++i)
                                    if (n0 + i < p.N) y[i] = __float2bfloat16_rn(__uint_as_float(r[i]));
                            }
                        } else {
                            float *y = reinterpret_cast<float *>(p.Y) + (size_t)m * p.ldy + n0;
                            if (n0 + 32 <= p.N) {
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    float4 v = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                                           __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
                                    if (EPI == 2) {
                                        const float4 o = reinterpret_cast<float4 *>(y)[i];
                                        v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                                    }
                                    reinterpret_cast<float4 *>(y)[i] = v;
                                }
                            } else {
                                for (int i = 0; i < 32; ++i)
                                    if (n0 + i < p.N) y[i] = (EPI == 2 ? y[i] : 0.f) + __uint_as_float(r[i]);
                            }
                        }
                    }
                } else {
                    store_swap(r, m, n0);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (warp == 2 && lane == 0) NNC_TRACE_EVENT(204, trk0, trk0, NNC_TRACE_NOW());
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
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)L::kTmemCols)
                     : "memory");
    }
}

// ---- host side ----------------------------------------------------------------------------------------

// bf16 matrix [rows][K], K contiguous; box = 64 columns (128 bytes) x box_rows, 128-byte swizzle, zero fill
bool make_map(CUtensorMap *map, const void *ptr, int rows, int K, int box_rows, bool fp16 = false) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, bool SWAP, int EPI, bool SPLIT, int KA, bool F16 = false>
cudaError_t launch_tc_ka(const LaunchCtx &lc, const bf16 *X, const bf16 *X_lo, const bf16 *W, void *Y, void *Y_lo, int T, int N,
                      int K, int ldy, int *status, const GemmScratch *scratch, const float *out_scale = nullptr) {
    using L = SmemLayout<BN, SWAP, SPLIT, KA>;
    auto kern = gemm_tc_kernel<BN, SWAP, EPI, SPLIT, KA, F16>;
    static unsigned long long attr_done = 0;   // per instantiation, one bit per device
    if (cudaError_t e = ensure_dynamic_smem(kern, L::kBytes, &attr_done); e != cudaSuccess) return e;
    CUtensorMap map_w, map_x, map_x_lo;
    GemmParams p;
    p.Y = Y; p.Y_lo = Y_lo; p.T = T; p.N = N; p.K = K; p.ldy = ldy; p.status = status; p.out_scale = out_scale;
    const int w_box = SWAP ? kBM : BN, x_box = SWAP ? BN : kBM;
    if (!make_map(&map_w, W, N, K, w_box, F16) || !make_map(&map_x, X, T, K, x_box, F16)) return cudaErrorInvalidValue;
    if (!make_map(&map_x_lo, SPLIT ? X_lo : X, T, K, x_box, F16)) return cudaErrorInvalidValue;
    if (!SWAP) {
        p.m_tiles = (T + kBM - 1) / kBM;
        p.n_tiles = (N + BN - 1) / BN;
    } else {
        p.m_tiles = (N + kBM - 1) / kBM;
        p.n_tiles = (T + BN - 1) / BN;
    }
    // Few tokens: the product is bound by streaming the weights.  Whole tiles dealt round-robin leave SMs idle in the
    // last round (or all the time, when there are fewer tiles than SMs), so the (tile, K stage) space is cut into one
    // equal contiguous range per CTA instead; tiles that straddle a cut are finished through partial tiles in scratch.
    p.stream = 0; p.part = nullptr; p.tickets = nullptr; p.part_bytes = 0;
    const int tiles = p.m_tiles * p.n_tiles;
    int grid = tiles < lc.sm_count ? tiles : lc.sm_count;
    if (SWAP && scratch && scratch->part && scratch->tickets) {
        const long long stages = (long long)tiles * (K / (kBK * KA));
        const int g = stages < lc.sm_count ? (int)stages : lc.sm_count;
        const double whole_tile_eff = (double)tiles / (((tiles + lc.sm_count - 1) / lc.sm_count) * (double)lc.sm_count);
        const size_t need = (size_t)2 * g * BN * kBM * sizeof(float);
        if (whole_tile_eff < 0.97 && need <= scratch->part_bytes && 2 * g <= scratch->n_tickets) {
            p.stream = 1; p.part = scratch->part; p.tickets = scratch->tickets; p.part_bytes = scratch->part_bytes;
            grid = g;
        }
    }
    if (lc.launches) ++*lc.launches;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = L::kBytes;
    cfg.stream = lc.stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = lc.pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, map_w, map_x, map_x_lo, p);
}

// Few tokens (weights on the M side): a stage carries 2 consecutive K slabs (three stages of 48 KB at <= 32 tokens,
// three of 64 KB at <= 64), each slab with its own full barrier.  Measured on the batch-32 decode step with a 192 KB
// ring: 2 slabs per stage 11.25 ms, 4 slabs (two stages of 96 KB) 11.33 ms, 1 slab (eight stages) 11.35 ms.
template <int BN, bool SWAP, int EPI, bool SPLIT>
cudaError_t launch_tc(const LaunchCtx &lc, const bf16 *X, const bf16 *X_lo, const bf16 *W, void *Y, void *Y_lo, int T, int N,
                      int K, int ldy, int *status, const GemmScratch *scratch) {
    if (SWAP && BN == 32 && K % (2 * kBK) == 0)
        return launch_tc_ka<BN, SWAP, EPI, SPLIT, (SWAP && BN == 32) ? 2 : 1>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, scratch);
    if (SWAP && BN == 64 && K % (2 * kBK) == 0)
        return launch_tc_ka<BN, SWAP, EPI, SPLIT, (SWAP && BN == 64) ? 2 : 1>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, scratch);
    return launch_tc_ka<BN, SWAP, EPI, SPLIT, 1>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, scratch);
}

template <int EPI, bool SPLIT>
cudaError_t dispatch(const LaunchCtx &lc, const bf16 *X, const bf16 *X_lo, const bf16 *W, void *Y, void *Y_lo, int T, int N,
                     int K, int ldy, int *status, const GemmScratch *sc, bool f16, const float *out_scale) {
    if (f16) {   // fp16 operands: the prompt-phase form only (tokens on the M side, one term)
        if (SPLIT || T <= 128) return cudaErrorInvalidValue;
        return launch_tc_ka<256, false, EPI, false, 1, true>(lc, X, nullptr, W, Y, Y_lo, T, N, K, ldy, status, sc, out_scale);
    }
    if (out_scale) return cudaErrorInvalidValue;
    if (T <= 32) return launch_tc<32, true, EPI, SPLIT>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, sc);
    if (T <= 64) return launch_tc<64, true, EPI, SPLIT>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, sc);
    if (T <= 128) return launch_tc<128, true, EPI, SPLIT>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, sc);
    return launch_tc<256, false, EPI, SPLIT>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, sc);
}

template <bool SPLIT>
cudaError_t dispatch_epi(const LaunchCtx &lc, const bf16 *X, const bf16 *X_lo, const bf16 *W, void *Y, void *Y_lo, int T,
                         int N, int K, int ldy, int epi, int *status, const GemmScratch *sc, bool f16, const float *out_scale) {
    switch (epi) {
        case kEpiStoreF32: return dispatch<0, SPLIT>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, sc, f16, out_scale);
        case kEpiStoreBf16: return dispatch<1, SPLIT>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, sc, f16, out_scale);
        case kEpiAccumF32: return dispatch<2, SPLIT>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, sc, f16, out_scale);
        case kEpiSwigluBf16: return dispatch<3, SPLIT>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, status, sc, f16, out_scale);
    }
    return cudaErrorInvalidValue;
}

}  // namespace

bool gemm_tc_available() { return get_encode() != nullptr; }

// Y[T][*] (row stride ldy) = epilogue(out_scale * (X + X_lo)[T][K] * W[N][K]^T).  Operands 16-byte aligned, K % 64 == 0.
// f16: X and W hold fp16 instead of bf16 (T > 128, no X_lo); the SwiGLU epilogue then writes fp16.
cudaError_t launch_gemm(const LaunchCtx &lc, const bf16 *X, const bf16 *X_lo, const bf16 *W, void *Y, void *Y_lo, int T,
                        int N, int K, int ldy, int epi, int *status, const GemmScratch *scratch, bool f16,
                        const float *out_scale) {
    if (T <= 0 || N <= 0 || K <= 0 || K % kBK != 0 || N % 8 != 0) return cudaErrorInvalidValue;
    if (((uintptr_t)X | (uintptr_t)X_lo | (uintptr_t)W | (uintptr_t)Y | (uintptr_t)Y_lo) & 15) return cudaErrorInvalidValue;
    // the epilogue stores 16-byte vectors per output row: the row pitch must keep them aligned
    const bool out_bf16 = epi == kEpiStoreBf16 || epi == kEpiSwigluBf16;
    if (ldy % (out_bf16 ? 8 : 4) != 0) return cudaErrorInvalidValue;
    if (epi == kEpiSwigluBf16 && N % 16 != 0) return cudaErrorInvalidValue;   // outputs leave in chunks of 8
    return X_lo ? dispatch_epi<true>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, epi, status, scratch, f16, out_scale)
                : dispatch_epi<false>(lc, X, X_lo, W, Y, Y_lo, T, N, K, ldy, epi, status, scratch, f16, out_scale);
}

}  // namespace nnc
