// One-time weight repack (and its inverse, for tests): strided row copies between bf16 matrices whose rows
// have the same length.  Concatenating Wq|Wk|Wv and interleaving gate/up rows are both instances of
// "destination row d0 + i*ds <- source row s0 + i*ss".  Pure bit moves, 16 bytes per thread, HBM-bound.
//
// Also here: the fp16 copy of a bf16 matrix that the prompt-phase GEMMs multiply with fp16 activations.  fp16 has more
// mantissa bits than bf16 but a narrow exponent range, so the copy holds W * 2^e with e chosen per matrix such that
// the largest magnitude lands in [2^14, 2^15): every weight down to 2^-32 of the largest one converts exactly (the 8
// significant bits of a bf16 value fit, and the scaling is a power of two); smaller ones round on the fp16 subnormal
// grid, an error below 2^-39 of the largest weight.  The GEMM epilogue multiplies by 2^-e.
#include <cuda_fp16.h>

#include "common.cuh"
#include "nnc_internal.h"

namespace nnc {

namespace {

__global__ void copy_rows_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, int rows, int chunks_per_row,
                                 int dst_row0, int dst_row_step, int src_row0, int src_row_step, int dst_rows_total,
                                 int src_rows_total) {
    const size_t total = (size_t)rows * chunks_per_row;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t r = i / chunks_per_row, c = i % chunks_per_row;
        const size_t dr = (size_t)dst_row0 + r * dst_row_step, sr = (size_t)src_row0 + r * src_row_step;
        if (NNC_BC(dr < (size_t)dst_rows_total && sr < (size_t)src_rows_total, 501))
            dst[dr * chunks_per_row + c] = src[sr * chunks_per_row + c];
    }
}

// checked build only: a kernel that reports one miss and touches no memory, so that a test can see the counter work
__global__ void bounds_check_selftest_kernel(int code) { (void)NNC_BC(code == 0, (unsigned)code); }

// max |w| over a bf16 matrix as fp32 bits (non-negative floats order like their bit patterns); NaNs are skipped
__global__ void absmax_bits_kernel(const uint4 *__restrict__ src, size_t n_chunks, uint32_t *__restrict__ max_bits) {
    uint32_t m = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_chunks; i += (size_t)gridDim.x * blockDim.x) {
        const uint4 v = src[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t a = (w[k] << 16) & 0x7fffffffu, b = w[k] & 0x7fff0000u;
            if (a <= 0x7f800000u && a > m) m = a;
            if (b <= 0x7f800000u && b > m) m = b;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m) atomicMax(max_bits, m);
}

// scales[0] = 2^e, scales[1] = 2^-e with 2^14 <= max * 2^e < 2^15 (e = 0 for an all-zero or non-finite maximum)
__global__ void f16_scale_kernel(const uint32_t *__restrict__ max_bits, float *__restrict__ scales) {
    const uint32_t b = *max_bits;
    int e = 0;
    if (b != 0 && b < 0x7f800000u) {
        int ex = (int)(b >> 23) - 127;           // floor(log2(max)) for normal values
        if ((b >> 23) == 0) ex = -127;           // bf16 subnormals: treat as the smallest normal binade
        e = 14 - ex;
        if (e > 120) e = 120;
        if (e < -120) e = -120;
    }
    scales[0] = exp2f((float)e);
    scales[1] = exp2f((float)-e);
}

__global__ void to_f16_scaled_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, size_t n_chunks,
                                     const float *__restrict__ scales) {
    const float sc = scales[0];
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_chunks; i += (size_t)gridDim.x * blockDim.x) {
        const uint4 v = src[i];
        uint4 o;
        o.x = pack_f16x2_sat(bf16_lo(v.x) * sc, bf16_hi(v.x) * sc);
        o.y = pack_f16x2_sat(bf16_lo(v.y) * sc, bf16_hi(v.y) * sc);
        o.z = pack_f16x2_sat(bf16_lo(v.z) * sc, bf16_hi(v.z) * sc);
        o.w = pack_f16x2_sat(bf16_lo(v.w) * sc, bf16_hi(v.w) * sc);
        dst[i] = o;
    }
}

// FP8 E4M3 row quantisation, one block per row: e = the smallest integer with max|w| <= 448 * 2^e; codes = round to
// nearest even of w * 2^-e onto the E4M3 grid (saturating; the hardware conversion); scale = 2^e.  The scaling by a
// power of two is exact, so host and device reach the same codes bit for bit.
__global__ void __launch_bounds__(256)
quantise_rows_e4m3_kernel(const bf16 *W, uint8_t *__restrict__ codes, float *__restrict__ scales,
                          bf16 *dequant /* may alias W: every thread reads a chunk before it writes that chunk */, int n_in) {
    __shared__ uint32_t red[8];
    const size_t row = blockIdx.x;
    const uint4 *src = reinterpret_cast<const uint4 *>(W + row * n_in);
    const int n8 = n_in / 8;
    uint32_t m = 0;
    for (int i = threadIdx.x; i < n8; i += 256) {
        const uint4 v = src[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t a = (w[k] << 16) & 0x7fffffffu, b = w[k] & 0x7fff0000u;
            if (a <= 0x7f800000u && a > m) m = a;
            if (b <= 0x7f800000u && b > m) m = b;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    m = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) m = max(m, red[w]);
    // amax = f * 2^E with f in [0.5, 1); 448 = 0.875 * 2^9, so e = E - 9 if f <= 0.875, else E - 8
    int e = 0;
    if (m != 0u && m < 0x7f800000u) {
        const float amax = __uint_as_float(m);
        int E;
        const float f = frexpf(amax, &E);
        e = (f <= 0.875f) ? E - 9 : E - 8;
        e = max(-127, min(127, e));
    }
    const float down = exp2f((float)-e), up = exp2f((float)e);
    if (threadIdx.x == 0) scales[row] = up;
    uint2 *dst = reinterpret_cast<uint2 *>(codes + row * n_in);
    uint4 *dq = dequant ? reinterpret_cast<uint4 *>(dequant + row * n_in) : nullptr;
    for (int i = threadIdx.x; i < n8; i += 256) {
        const uint4 v = src[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t c[4];   // two codes each (low 16 bits)
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint16_t pair;
            const float lo = bf16_lo(w[k]) * down, hi = bf16_hi(w[k]) * down;
            asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pair) : "f"(hi), "f"(lo));
            c[k] = pair;
        }
        dst[i] = make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16));
        if (dq) {
            uint32_t o[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                uint32_t h2;
                asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)c[k]));
                const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
                o[k] = pack_bf16x2(f.x * up, f.y * up);   // at most 4 significant bits times a power of two: exact
            }
            dq[i] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

}  // namespace

cudaError_t launch_quantise_rows_e4m3(const LaunchCtx &lc, const bf16 *W, uint8_t *codes, float *scales, bf16 *dequant,
                                      int n_out, int n_in) {
    if (n_out <= 0 || n_in <= 0 || n_in % 8) return cudaErrorInvalidValue;
    LaunchCtx plain = lc;
    plain.pdl = false;
    return launch(plain, quantise_rows_e4m3_kernel, dim3((unsigned)n_out), dim3(256), W, codes, scales, dequant, n_in);
}

// dst (fp16 bits) = src (bf16) * 2^e; scales: DEVICE float[2] receiving {2^e, 2^-e}; max_bits: DEVICE scratch word.
// Stream-ordered, no host synchronisation.
cudaError_t launch_to_f16_scaled(const LaunchCtx &lc, const bf16 *src, void *dst, size_t n, float *scales, uint32_t *max_bits) {
    if (n % 8) return cudaErrorInvalidValue;
    const size_t chunks = n / 8;
    size_t blocks = (chunks + 255) / 256;
    const size_t cap = (size_t)lc.sm_count * 16;
    if (blocks > cap) blocks = cap;
    if (blocks == 0) return cudaSuccess;
    LaunchCtx plain = lc;
    plain.pdl = false;
    cudaError_t e = cudaMemsetAsync(max_bits, 0, 4, lc.stream);
    if (e != cudaSuccess) return e;
    e = launch(plain, absmax_bits_kernel, dim3((unsigned)blocks), dim3(256), reinterpret_cast<const uint4 *>(src), chunks, max_bits);
    if (e != cudaSuccess) return e;
    e = launch(plain, f16_scale_kernel, dim3(1), dim3(1), (const uint32_t *)max_bits, scales);
    if (e != cudaSuccess) return e;
    return launch(plain, to_f16_scaled_kernel, dim3((unsigned)blocks), dim3(256), reinterpret_cast<const uint4 *>(src),
                  reinterpret_cast<uint4 *>(dst), chunks, (const float *)scales);
}

cudaError_t launch_copy_rows(const LaunchCtx &lc, const bf16 *src, bf16 *dst, int rows, int K, int dst_row0,
                             int dst_row_step, int src_row0, int src_row_step) {
    if (K % 8) return cudaErrorInvalidValue;
    const size_t total = (size_t)rows * (K / 8);
    size_t blocks = (total + 255) / 256;
    const size_t cap = (size_t)lc.sm_count * 16;
    if (blocks > cap) blocks = cap;
    if (blocks == 0) return cudaSuccess;
    LaunchCtx plain = lc;
    plain.pdl = false;
    // the last row touched on either side bounds the matrices from below: what the checked build compares with
    const int dst_rows_total = dst_row0 + (rows - 1) * dst_row_step + 1, src_rows_total = src_row0 + (rows - 1) * src_row_step + 1;
    return launch(plain, copy_rows_kernel, dim3((unsigned)blocks), dim3(256), reinterpret_cast<const uint4 *>(src),
                  reinterpret_cast<uint4 *>(dst), rows, K / 8, dst_row0, dst_row_step, src_row0, src_row_step, dst_rows_total,
                  src_rows_total);
}

cudaError_t launch_bounds_check_selftest(const LaunchCtx &lc, int code) {
    LaunchCtx plain = lc;
    plain.pdl = false;
    return launch(plain, bounds_check_selftest_kernel, dim3(1), dim3(1), code);
}

}  // namespace nnc
