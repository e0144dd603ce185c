// One-time weight repack (and its inverse, for tests): strided row copies between bf16 matrices whose rows
// have the same length.  Concatenating Wq|Wk|Wv and interleaving gate/up rows are both instances of
// "destination row d0 + i*ds <- source row s0 + i*ss".  Pure bit moves, 16 bytes per thread, HBM-bound.
#include "common.cuh"
#include "nnc_internal.h"

namespace nnc {

namespace {

__global__ void copy_rows_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, int rows, int chunks_per_row,
                                 int dst_row0, int dst_row_step, int src_row0, int src_row_step) {
    const size_t total = (size_t)rows * chunks_per_row;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t r = i / chunks_per_row, c = i % chunks_per_row;
        dst[((size_t)dst_row0 + r * dst_row_step) * chunks_per_row + c] =
            src[((size_t)src_row0 + r * src_row_step) * chunks_per_row + c];
    }
}

}  // namespace

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
    return launch(plain, copy_rows_kernel, dim3((unsigned)blocks), dim3(256), reinterpret_cast<const uint4 *>(src),
                  reinterpret_cast<uint4 *>(dst), rows, K / 8, dst_row0, dst_row_step, src_row0, src_row_step);
}

}  // namespace nnc
