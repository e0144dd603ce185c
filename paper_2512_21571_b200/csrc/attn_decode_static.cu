// nnc_op_attn_decode_static: the split-K flash-decode operation for callers that cannot allocate.
//
// Some users of this library run where device allocation is off the table: inside a stream-ordered region
// that must not synchronise, in a process whose memory pool is owned and fully handed out by another runtime,
// or in a plug-in that is only ever given its input and output buffers.  nnc_op_attn_decode asks such a
// caller for a scratch buffer it has no way to produce.  This variant keeps the scratch (split-K partials and
// the per-head ticket words) in a fixed array that is part of the library image instead, so the call needs
// nothing beyond its inputs and outputs and never calls cudaMalloc, cudaFree or any allocating routine.
//
// Cost and limits of that choice:
//   - the array is NNC_ATTN_STATIC_SCRATCH_BYTES large and every GPU that loads the library holds it until
//     the process exits;
//   - problems whose scratch need exceeds it are refused with NNC_ERR_CAPACITY (nothing is launched);
//   - all calls on a device share the one array, which keeps whatever the previous call left: the ticket
//     words are cleared at the start of every call, and two calls that overlap on the GPU (different streams,
//     or different host threads) race on it -- serialise them;
//   - the first call on each device looks up the array's device address (cudaGetSymbolAddress) under a
//     host lock; make that first call outside any stream capture.
#include <mutex>
#include <stdio.h>

#include "nnc_internal.h"

using namespace nnc;

namespace {

// In host code this name is only a handle for the runtime's symbol calls, never a device address.
static __device__ __align__(256) unsigned char g_attn_static_scratch[NNC_ATTN_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_lock;
void *g_scratch_addr[kMaxDevices];  // device address of the array, per device ordinal; null = not looked up yet

// Device address of the scratch array on the current device; looked up once per device.
cudaError_t scratch_for_current_device(void **out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> guard(g_setup_lock);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_attn_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int nnc_op_attn_decode_static(const float *q, const void *kcache, const void *vcache, float *out,
                                         int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t max_seq,
                                         int32_t n_ctx, void *cuda_stream) {
    if (!q || !kcache || !vcache || !out) return NNC_ERR_INVALID_ARG;
    if (batch <= 0 || n_kv_heads <= 0 || n_q_heads <= 0 || n_q_heads % n_kv_heads || n_ctx <= 0 || n_ctx > max_seq)
        return NNC_ERR_INVALID_ARG;
    const int G = n_q_heads / n_kv_heads;
    if (!(G == 1 || G == 2 || G == 4 || G == 8)) return NNC_ERR_INVALID_ARG;
    const size_t need = nnc_attn_scratch_bytes(batch, n_q_heads, n_ctx);
    if (need == 0 || need > (size_t)NNC_ATTN_STATIC_SCRATCH_BYTES) {
        fprintf(stderr,
                "nnc_op_attn_decode_static: batch %d x %d query heads needs %zu bytes of scratch, the built-in array "
                "holds %zu; use nnc_op_attn_decode with a caller-supplied buffer\n",
                batch, n_q_heads, need, (size_t)NNC_ATTN_STATIC_SCRATCH_BYTES);
        return NNC_ERR_CAPACITY;
    }
    void *scratch = nullptr;
    if (scratch_for_current_device(&scratch) != cudaSuccess) return NNC_ERR_CUDA;
    // same carve-up and launch as the caller-scratch variant, on the built-in array
    return nnc_op_attn_decode(q, kcache, vcache, out, batch, n_q_heads, n_kv_heads, max_seq, n_ctx, scratch, cuda_stream);
}
