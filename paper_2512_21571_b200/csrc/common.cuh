// Device-side helpers shared by the kernels of libnnc: bf16 unpacking, warp reductions, streaming loads,
// programmatic-dependent-launch controls.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace nnc {

constexpr int kHeadDim = 128;
constexpr int kWarp = 32;

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ float bf16_bits_to_f32(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }

// round-to-nearest-even fp32 -> bf16 bit pattern
__device__ __forceinline__ uint16_t f32_to_bf16_bits(float f) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    return (uint32_t)f32_to_bf16_bits(lo) | ((uint32_t)f32_to_bf16_bits(hi) << 16);
}

// two floats -> packed fp16 pair (lo in bits 0..15), round to nearest even, saturating at +-65504 instead of infinity
__device__ __forceinline__ uint32_t pack_f16x2_sat(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// 16-byte read-only streaming load: weights and cache lines are used once per step, keep them out of L1.
__device__ __forceinline__ uint4 ldg_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Programmatic dependent launch: a kernel launched with the programmatic-stream-serialization attribute may
// start while its predecessor drains.  Everything that reads the predecessor's output sits after
// pdl_wait(); weight prefetches (which depend on nothing) sit before it.  Without the attribute both are
// no-ops.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- bounds-checked debugging build (-DNNC_BOUNDS_CHECK) -------------------------------------------------
// The normal library trusts the extents its launchers computed.  The checked build compares the indices that rest
// on such an assumption (a cache position against the cache capacity, a row range against the matrix, a scratch
// slot against the scratch size) with the extent at the point of use: a miss is COUNTED in a device word and the
// access is skipped -- never a trap, never an out-of-range access -- and nnc_bounds_check_report() reads the count
// and the code of the first miss.  NNC_BC(cond, code) evaluates to `cond` in the checked build and to `true` in the
// normal one, so it wraps only conditions the normal build does not need; guards that are part of a kernel's logic
// stay ordinary `if`s.  Each translation unit holds its own counter (no relocatable device code) and registers a
// reader for it.
#ifdef NNC_BOUNDS_CHECK
static __device__ unsigned g_bc_words[2];   // {misses, code of the first miss}
void bc_register(void (*read_and_clear)(unsigned *misses, unsigned *first_code));
static void bc_read_this_tu(unsigned *misses, unsigned *first_code) {
    unsigned w[2] = {0, 0}, zero[2] = {0, 0};
    cudaMemcpyFromSymbol(w, g_bc_words, sizeof(w));
    cudaMemcpyToSymbol(g_bc_words, zero, sizeof(zero));
    *misses = w[0];
    *first_code = w[1];
}
namespace { struct BcRegistrar { BcRegistrar() { bc_register(&bc_read_this_tu); } } g_bc_registrar; }
__device__ __forceinline__ bool bc_check(bool ok, unsigned code) {
    if (!ok && atomicAdd(&g_bc_words[0], 1u) == 0u) g_bc_words[1] = code;
    return ok;
}
#define NNC_BC(cond, code) ::nnc::bc_check((cond), (code))
#else
#define NNC_BC(cond, code) true
#endif

// ---- per-CTA timeline records (tracing builds only: -DNNC_TRACE) -----------------------------------------
// Every CTA appends {kernel id, block, SM, start, end} (globaltimer ns) to a device buffer when it exits;
// nnc_trace_dump() copies the buffer to the host.  Compiled out of the normal library.  Each translation unit
// holds its own copy of the two pointers (no relocatable device code) and registers a binder for them.
#ifndef NNC_TRACE_ALL_CTAS
#define NNC_TRACE_ALL_CTAS 0   // tracing builds may record per-unit events of every CTA instead of CTA 0's only
#endif
#ifdef NNC_TRACE
struct TraceRec { unsigned kid, block, smid, mark; unsigned long long t0, t1; unsigned mark2, mark3, pad0, pad1; };
constexpr unsigned kTraceMax = 1u << 20;
static __device__ TraceRec *g_trace_buf;
static __device__ unsigned *g_trace_cnt;
void trace_register(void (*bind)(TraceRec *, unsigned *));
static void trace_bind_this_tu(TraceRec *buf, unsigned *cnt) {
    cudaMemcpyToSymbol(g_trace_buf, &buf, sizeof(buf));
    cudaMemcpyToSymbol(g_trace_cnt, &cnt, sizeof(cnt));
}
namespace { struct TraceRegistrar { TraceRegistrar() { trace_register(&trace_bind_this_tu); } } g_trace_registrar; }
struct TraceScope {
    unsigned kid, mark, mark2, mark3, c0; unsigned long long t0;   // c0: SM cycle counter at entry (the record keeps the cycles spent)
    __device__ __forceinline__ unsigned since() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return (unsigned)(t - t0); }
    __device__ __forceinline__ void set_mark() { mark = since(); }
    __device__ __forceinline__ void set_mark2() { mark2 = since(); }
    __device__ __forceinline__ void set_mark3() { mark3 = since(); }
    __device__ __forceinline__ TraceScope(unsigned k) : kid(k), mark(0), mark2(0), mark3(0) {
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
        asm volatile("mov.u32 %0, %clock;" : "=r"(c0));
    }
    __device__ __forceinline__ ~TraceScope() {
        if (threadIdx.x == 0 && g_trace_buf) {
            unsigned long long t1; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
            unsigned sm; asm volatile("mov.u32 %0, %smid;" : "=r"(sm));
            unsigned c1; asm volatile("mov.u32 %0, %clock;" : "=r"(c1));
            const unsigned i = atomicAdd(g_trace_cnt, 1u);
            if (i < kTraceMax) g_trace_buf[i] = TraceRec{kid, blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z), sm, mark, t0, t1, mark2, mark3, c1 - c0, 0};
        }
    }
};
__device__ __forceinline__ unsigned long long trace_now() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
// free-standing record: [t0, t1] plus one extra interval end (mark = t_mark - t0)
__device__ __forceinline__ void trace_event(unsigned kid, unsigned long long t0, unsigned long long t_mark, unsigned long long t1) {
    if (!g_trace_buf) return;
    unsigned sm; asm volatile("mov.u32 %0, %smid;" : "=r"(sm));
    const unsigned i = atomicAdd(g_trace_cnt, 1u);
    if (i < kTraceMax) g_trace_buf[i] = TraceRec{kid, blockIdx.x, sm, (unsigned)(t_mark - t0), t0, t1, 0, 0, 0, 0};
}
#define NNC_TRACE_EVENT(kid, t0, tm, t1) trace_event(kid, t0, tm, t1)
#define NNC_TRACE_NOW() trace_now()
#define NNC_TRACE_SCOPE(kid) TraceScope nnc_trace_scope__(kid)
#define NNC_TRACE_MARK() nnc_trace_scope__.set_mark()
#define NNC_TRACE_MARK2() nnc_trace_scope__.set_mark2()
#define NNC_TRACE_MARK3() nnc_trace_scope__.set_mark3()
#else
#define NNC_TRACE_EVENT(kid, t0, tm, t1)
#define NNC_TRACE_NOW() 0ull
#define NNC_TRACE_SCOPE(kid)
#define NNC_TRACE_MARK()
#define NNC_TRACE_MARK2()
#define NNC_TRACE_MARK3()
#endif

}  // namespace nnc
