// Shared device/host helpers of the vgc CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdio>
#include <cstdlib>

#include "vgc.h"

#ifndef __CUDA_ARCH__
#define VGC_HOST_ONLY 1
#endif

namespace vgc {

constexpr int kWarp = 32;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// VGC_DEBUG=1 in the environment (read once): a failing CUDA call is named on stderr before the status is returned
inline bool debug_enabled()
{
    static const bool on = getenv("VGC_DEBUG") != nullptr;
    return on;
}
inline void report_cuda_error(cudaError_t e, const char *what, const char *file, int line)
{
    if (debug_enabled()) fprintf(stderr, "vgc: %s:%d: %s -> %s\n", file, line, what, cudaGetErrorString(e));
}
#define VGC_CUDA_OK(expr)                                                  \
    do {                                                                   \
        const cudaError_t vgc_e_ = (expr);                                 \
        if (vgc_e_ != cudaSuccess) {                                       \
            ::vgc::report_cuda_error(vgc_e_, #expr, __FILE__, __LINE__);   \
            return VGC_ERR_CUDA;                                           \
        }                                                                  \
    } while (0)

// Number of kernels this library has enqueued since it was loaded (benchmark bookkeeping).
extern unsigned long long g_launches;
inline void count_launch(unsigned k = 1) { g_launches += k; }

__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31; }

__device__ __forceinline__ uint64_t ld_volatile_u64(const uint64_t *p)
{
    uint64_t v;
    asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_volatile_u64(uint64_t *p, uint64_t v)
{
    asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_volatile_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Streaming (evict-first) 128-bit accesses for data touched once per call.
__device__ __forceinline__ float4 ld_stream_f4(const float *p)
{
    float4 v;
    asm volatile("ld.global.cs.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream_f4(float *p, float4 v)
{
    asm volatile("st.global.cs.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}

// Index of the weight tensor holding flat index i: the k with offs[k] <= i < offs[k+1].
// offs has K+1 non-decreasing entries, offs[0] = 0; empty tensors are skipped.
__device__ __forceinline__ int group_of(const uint32_t *offs, int K, uint32_t i)
{
    int lo = 0, hi = K;   // invariant: offs[lo] <= i, answer in [lo, hi)
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (offs[mid] <= i) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ uint64_t warp_sum_u64(uint64_t x)
{
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
    return x;
}

}  // namespace vgc
