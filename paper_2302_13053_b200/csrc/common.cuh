// Shared host/device helpers of the retexo CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "retexo.h"

namespace retexo {

constexpr int kWarp = 32;
constexpr size_t kAlign = 256;

inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

// Bump allocator over the caller's workspace (host-side pointer arithmetic only).
struct Arena {
    char* base;
    size_t cap;
    size_t off;
    Arena(void* p, size_t bytes) : base(static_cast<char*>(p)), cap(bytes), off(0) {}
    template <typename T>
    T* take(size_t count) {
        size_t bytes = align_up(count * sizeof(T));
        T* p = reinterpret_cast<T*>(base + off);
        off += bytes;
        return p;
    }
    bool ok() const { return off <= cap; }
};

// Same arithmetic without a buffer, for the *_workspace_size queries.
struct Sizer {
    size_t off = 0;
    template <typename T>
    void take(size_t count) { off += align_up(count * sizeof(T)); }
};

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline int sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return n;
}

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? RETEXO_OK : RETEXO_ERR_CUDA; }

#define RETEXO_CUDA_TRY(expr)                                  \
    do {                                                       \
        if ((expr) != cudaSuccess) {                           \
            (void)cudaGetLastError();                          \
            return RETEXO_ERR_CUDA;                            \
        }                                                      \
    } while (0)

#define RETEXO_TRY(expr)                  \
    do {                                  \
        int rc__ = (expr);                \
        if (rc__ != RETEXO_OK) return rc__; \
    } while (0)

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

__device__ __forceinline__ float bf16_to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ __nv_bfloat16 f32_to_bf16(float v) { return __float2bfloat16_rn(v); }
// value of v after rounding to bf16, kept as fp32
__device__ __forceinline__ float round_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

}  // namespace retexo
