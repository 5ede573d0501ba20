// Shared host/device helpers of libgnn_b200 (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "gnn.h"

#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ < 1000)
#error "libgnn_b200 is written for sm_100a"
#endif

namespace gnn {

void set_error(const char* fmt, ...);

#define GNN_FAIL(code, ...)            \
    do {                               \
        ::gnn::set_error(__VA_ARGS__); \
        return (code);                 \
    } while (0)

#define GNN_REQUIRE(cond, code, ...)              \
    do {                                          \
        if (!(cond)) GNN_FAIL(code, __VA_ARGS__); \
    } while (0)

// after a launch: report launch-configuration errors without synchronising
#define GNN_CHECK_LAUNCH(name)                                                                 \
    do {                                                                                       \
        cudaError_t e_ = cudaGetLastError();                                                   \
        if (e_ != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "%s: %s", name, cudaGetErrorString(e_)); \
    } while (0)

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline cudaStream_t as_stream(gnn_stream s) { return reinterpret_cast<cudaStream_t>(s); }
static inline int elem_size(gnn_dtype d) { return d == GNN_F32 ? 4 : 2; }
static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }
// grid for a grid-stride loop over n items
static inline int grid_for(int64_t n, int threads) {
    int64_t b = ceil_div(n > 0 ? n : 1, threads);
    int64_t cap = 148 * 32;
    return (int)(b < cap ? b : cap);
}

// ---------------------------------------------------------------- device helpers
#ifdef __CUDACC__

// 16-byte global loads/stores with L2 cache policies (createpolicy + .L2::cache_hint).
//   feature rows that are gathered many times: keep in L2 (evict_last)
//   index / weight / output streams touched once: evict_first, no L1 allocation
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
#ifndef PF_L1_POLICY
#define PF_L1_POLICY 0
#endif
__device__ __forceinline__ uint4 ld_hint16(const void* p, uint64_t pol) {
    uint4 v;
#if PF_L1_POLICY == 0
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
#elif PF_L1_POLICY == 1
    asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
#else
    asm volatile("ld.global.nc.L1::evict_last.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
#endif
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ int ld_hint_i32(const int* p, uint64_t pol) {
    int v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.s32 %0, [%1], %2;" : "=r"(v) : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ float ld_hint_f32(const float* p, uint64_t pol) {
    float v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.f32 %0, [%1], %2;" : "=f"(v) : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ void st_stream16(void* p, uint4 v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}

// One 16-byte chunk of a feature row as fp32 lanes: 4 values for f32, 8 for bf16.
template <typename T>
struct Chunk;
template <>
struct Chunk<float> {
    static constexpr int N = 4;
    __device__ __forceinline__ static void unpack(uint4 u, float* f) {
        f[0] = __uint_as_float(u.x);
        f[1] = __uint_as_float(u.y);
        f[2] = __uint_as_float(u.z);
        f[3] = __uint_as_float(u.w);
    }
    __device__ __forceinline__ static uint4 pack(const float* f) {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                          __float_as_uint(f[3]));
    }
};
template <>
struct Chunk<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ __forceinline__ static void unpack(uint4 u, float* f) {
        // bf16 -> f32 is a 16-bit shift: exact
        f[0] = __uint_as_float(u.x << 16);
        f[1] = __uint_as_float(u.x & 0xFFFF0000u);
        f[2] = __uint_as_float(u.y << 16);
        f[3] = __uint_as_float(u.y & 0xFFFF0000u);
        f[4] = __uint_as_float(u.z << 16);
        f[5] = __uint_as_float(u.z & 0xFFFF0000u);
        f[6] = __uint_as_float(u.w << 16);
        f[7] = __uint_as_float(u.w & 0xFFFF0000u);
    }
    __device__ __forceinline__ static uint32_t pack2(float lo, float hi) {
        __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);  // round to nearest even
        return *reinterpret_cast<uint32_t*>(&b);
    }
    __device__ __forceinline__ static uint4 pack(const float* f) {
        return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]),
                          pack2(f[6], f[7]));
    }
};

// first index r in [0, n] with a[r] >= v  (a non-decreasing, n entries)
__device__ __forceinline__ int lower_bound_i64(const int64_t* a, int n, int64_t v) {
    int lo = 0, hi = n;
    while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (a[mid] < v) lo = mid + 1; else hi = mid;
    }
    return lo;
}

#endif  // __CUDACC__
}  // namespace gnn
