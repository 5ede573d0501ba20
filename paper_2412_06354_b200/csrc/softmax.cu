// Edge softmax over the incoming edges of each node, per head (the attention normalisation of
// the GAT layer named in Sec. 3 "Graph Convolutional Layers"), forward and backward.
// Logits and coefficients are [E,H] in CSR order, so a node's incoming edges are contiguous.
//
// One warp per row for ordinary rows; rows longer than SM_LONG_ROW positions are left to a
// second kernel that gives each of them a whole block, and rows longer than SM_HUB_ROW positions
// (4, 8, 16 or 32 heads) a cluster of eight blocks that combine their results through distributed
// shared memory.  Reductions use fixed shuffle / shared memory trees and a fixed block order, so
// results are bit-reproducible.  All arithmetic is fp32.
#include <mutex>

#include "common.cuh"
#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace gnn {

constexpr int SM_LONG_ROW = 512;  // positions (12 M-edge power-law graph, 8 heads: 2048 is 2 % / 16 % slower forward / backward)
constexpr int SM_BLOCK = 256;

template <typename T> __device__ __forceinline__ float ld_as_f32(const T* p, size_t i);
template <> __device__ __forceinline__ float ld_as_f32<float>(const float* p, size_t i) { return p[i]; }
template <> __device__ __forceinline__ float ld_as_f32<__nv_bfloat16>(const __nv_bfloat16* p, size_t i) { return __bfloat162float(p[i]); }
template <typename T> __device__ __forceinline__ void st_from_f32(T* p, size_t i, float v);
template <> __device__ __forceinline__ void st_from_f32<float>(float* p, size_t i, float v) { p[i] = v; }
template <> __device__ __forceinline__ void st_from_f32<__nv_bfloat16>(__nv_bfloat16* p, size_t i, float v) { p[i] = __float2bfloat16_rn(v); }

struct MaxOp { static __device__ __forceinline__ float id() { return -INFINITY; } static __device__ __forceinline__ float f(float a, float b) { return fmaxf(a, b); } };
struct SumOp { static __device__ __forceinline__ float id() { return 0.f; } static __device__ __forceinline__ float f(float a, float b) { return a + b; } };

// Reduce v over the threads of the group (warp: NT = 32, block: NT = SM_BLOCK) that share the
// same head, i.e. the same (thread id mod H); H is a power of two dividing 32.  Every thread of
// a head class gets the result.
template <class Op, int NT>
__device__ __forceinline__ float reduce_same_head(float v, int H, float* red) {
    const int lane = threadIdx.x & 31;
    for (int o = 16; o >= H; o >>= 1) {
        float other = __shfl_xor_sync(0xffffffffu, v, o);
        v = ((lane & o) == 0) ? Op::f(v, other) : Op::f(other, v);
    }
    if (NT > 32) {
        __syncthreads();
        if (lane < H) red[(threadIdx.x >> 5) * 32 + lane] = v;
        __syncthreads();
        float r = Op::id();
        for (int w = 0; w < NT / 32; ++w) r = Op::f(r, red[w * 32 + (lane % H)]);
        v = r;
    }
    return v;
}

// One row, H a power of two <= 32: thread tid of NT handles flat elements a*H + tid + k*NT,
// whose head is tid mod H throughout.
template <typename T, int NT>
__device__ __forceinline__ void softmax_row_pow2(const T* s, T* alpha, int64_t a, int64_t b, int H, int row,
                                                 float* rowmax, float* rowsum, float* red) {
    const int tid = NT == 32 ? (threadIdx.x & 31) : threadIdx.x;
    const size_t lo = (size_t)a * H, hi = (size_t)b * H;
    float m = -INFINITY;
    for (size_t t = lo + tid; t < hi; t += NT) m = fmaxf(m, ld_as_f32(s, t));
    m = reduce_same_head<MaxOp, NT>(m, H, red);
    float z = 0.f;
    for (size_t t = lo + tid; t < hi; t += NT) z += expf(ld_as_f32(s, t) - m);
    z = reduce_same_head<SumOp, NT>(z, H, red);
    for (size_t t = lo + tid; t < hi; t += NT) st_from_f32(alpha, t, expf(ld_as_f32(s, t) - m) / z);
    if (tid < H && b > a) {
        if (rowmax) rowmax[(size_t)row * H + tid] = m;
        if (rowsum) rowsum[(size_t)row * H + tid] = z;
    }
}

// Any H: one head at a time, threads stride over the positions of the row.
template <typename T, int NT>
__device__ __forceinline__ void softmax_row_any(const T* s, T* alpha, int64_t a, int64_t b, int H, int row,
                                                float* rowmax, float* rowsum, float* red) {
    const int tid = NT == 32 ? (threadIdx.x & 31) : threadIdx.x;
    for (int h = 0; h < H; ++h) {
        float m = -INFINITY;
        for (int64_t p = a + tid; p < b; p += NT) m = fmaxf(m, ld_as_f32(s, (size_t)p * H + h));
        m = reduce_same_head<MaxOp, NT>(m, 1, red);
        float z = 0.f;
        for (int64_t p = a + tid; p < b; p += NT) z += expf(ld_as_f32(s, (size_t)p * H + h) - m);
        z = reduce_same_head<SumOp, NT>(z, 1, red);
        for (int64_t p = a + tid; p < b; p += NT) st_from_f32(alpha, (size_t)p * H + h, expf(ld_as_f32(s, (size_t)p * H + h) - m) / z);
        if (tid == 0 && b > a) {
            if (rowmax) rowmax[(size_t)row * H + h] = m;
            if (rowsum) rowsum[(size_t)row * H + h] = z;
        }
    }
}

// ds = alpha * (dalpha - sum_row alpha*dalpha)
template <typename T, int NT>
__device__ __forceinline__ void softmax_bwd_row(const T* alpha, const T* dalpha, T* ds, int64_t a, int64_t b,
                                                int H, bool pow2, float* red) {
    const int tid = NT == 32 ? (threadIdx.x & 31) : threadIdx.x;
    if (pow2) {
        const size_t lo = (size_t)a * H, hi = (size_t)b * H;
        float d = 0.f;
        for (size_t t = lo + tid; t < hi; t += NT) d = fmaf(ld_as_f32(alpha, t), ld_as_f32(dalpha, t), d);
        d = reduce_same_head<SumOp, NT>(d, H, red);
        for (size_t t = lo + tid; t < hi; t += NT) st_from_f32(ds, t, ld_as_f32(alpha, t) * (ld_as_f32(dalpha, t) - d));
    } else {
        for (int h = 0; h < H; ++h) {
            float d = 0.f;
            for (int64_t p = a + tid; p < b; p += NT) d = fmaf(ld_as_f32(alpha, (size_t)p * H + h), ld_as_f32(dalpha, (size_t)p * H + h), d);
            d = reduce_same_head<SumOp, NT>(d, 1, red);
            for (int64_t p = a + tid; p < b; p += NT) {
                const size_t t = (size_t)p * H + h;
                st_from_f32(ds, t, ld_as_f32(alpha, t) * (ld_as_f32(dalpha, t) - d));
            }
        }
    }
}

// ---- a warp per row with 16-byte (fp32) / 8-byte (bf16) loads: H = 4, 8, 16 or 32.  A lane takes chunks of four
// consecutive values; its chunks are 128 values apart, a multiple of H, so the four heads of a lane never change and
// lanes that are equal modulo H/4 hold the same heads.  Rows of up to 512 values (64 positions at 8 heads) are read
// once and stay in registers through all steps.
template <typename T> __device__ __forceinline__ void ld4(const T* p, size_t i, float* v);
template <> __device__ __forceinline__ void ld4<float>(const float* p, size_t i, float* v) {
    const float4 q = *reinterpret_cast<const float4*>(p + i);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
template <> __device__ __forceinline__ void ld4<__nv_bfloat16>(const __nv_bfloat16* p, size_t i, float* v) {
    const uint2 q = *reinterpret_cast<const uint2*>(p + i);
    v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xFFFF0000u);
    v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xFFFF0000u);
}
template <typename T> __device__ __forceinline__ void st4(T* p, size_t i, const float* v);
template <> __device__ __forceinline__ void st4<float>(float* p, size_t i, const float* v) {
    *reinterpret_cast<float4*>(p + i) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ __forceinline__ void st4<__nv_bfloat16>(__nv_bfloat16* p, size_t i, const float* v) {
    const __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
    *reinterpret_cast<uint2*>(p + i) = make_uint2(*reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b));
}
template <class Op>
__device__ __forceinline__ void reduce_heads4(float* v, int H) {
    const int lane = threadIdx.x & 31, lo = H / 4;
    for (int o = 16; o >= lo; o >>= 1)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float other = __shfl_xor_sync(0xffffffffu, v[j], o);
            v[j] = ((lane & o) == 0) ? Op::f(v[j], other) : Op::f(other, v[j]);
        }
}
constexpr int V4_U = 4;  // chunks a lane keeps in registers

template <typename T>
__device__ __forceinline__ void softmax_row_vec4(const T* __restrict__ s, T* __restrict__ alpha, int64_t a, int64_t b, int H, int row,
                                                 float* rowmax, float* rowsum) {
    const int lane = threadIdx.x & 31;
    const size_t lo = (size_t)a * H;
    const int nch = (int)(((b - a) * H) >> 2);
    float m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY}, z[4] = {0.f, 0.f, 0.f, 0.f};
    if (nch <= 32 * V4_U) {
        float v[V4_U][4];
#pragma unroll
        for (int u = 0; u < V4_U; ++u)
            if (lane + 32 * u < nch) ld4(s, lo + 4 * (size_t)(lane + 32 * u), v[u]);
#pragma unroll
        for (int u = 0; u < V4_U; ++u)
            if (lane + 32 * u < nch)
#pragma unroll
                for (int j = 0; j < 4; ++j) m[j] = fmaxf(m[j], v[u][j]);
        reduce_heads4<MaxOp>(m, H);
#pragma unroll
        for (int u = 0; u < V4_U; ++u)
            if (lane + 32 * u < nch)
#pragma unroll
                for (int j = 0; j < 4; ++j) { v[u][j] = expf(v[u][j] - m[j]); z[j] += v[u][j]; }
        reduce_heads4<SumOp>(z, H);
#pragma unroll
        for (int u = 0; u < V4_U; ++u)
            if (lane + 32 * u < nch) {
#pragma unroll
                for (int j = 0; j < 4; ++j) v[u][j] = v[u][j] / z[j];
                st4(alpha, lo + 4 * (size_t)(lane + 32 * u), v[u]);
            }
    } else {
        float v[4];
        for (int c = lane; c < nch; c += 32) {
            ld4(s, lo + 4 * (size_t)c, v);
#pragma unroll
            for (int j = 0; j < 4; ++j) m[j] = fmaxf(m[j], v[j]);
        }
        reduce_heads4<MaxOp>(m, H);
        for (int c = lane; c < nch; c += 32) {
            ld4(s, lo + 4 * (size_t)c, v);
#pragma unroll
            for (int j = 0; j < 4; ++j) z[j] += expf(v[j] - m[j]);
        }
        reduce_heads4<SumOp>(z, H);
        for (int c = lane; c < nch; c += 32) {
            ld4(s, lo + 4 * (size_t)c, v);
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = expf(v[j] - m[j]) / z[j];
            st4(alpha, lo + 4 * (size_t)c, v);
        }
    }
    if (lane < H / 4) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (rowmax) rowmax[(size_t)row * H + 4 * lane + j] = m[j];
            if (rowsum) rowsum[(size_t)row * H + 4 * lane + j] = z[j];
        }
    }
}

// ds = alpha * (dalpha - sum_row alpha*dalpha), same lane layout
template <typename T>
__device__ __forceinline__ void softmax_bwd_row_vec4(const T* __restrict__ alpha, const T* __restrict__ dalpha, T* __restrict__ ds,
                                                     int64_t a, int64_t b, int H) {
    const int lane = threadIdx.x & 31;
    const size_t lo = (size_t)a * H;
    const int nch = (int)(((b - a) * H) >> 2);
    float d[4] = {0.f, 0.f, 0.f, 0.f};
    if (nch <= 32 * V4_U) {
        float al[V4_U][4], da[V4_U][4];
#pragma unroll
        for (int u = 0; u < V4_U; ++u)
            if (lane + 32 * u < nch) {
                ld4(alpha, lo + 4 * (size_t)(lane + 32 * u), al[u]);
                ld4(dalpha, lo + 4 * (size_t)(lane + 32 * u), da[u]);
            }
#pragma unroll
        for (int u = 0; u < V4_U; ++u)
            if (lane + 32 * u < nch)
#pragma unroll
                for (int j = 0; j < 4; ++j) d[j] = fmaf(al[u][j], da[u][j], d[j]);
        reduce_heads4<SumOp>(d, H);
#pragma unroll
        for (int u = 0; u < V4_U; ++u)
            if (lane + 32 * u < nch) {
#pragma unroll
                for (int j = 0; j < 4; ++j) da[u][j] = al[u][j] * (da[u][j] - d[j]);
                st4(ds, lo + 4 * (size_t)(lane + 32 * u), da[u]);
            }
    } else {
        float x[4], y[4];
        for (int c = lane; c < nch; c += 32) {
            ld4(alpha, lo + 4 * (size_t)c, x);
            ld4(dalpha, lo + 4 * (size_t)c, y);
#pragma unroll
            for (int j = 0; j < 4; ++j) d[j] = fmaf(x[j], y[j], d[j]);
        }
        reduce_heads4<SumOp>(d, H);
        for (int c = lane; c < nch; c += 32) {
            ld4(alpha, lo + 4 * (size_t)c, x);
            ld4(dalpha, lo + 4 * (size_t)c, y);
#pragma unroll
            for (int j = 0; j < 4; ++j) y[j] = x[j] * (y[j] - d[j]);
            st4(ds, lo + 4 * (size_t)c, y);
        }
    }
}

// ---- a block per row with the same 16-byte / 8-byte accesses.  Thread t takes chunks t, t + SM_BLOCK, ...: 4 * SM_BLOCK
// values apart, a multiple of H, so its four heads never change.  A head's value is reduced over the lanes of a warp,
// then over the warps in warp order through shared memory (red: SM_BLOCK floats); every thread gets the result.
template <class Op>
__device__ __forceinline__ void reduce_heads4_block(float* v, int H, float* red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, lo = H / 4;
    reduce_heads4<Op>(v, H);
    __syncthreads();  // red is free again
    if (lane < lo)
#pragma unroll
        for (int j = 0; j < 4; ++j) red[w * 32 + 4 * lane + j] = v[j];
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float r = red[4 * (lane % lo) + j];
        for (int q = 1; q < SM_BLOCK / 32; ++q) r = Op::f(r, red[q * 32 + 4 * (lane % lo) + j]);
        v[j] = r;
    }
}

// Chunks t, t + SM_BLOCK, ... of a row, VB_U loads in flight per thread: body(chunk index, slot) after the loads
// of a batch were issued.
constexpr int VB_U = 4;
template <typename T, class Body>
__device__ __forceinline__ void for_chunks4(const T* __restrict__ p, size_t lo, int64_t nch, Body body, int64_t first = 0) {
    for (int64_t c0 = first + threadIdx.x; c0 < nch; c0 += VB_U * SM_BLOCK) {  // first: a multiple of SM_BLOCK
        float v[VB_U][4];
#pragma unroll
        for (int u = 0; u < VB_U; ++u)
            if (c0 + u * SM_BLOCK < nch) ld4(p, lo + 4 * (size_t)(c0 + u * SM_BLOCK), v[u]);
#pragma unroll
        for (int u = 0; u < VB_U; ++u)
            if (c0 + u * SM_BLOCK < nch) body(c0 + u * SM_BLOCK, v[u]);
    }
}

template <typename T>
__device__ __forceinline__ void softmax_row_vec4_block(const T* __restrict__ s, T* __restrict__ alpha, int64_t a, int64_t b, int H, int row,
                                                       float* rowmax, float* rowsum, float* red) {
    const size_t lo = (size_t)a * H;
    const int64_t nch = ((b - a) * H) >> 2;
    float m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY}, z[4] = {0.f, 0.f, 0.f, 0.f};
    for_chunks4(s, lo, nch, [&](int64_t, float* v) {
#pragma unroll
        for (int j = 0; j < 4; ++j) m[j] = fmaxf(m[j], v[j]);
    });
    reduce_heads4_block<MaxOp>(m, H, red);
    for_chunks4(s, lo, nch, [&](int64_t, float* v) {
#pragma unroll
        for (int j = 0; j < 4; ++j) z[j] += expf(v[j] - m[j]);
    });
    reduce_heads4_block<SumOp>(z, H, red);
    for_chunks4(s, lo, nch, [&](int64_t c, float* v) {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = expf(v[j] - m[j]) / z[j];
        st4(alpha, lo + 4 * (size_t)c, v);
    });
    if (threadIdx.x < H / 4) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (rowmax) rowmax[(size_t)row * H + 4 * threadIdx.x + j] = m[j];
            if (rowsum) rowsum[(size_t)row * H + 4 * threadIdx.x + j] = z[j];
        }
    }
}

template <typename T>
__device__ __forceinline__ void softmax_bwd_row_vec4_block(const T* __restrict__ alpha, const T* __restrict__ dalpha, T* __restrict__ ds,
                                                           int64_t a, int64_t b, int H, float* red) {
    const size_t lo = (size_t)a * H;
    const int64_t nch = ((b - a) * H) >> 2;
    float d[4] = {0.f, 0.f, 0.f, 0.f};
    for_chunks4(alpha, lo, nch, [&](int64_t c, float* x) {
        float y[4];
        ld4(dalpha, lo + 4 * (size_t)c, y);
#pragma unroll
        for (int j = 0; j < 4; ++j) d[j] = fmaf(x[j], y[j], d[j]);
    });
    reduce_heads4_block<SumOp>(d, H, red);
    for_chunks4(alpha, lo, nch, [&](int64_t c, float* x) {
        float y[4];
        ld4(dalpha, lo + 4 * (size_t)c, y);
#pragma unroll
        for (int j = 0; j < 4; ++j) y[j] = x[j] * (y[j] - d[j]);
        st4(ds, lo + 4 * (size_t)c, y);
    });
}

// ---- rows of more than SM_HUB_ROW positions: a cluster of SM_CLUSTER blocks per row.  Block k takes a contiguous
// share of the chunks (a multiple of SM_BLOCK, so that a thread keeps its heads), reduces it as above, leaves the
// per-head result in its shared memory, and after a cluster barrier every block combines the SM_CLUSTER results in
// block order, read through distributed shared memory.  Two result buffers alternate, so a buffer is written
// again only after a later barrier than the one its readers passed.
constexpr int SM_HUB_ROW = 8192;  // positions (2048 and 32768: 5-14 % slower on the same graph)
constexpr int SM_LONG_MINB = 3;   // blocks per SM the long-row kernels are compiled for: they are bound by the loads in
                                  // flight per SM (forward, same graph: 865 / 565 / 481 / 486 us at 1 / 2 / 3 / 4)
constexpr int SM_CLUSTER = 8;

struct HubRows {
    int list[SM_CLUSTER * SM_BLOCK];
    int count;
    float res[2][32];
};

template <class Op>
__device__ __forceinline__ void reduce_heads4_cluster(float* v, int H, float* red, float* res, cg::cluster_group& cluster) {
    const int lane = threadIdx.x & 31, lo = H / 4;
    reduce_heads4_block<Op>(v, H, red);
    if (threadIdx.x < lo)
#pragma unroll
        for (int j = 0; j < 4; ++j) res[4 * threadIdx.x + j] = v[j];
    cluster.sync();
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float r = cluster.map_shared_rank(res, 0)[4 * (lane % lo) + j];
        for (int q = 1; q < SM_CLUSTER; ++q) r = Op::f(r, cluster.map_shared_rank(res, q)[4 * (lane % lo) + j]);
        v[j] = r;
    }
}

// this block's chunks [first, last) of a row of nch chunks
__device__ __forceinline__ void hub_share(int64_t nch, int rank, int64_t* first, int64_t* last) {
    int64_t per = (nch + SM_CLUSTER - 1) / SM_CLUSTER;
    per = (per + SM_BLOCK - 1) / SM_BLOCK * SM_BLOCK;
    *first = rank * per < nch ? rank * per : nch;
    *last = *first + per < nch ? *first + per : nch;
}

template <typename T>
__device__ __forceinline__ void softmax_row_vec4_cluster(const T* __restrict__ s, T* __restrict__ alpha, int64_t a, int64_t b, int H, int row,
                                                         float* rowmax, float* rowsum, float* red, HubRows& hub, cg::cluster_group& cluster) {
    const size_t lo = (size_t)a * H;
    int64_t first, last;
    hub_share(((b - a) * H) >> 2, (int)cluster.block_rank(), &first, &last);
    float m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY}, z[4] = {0.f, 0.f, 0.f, 0.f};
    for_chunks4(s, lo, last, [&](int64_t, float* v) {
#pragma unroll
        for (int j = 0; j < 4; ++j) m[j] = fmaxf(m[j], v[j]);
    }, first);
    reduce_heads4_cluster<MaxOp>(m, H, red, hub.res[0], cluster);
    for_chunks4(s, lo, last, [&](int64_t, float* v) {
#pragma unroll
        for (int j = 0; j < 4; ++j) z[j] += expf(v[j] - m[j]);
    }, first);
    reduce_heads4_cluster<SumOp>(z, H, red, hub.res[1], cluster);
    for_chunks4(s, lo, last, [&](int64_t c, float* v) {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = expf(v[j] - m[j]) / z[j];
        st4(alpha, lo + 4 * (size_t)c, v);
    }, first);
    if (cluster.block_rank() == 0 && threadIdx.x < H / 4) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (rowmax) rowmax[(size_t)row * H + 4 * threadIdx.x + j] = m[j];
            if (rowsum) rowsum[(size_t)row * H + 4 * threadIdx.x + j] = z[j];
        }
    }
}

template <typename T>
__device__ __forceinline__ void softmax_bwd_row_vec4_cluster(const T* __restrict__ alpha, const T* __restrict__ dalpha, T* __restrict__ ds,
                                                             int64_t a, int64_t b, int H, float* red, float* res, cg::cluster_group& cluster) {
    const size_t lo = (size_t)a * H;
    int64_t first, last;
    hub_share(((b - a) * H) >> 2, (int)cluster.block_rank(), &first, &last);
    float d[4] = {0.f, 0.f, 0.f, 0.f};
    for_chunks4(alpha, lo, last, [&](int64_t c, float* x) {
        float y[4];
        ld4(dalpha, lo + 4 * (size_t)c, y);
#pragma unroll
        for (int j = 0; j < 4; ++j) d[j] = fmaf(x[j], y[j], d[j]);
    }, first);
    reduce_heads4_cluster<SumOp>(d, H, red, res, cluster);
    for_chunks4(alpha, lo, last, [&](int64_t c, float* x) {
        float y[4];
        ld4(dalpha, lo + 4 * (size_t)c, y);
#pragma unroll
        for (int j = 0; j < 4; ++j) y[j] = x[j] * (y[j] - d[j]);
        st4(ds, lo + 4 * (size_t)c, y);
    }, first);
}

static __host__ __device__ inline bool head_pow2(int H) { return H >= 1 && H <= 32 && (H & (H - 1)) == 0; }

// Row loops.  LONG = false: every warp strides over the rows and takes the ones of at most
// SM_LONG_ROW positions.  LONG = true: every block takes a contiguous share of the rows, scans it
// NT rows at a time (one rowptr pair per thread), lists the rows longer than SM_LONG_ROW in shared
// memory and works through the list with all its threads.  The list order varies from run to run;
// each row's arithmetic does not depend on it.
struct LongRows {
    int list[512];
    int count;
};

// SUB (non-LONG only): threads per row, 32 (a warp) or 8; LO: rows of at most LO positions belong to another kernel.
template <bool LONG, int NT, int THRESH = SM_LONG_ROW, int SUB = 32, int LO = -1, class Body>
__device__ __forceinline__ void for_each_row(const int64_t* __restrict__ rowptr, int N, LongRows& L, Body body) {
    if (LONG) {
        const int per = (N + (int)gridDim.x - 1) / (int)gridDim.x;
        const int r0 = (int)blockIdx.x * per, r1 = min(N, r0 + per);
        for (int base = r0; base < r1; base += NT) {
            __syncthreads();  // every thread is done with the previous list
            if (threadIdx.x == 0) L.count = 0;
            __syncthreads();
            const int r = base + (int)threadIdx.x;
            if (r < r1 && rowptr[r + 1] - rowptr[r] > THRESH) L.list[atomicAdd(&L.count, 1)] = r;
            __syncthreads();
            const int n = L.count;
            for (int i = 0; i < n; ++i) {
                const int row = L.list[i];
                body(row, rowptr[row], rowptr[row + 1]);
            }
        }
    } else {
        int row = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) / SUB);
        const int stride = (int)((gridDim.x * (int64_t)blockDim.x) / SUB);
        for (; row < N; row += stride) {
            const int64_t a = rowptr[row], b = rowptr[row + 1];
            if (b - a > THRESH || b - a <= LO) continue;  // uniform per group of SUB threads
            body(row, a, b);
        }
    }
}

// Long rows for a grid of clusters, in two phases.  First every block alone: it takes a contiguous share of the rows,
// scans it NT rows at a time and works through the rows above THRESH positions (up to SM_HUB_ROW when hubs is set).
// Then, when hubs is set, every cluster: its blocks scan SM_CLUSTER * NT rows of the cluster's share at a time and
// append the rows above SM_HUB_ROW positions to block 0's list (atomics on distributed shared memory), and the
// whole cluster takes those rows one by one.  Every block of a cluster passes the same number of cluster barriers:
// the windows depend on the cluster's share alone, and the number of hub rows is read from block 0 after a barrier.
// The list orders vary from run to run; no row's arithmetic depends on them.
template <int NT, int THRESH, class Body, class HubBody>
__device__ __forceinline__ void for_each_long_row_cluster(const int64_t* __restrict__ rowptr, int N, bool hubs, LongRows& L, HubRows& Hb,
                                                          cg::cluster_group& cluster, Body body, HubBody hub_body) {
    {
        const int per = (N + (int)gridDim.x - 1) / (int)gridDim.x;
        const int r0 = (int)blockIdx.x * per < N ? (int)blockIdx.x * per : N, r1 = min(N, r0 + per);
        for (int base = r0; base < r1; base += NT) {
            __syncthreads();  // every thread is done with the previous list
            if (threadIdx.x == 0) L.count = 0;
            __syncthreads();
            const int r = base + (int)threadIdx.x;
            if (r < r1) {
                const int64_t len = rowptr[r + 1] - rowptr[r];
                if (len > THRESH && !(hubs && len > SM_HUB_ROW)) L.list[atomicAdd(&L.count, 1)] = r;
            }
            __syncthreads();
            const int n = L.count;
            for (int i = 0; i < n; ++i) {
                const int row = L.list[i];
                body(row, rowptr[row], rowptr[row + 1]);
            }
        }
    }
    if (!hubs) return;  // the same for every block of the grid
    const int rank = (int)cluster.block_rank();
    const int clusters = (int)gridDim.x / SM_CLUSTER, me = (int)blockIdx.x / SM_CLUSTER;
    const int per = (N + clusters - 1) / clusters;
    const int r0 = me * per < N ? me * per : N, r1 = min(N, r0 + per);
    int* count0 = cluster.map_shared_rank(&Hb.count, 0);
    int* list0 = cluster.map_shared_rank(Hb.list, 0);
    for (int base = r0; base < r1; base += SM_CLUSTER * NT) {
        if (threadIdx.x == 0) Hb.count = 0;
        cluster.sync();  // block 0's counter is reset
        const int r = base + rank * NT + (int)threadIdx.x;
        if (r < r1 && rowptr[r + 1] - rowptr[r] > SM_HUB_ROW) list0[atomicAdd(count0, 1)] = r;
        cluster.sync();  // the list is complete
        const int nh = *count0;
        for (int i = 0; i < nh; ++i) {
            const int row = list0[i];
            hub_body(row, rowptr[row], rowptr[row + 1], i);
        }
        cluster.sync();  // nobody reads the list or a result buffer any more
    }
}

template <typename T>
__global__ void __cluster_dims__(SM_CLUSTER, 1, 1) __launch_bounds__(SM_BLOCK, SM_LONG_MINB)
edge_softmax_long_kernel(const int64_t* __restrict__ rowptr, int N, const T* __restrict__ s, int H,
                         T* __restrict__ alpha, float* __restrict__ rowmax, float* __restrict__ rowsum) {
    __shared__ float red[SM_BLOCK];
    __shared__ LongRows lrows;
    __shared__ HubRows hub;
    cg::cluster_group cluster = cg::this_cluster();
    const bool vec4 = H >= 4 && head_pow2(H) && ((reinterpret_cast<uintptr_t>(s) | reinterpret_cast<uintptr_t>(alpha)) & (4 * sizeof(T) - 1)) == 0;
    for_each_long_row_cluster<SM_BLOCK, SM_LONG_ROW>(
        rowptr, N, vec4, lrows, hub, cluster,
        [&](int row, int64_t a, int64_t b) {
            if (vec4) softmax_row_vec4_block<T>(s, alpha, a, b, H, row, rowmax, rowsum, red);
            else if (head_pow2(H)) softmax_row_pow2<T, SM_BLOCK>(s, alpha, a, b, H, row, rowmax, rowsum, red);
            else softmax_row_any<T, SM_BLOCK>(s, alpha, a, b, H, row, rowmax, rowsum, red);
        },
        [&](int row, int64_t a, int64_t b, int) { softmax_row_vec4_cluster<T>(s, alpha, a, b, H, row, rowmax, rowsum, red, hub, cluster); });
}

template <typename T>
__global__ void __cluster_dims__(SM_CLUSTER, 1, 1) __launch_bounds__(SM_BLOCK)
edge_softmax_backward_long_kernel(const int64_t* __restrict__ rowptr, int N, const T* __restrict__ alpha,
                                  const T* __restrict__ dalpha, int H, T* __restrict__ ds) {
    __shared__ float red[SM_BLOCK];
    __shared__ LongRows lrows;
    __shared__ HubRows hub;
    cg::cluster_group cluster = cg::this_cluster();
    const bool vec4 = H >= 4 && head_pow2(H) &&
                      ((reinterpret_cast<uintptr_t>(alpha) | reinterpret_cast<uintptr_t>(dalpha) | reinterpret_cast<uintptr_t>(ds)) & (4 * sizeof(T) - 1)) == 0;
    for_each_long_row_cluster<SM_BLOCK, SM_LONG_ROW>(
        rowptr, N, vec4, lrows, hub, cluster,
        [&](int, int64_t a, int64_t b) {
            if (vec4) softmax_bwd_row_vec4_block<T>(alpha, dalpha, ds, a, b, H, red);
            else softmax_bwd_row<T, SM_BLOCK>(alpha, dalpha, ds, a, b, H, head_pow2(H), red);
        },
        // one result buffer per parity of the hub's place in the list: it is written again two barriers later
        [&](int, int64_t a, int64_t b, int i) { softmax_bwd_row_vec4_cluster<T>(alpha, dalpha, ds, a, b, H, red, hub.res[i & 1], cluster); });
}

template <typename T, bool LONG>
__global__ void __launch_bounds__(SM_BLOCK)
edge_softmax_kernel(const int64_t* __restrict__ rowptr, int N, const T* __restrict__ s, int H,
                    T* __restrict__ alpha, float* __restrict__ rowmax, float* __restrict__ rowsum) {
    __shared__ float red[SM_BLOCK];
    __shared__ LongRows lrows;
    // four heads per lane and 16-byte / 8-byte accesses: H = 4 .. 32, a power of two, and aligned arrays
    const bool vec4 = H >= 4 && head_pow2(H) && ((reinterpret_cast<uintptr_t>(s) | reinterpret_cast<uintptr_t>(alpha)) & (4 * sizeof(T) - 1)) == 0;
    for_each_row<LONG, SM_BLOCK>(rowptr, N, lrows, [&](int row, int64_t a, int64_t b) {
        if (b == a) {
            if ((threadIdx.x & 31) < H) {
                if (rowmax) rowmax[(size_t)row * H + (threadIdx.x & 31)] = 0.f;
                if (rowsum) rowsum[(size_t)row * H + (threadIdx.x & 31)] = 0.f;
            }
            return;
        }
        if (!LONG && vec4) softmax_row_vec4<T>(s, alpha, a, b, H, row, rowmax, rowsum);
        else if (vec4) softmax_row_vec4_block<T>(s, alpha, a, b, H, row, rowmax, rowsum, red);
        else if (head_pow2(H)) softmax_row_pow2<T, LONG ? SM_BLOCK : 32>(s, alpha, a, b, H, row, rowmax, rowsum, red);
        else softmax_row_any<T, LONG ? SM_BLOCK : 32>(s, alpha, a, b, H, row, rowmax, rowsum, red);
    });
}

template <typename T, bool LONG>
__global__ void __launch_bounds__(SM_BLOCK)
edge_softmax_backward_kernel(const int64_t* __restrict__ rowptr, int N, const T* __restrict__ alpha,
                             const T* __restrict__ dalpha, int H, T* __restrict__ ds) {
    __shared__ float red[SM_BLOCK];
    __shared__ LongRows lrows;
    const bool vec4 = H >= 4 && head_pow2(H) &&
                      ((reinterpret_cast<uintptr_t>(alpha) | reinterpret_cast<uintptr_t>(dalpha) | reinterpret_cast<uintptr_t>(ds)) & (4 * sizeof(T) - 1)) == 0;
    for_each_row<LONG, SM_BLOCK>(rowptr, N, lrows, [&](int, int64_t a, int64_t b) {
        if (b == a) return;
        if (!LONG && vec4) softmax_bwd_row_vec4<T>(alpha, dalpha, ds, a, b, H);
        else if (vec4) softmax_bwd_row_vec4_block<T>(alpha, dalpha, ds, a, b, H, red);
        else softmax_bwd_row<T, LONG ? SM_BLOCK : 32>(alpha, dalpha, ds, a, b, H, head_pow2(H), red);
    });
}

// GAT attention coefficients in one kernel: logits z = LeakyReLU(al[col[p],h] + ar[i,h]) are written
// to alpha in the first pass (each thread re-reads only what it wrote), then normalised in place.
// H is a power of two <= 32.
template <bool LONG>
__global__ void __launch_bounds__(SM_BLOCK)
gat_alpha_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col, int N, int H,
                 const float* __restrict__ al, const float* __restrict__ ar, float slope, float* __restrict__ alpha) {
    __shared__ float red[SM_BLOCK];
    constexpr int NT = LONG ? SM_BLOCK : 32;
    const int tid = LONG ? threadIdx.x : (threadIdx.x & 31);
    const int h = tid % H;
    __shared__ LongRows lrows;
    for_each_row<LONG, SM_BLOCK>(rowptr, N, lrows, [&](int row, int64_t a, int64_t b) {
        if (b == a) return;
        const size_t lo = (size_t)a * H, hi = (size_t)b * H;
        const float arv = ar[(size_t)row * H + h];
        float m = -INFINITY;
        for (size_t t = lo + tid; t < hi; t += NT) {
            float z = al[(size_t)col[t / H] * H + h] + arv;
            z = z > 0.f ? z : slope * z;
            alpha[t] = z;
            m = fmaxf(m, z);
        }
        m = reduce_same_head<MaxOp, NT>(m, H, red);
        float zs = 0.f;
        for (size_t t = lo + tid; t < hi; t += NT) zs += expf(alpha[t] - m);
        zs = reduce_same_head<SumOp, NT>(zs, H, red);
        for (size_t t = lo + tid; t < hi; t += NT) alpha[t] = expf(alpha[t] - m) / zs;
    });
}

// ---- position-per-lane layout for H = 4*HV heads: a lane owns whole positions (all heads of an
// edge as HV float4), so a row of up to 32 edges is one vector load per array per lane, and the
// per-head reductions run over lanes (warp) or over lanes and warps (block, long rows).
// NT < 32: the reduction runs over aligned groups of NT lanes, which may have diverged from the other
// groups of the warp, so the shuffles name only the group's lanes.
template <int HV, int NT, bool IS_MAX>
__device__ __forceinline__ void reduce_heads(float (&v)[4 * HV], float* red) {
    constexpr int W = NT < 32 ? NT : 32;
    const unsigned mask = W == 32 ? 0xffffffffu : (((1u << W) - 1u) << ((threadIdx.x & 31) / W * W));
#pragma unroll
    for (int j = 0; j < 4 * HV; ++j) {
#pragma unroll
        for (int o = W / 2; o > 0; o >>= 1) {
            const float other = __shfl_xor_sync(mask, v[j], o);
            v[j] = IS_MAX ? fmaxf(v[j], other) : (((threadIdx.x & o) == 0) ? v[j] + other : other + v[j]);
        }
    }
    if (NT > 32) {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        __syncthreads();
        if (lane == 0) {
#pragma unroll
            for (int j = 0; j < 4 * HV; ++j) red[warp * 32 + j] = v[j];
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < 4 * HV; ++j) {
            float r = IS_MAX ? -INFINITY : 0.f;
            for (int w = 0; w < NT / 32; ++w) r = IS_MAX ? fmaxf(r, red[w * 32 + j]) : r + red[w * 32 + j];
            v[j] = r;
        }
    }
}

constexpr int PL_BLOCK = 512;     // threads per long row
constexpr int PL_LONG_ROW = 1024;  // rows above this many positions get a block instead of a warp (256: +2 % on the attention workload, 2048: +13 %)
// positions per thread and batch (their loads are all in flight together): 32 head values per thread
__host__ __device__ constexpr int pl_unroll(int HV) { return HV <= 2 ? 4 : (HV == 4 ? 2 : 1); }

// Attention coefficients of one row.  The threads take the row in batches of NT*PL_UNR positions;
// the gathers of a batch (col, then al[col]) are independent.  A row that fits in one batch (the
// common case) keeps its logits in registers through the max, sum and normalise steps; longer rows
// park the logits in alpha and re-read them.
template <int HV, bool LONG, int SUB = 32>
__global__ void __launch_bounds__(LONG ? PL_BLOCK : SM_BLOCK, LONG ? 1 : (HV <= 2 ? 3 : 2))
gat_alpha_pl_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col, int N,
                    const float* __restrict__ al, const float* __restrict__ ar, float slope, float* __restrict__ alpha) {
    constexpr int H = 4 * HV, NT = LONG ? PL_BLOCK : SUB, U = LONG ? pl_unroll(HV) : (pl_unroll(HV) > 2 ? 2 : pl_unroll(HV));
    // three kernels share the rows: SUB = 8 takes rows that fit one batch of 8 threads, SUB = 32 the rest up to
    // PL_LONG_ROW, LONG the longer ones
    constexpr int ROW_MAX = LONG ? PL_LONG_ROW : (SUB == 8 ? 8 * U : PL_LONG_ROW), ROW_LO = (!LONG && SUB == 32) ? 8 * U : -1;
    __shared__ float red[LONG ? (PL_BLOCK / 32) * 32 : 1];
    const int tid = LONG ? threadIdx.x : (threadIdx.x & (SUB - 1));
    __shared__ LongRows lrows;
    for_each_row<LONG, PL_BLOCK, ROW_MAX, SUB, ROW_LO>(rowptr, N, lrows, [&](int row, int64_t a, int64_t b) {
        if (b == a) return;
        float arv[H], m[H], zs[H];
#pragma unroll
        for (int q = 0; q < HV; ++q) {
            const float4 t = reinterpret_cast<const float4*>(ar + (size_t)row * H)[q];
            arv[4 * q] = t.x; arv[4 * q + 1] = t.y; arv[4 * q + 2] = t.z; arv[4 * q + 3] = t.w;
        }
#pragma unroll
        for (int j = 0; j < H; ++j) { m[j] = -INFINITY; zs[j] = 0.f; }
        const bool one_batch = (b - a) <= (int64_t)NT * U;
        float z[U][H];
        for (int64_t p0 = a + tid; p0 < b + tid; p0 += (int64_t)NT * U) {  // uniform trip count: p0 - tid < b
            int c[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t p = p0 + (int64_t)u * NT;
                c[u] = p < b ? col[p] : -1;
            }
            float4 t[U][HV];
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (c[u] >= 0) {
#pragma unroll
                    for (int q = 0; q < HV; ++q) t[u][q] = reinterpret_cast<const float4*>(al + (size_t)c[u] * H)[q];
                }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (c[u] < 0) continue;
#pragma unroll
                for (int q = 0; q < HV; ++q) {
                    const float v[4] = {t[u][q].x + arv[4 * q], t[u][q].y + arv[4 * q + 1], t[u][q].z + arv[4 * q + 2], t[u][q].w + arv[4 * q + 3]};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float zz = v[j] > 0.f ? v[j] : slope * v[j];
                        z[u][4 * q + j] = zz;
                        m[4 * q + j] = fmaxf(m[4 * q + j], zz);
                    }
                }
                if (!one_batch) {
                    float4* out = reinterpret_cast<float4*>(alpha + (size_t)(p0 + (int64_t)u * NT) * H);
#pragma unroll
                    for (int q = 0; q < HV; ++q) out[q] = make_float4(z[u][4 * q], z[u][4 * q + 1], z[u][4 * q + 2], z[u][4 * q + 3]);
                }
            }
        }
        reduce_heads<HV, NT, true>(m, red);
        if (one_batch) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (a + tid + (int64_t)u * NT >= b) continue;
#pragma unroll
                for (int j = 0; j < H; ++j) {
                    z[u][j] = expf(z[u][j] - m[j]);
                    zs[j] += z[u][j];
                }
            }
            reduce_heads<HV, NT, false>(zs, red);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t p = a + tid + (int64_t)u * NT;
                if (p >= b) continue;
                float4* out = reinterpret_cast<float4*>(alpha + (size_t)p * H);
#pragma unroll
                for (int q = 0; q < HV; ++q)
                    out[q] = make_float4(z[u][4 * q] / zs[4 * q], z[u][4 * q + 1] / zs[4 * q + 1], z[u][4 * q + 2] / zs[4 * q + 2],
                                         z[u][4 * q + 3] / zs[4 * q + 3]);
            }
            return;
        }
#pragma unroll 4
        for (int64_t p = a + tid; p < b; p += NT) {
            const float4* in = reinterpret_cast<const float4*>(alpha + (size_t)p * H);
#pragma unroll
            for (int q = 0; q < HV; ++q) {
                const float4 t = in[q];
                zs[4 * q] += expf(t.x - m[4 * q]); zs[4 * q + 1] += expf(t.y - m[4 * q + 1]);
                zs[4 * q + 2] += expf(t.z - m[4 * q + 2]); zs[4 * q + 3] += expf(t.w - m[4 * q + 3]);
            }
        }
        reduce_heads<HV, NT, false>(zs, red);
#pragma unroll 4
        for (int64_t p = a + tid; p < b; p += NT) {
            float4* io = reinterpret_cast<float4*>(alpha + (size_t)p * H);
#pragma unroll
            for (int q = 0; q < HV; ++q) {
                const float4 t = io[q];
                io[q] = make_float4(expf(t.x - m[4 * q]) / zs[4 * q], expf(t.y - m[4 * q + 1]) / zs[4 * q + 1],
                                    expf(t.z - m[4 * q + 2]) / zs[4 * q + 2], expf(t.w - m[4 * q + 3]) / zs[4 * q + 3]);
            }
        }
    });
}

// backward rows: d[h] = sum_p alpha*dalpha; dz = alpha*(dalpha - d)*LeakyReLU'(z), written over dalpha; dar = sum_p dz
template <int HV, bool LONG, int SUB = 32>
__global__ void __launch_bounds__(LONG ? PL_BLOCK : SM_BLOCK, LONG ? 1 : (HV <= 2 ? 3 : 2))
gat_rows_bwd_pl_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col, int N,
                       const float* __restrict__ alpha, float* __restrict__ dalpha_dz, const float* __restrict__ al,
                       const float* __restrict__ ar, float slope, float* __restrict__ dar) {
    constexpr int H = 4 * HV, NT = LONG ? PL_BLOCK : SUB, U = LONG ? pl_unroll(HV) : (pl_unroll(HV) > 2 ? 2 : pl_unroll(HV));
    // three kernels share the rows: SUB = 8 takes rows that fit one batch of 8 threads, SUB = 32 the rest up to
    // PL_LONG_ROW, LONG the longer ones
    constexpr int ROW_MAX = LONG ? PL_LONG_ROW : (SUB == 8 ? 8 * U : PL_LONG_ROW), ROW_LO = (!LONG && SUB == 32) ? 8 * U : -1;
    __shared__ float red[LONG ? (PL_BLOCK / 32) * 32 : 1];
    const int tid = LONG ? threadIdx.x : (threadIdx.x & (SUB - 1));
    __shared__ LongRows lrows;
    for_each_row<LONG, PL_BLOCK, ROW_MAX, SUB, ROW_LO>(rowptr, N, lrows, [&](int row, int64_t a, int64_t b) {
        if (b == a) {
            for (int j = tid; j < H; j += NT) dar[(size_t)row * H + j] = 0.f;
            return;
        }
        float arv[H], d[H], sdz[H];
#pragma unroll
        for (int q = 0; q < HV; ++q) {
            const float4 t = reinterpret_cast<const float4*>(ar + (size_t)row * H)[q];
            arv[4 * q] = t.x; arv[4 * q + 1] = t.y; arv[4 * q + 2] = t.z; arv[4 * q + 3] = t.w;
        }
#pragma unroll
        for (int j = 0; j < H; ++j) { d[j] = 0.f; sdz[j] = 0.f; }
#pragma unroll 4
        for (int64_t p = a + tid; p < b; p += NT) {
            const float4* ap = reinterpret_cast<const float4*>(alpha + (size_t)p * H);
            const float4* dp = reinterpret_cast<const float4*>(dalpha_dz + (size_t)p * H);
#pragma unroll
            for (int q = 0; q < HV; ++q) {
                const float4 x = ap[q], y = dp[q];
                d[4 * q] = fmaf(x.x, y.x, d[4 * q]); d[4 * q + 1] = fmaf(x.y, y.y, d[4 * q + 1]);
                d[4 * q + 2] = fmaf(x.z, y.z, d[4 * q + 2]); d[4 * q + 3] = fmaf(x.w, y.w, d[4 * q + 3]);
            }
        }
        reduce_heads<HV, NT, false>(d, red);
        // second pass in batches of U positions per thread: the col -> al gathers of a batch overlap
        for (int64_t p0 = a + tid; p0 < b + tid; p0 += (int64_t)NT * U) {
            int c[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t p = p0 + (int64_t)u * NT;
                c[u] = p < b ? col[p] : -1;
            }
            float4 t[U][HV];
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (c[u] >= 0) {
#pragma unroll
                    for (int q = 0; q < HV; ++q) t[u][q] = reinterpret_cast<const float4*>(al + (size_t)c[u] * H)[q];
                }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (c[u] < 0) continue;
                const int64_t p = p0 + (int64_t)u * NT;
                const float4* ap = reinterpret_cast<const float4*>(alpha + (size_t)p * H);
                float4* dp = reinterpret_cast<float4*>(dalpha_dz + (size_t)p * H);
#pragma unroll
                for (int q = 0; q < HV; ++q) {
                    const float4 x = ap[q], y = dp[q];
                    const float z[4] = {t[u][q].x + arv[4 * q], t[u][q].y + arv[4 * q + 1], t[u][q].z + arv[4 * q + 2], t[u][q].w + arv[4 * q + 3]};
                    const float xa[4] = {x.x, x.y, x.z, x.w}, ya[4] = {y.x, y.y, y.z, y.w};
                    float o[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        o[j] = xa[j] * (ya[j] - d[4 * q + j]) * (z[j] > 0.f ? 1.f : slope);
                        sdz[4 * q + j] += o[j];
                    }
                    dp[q] = make_float4(o[0], o[1], o[2], o[3]);
                }
            }
        }
        reduce_heads<HV, NT, false>(sdz, red);
        if (tid == 0) {
#pragma unroll
            for (int j = 0; j < H; ++j) dar[(size_t)row * H + j] = sdz[j];
        }
    });
}

static int row_grid(int N, bool is_long) {
    const int64_t want = is_long ? N : ceil_div((int64_t)N * 32, SM_BLOCK);
    const int64_t cap = 148 * 8;
    return (int)(want < cap ? (want > 0 ? want : 1) : cap);
}

// grid of whole clusters for the long rows: a block per row up to eight blocks per SM
static int row_grid_cluster(int N) {
    const int64_t want = ceil_div((int64_t)N, SM_CLUSTER), cap = 148;
    return SM_CLUSTER * (int)(want < cap ? (want > 0 ? want : 1) : cap);
}

// grid for a row-strided kernel: one warp per row up to a few waves; one block per row for long rows
static int row_grid_pl(int N, bool is_long) {
    const int64_t want = is_long ? N : ceil_div((int64_t)N * 32, SM_BLOCK);
    const int64_t cap = is_long ? 148 * 2 : (int64_t)148 * 64;
    return (int)(want < cap ? (want > 0 ? want : 1) : cap);
}

// eight threads per row
static int row_grid_sub(int N) {
    const int64_t want = ceil_div((int64_t)N * 8, SM_BLOCK), cap = (int64_t)148 * 64;
    return (int)(want < cap ? (want > 0 ? want : 1) : cap);
}

// The three row tiers (8 threads, a warp, a block per row) touch disjoint rows and none of them fills the
// machine alone (the block tier runs two blocks per SM and is as long as its longest row).  They run side by
// side: the block tier on the caller's stream, the other two on two helper streams that are forked from the
// caller's stream and joined back into it with events, so the call keeps its place in the caller's stream order.
// The helper streams and events are created on the first call on a device (make that call outside any stream
// capture); if they cannot be had, the tiers run one after the other.
struct TierStreams {
    cudaStream_t s[2];
    cudaEvent_t fork, join[2];
    int state;  // 0: not tried, 1: ready, -1: unavailable
};
static std::mutex g_tier_mutex;
static TierStreams g_tier[64];

// the current device's helper streams, created on first use; nullptr if they cannot be had (call with the mutex held)
static TierStreams* tier_streams() {
    int dev = -1;
    TierStreams* t = nullptr;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
        t = &g_tier[dev];
        if (t->state == 0) {
            bool ok = cudaStreamCreateWithFlags(&t->s[0], cudaStreamNonBlocking) == cudaSuccess &&
                      cudaStreamCreateWithFlags(&t->s[1], cudaStreamNonBlocking) == cudaSuccess &&
                      cudaEventCreateWithFlags(&t->fork, cudaEventDisableTiming) == cudaSuccess &&
                      cudaEventCreateWithFlags(&t->join[0], cudaEventDisableTiming) == cudaSuccess &&
                      cudaEventCreateWithFlags(&t->join[1], cudaEventDisableTiming) == cudaSuccess;
            t->state = ok ? 1 : -1;
            if (!ok) (void)cudaGetLastError();
        }
        if (t->state != 1) t = nullptr;
    }
    return t;
}

// A side branch of the caller's stream: work enqueued on the returned stream starts after everything enqueued on
// st so far; side_join makes st wait for it.  Returns st itself if no helper stream is available.
cudaStream_t side_fork(cudaStream_t st) {
    std::lock_guard<std::mutex> lock(g_tier_mutex);
    TierStreams* t = tier_streams();
    if (!t || cudaEventRecord(t->fork, st) != cudaSuccess || cudaStreamWaitEvent(t->s[0], t->fork, 0) != cudaSuccess) {
        (void)cudaGetLastError();
        return st;
    }
    return t->s[0];
}
void side_join(cudaStream_t st, cudaStream_t side) {
    if (side == st) return;
    std::lock_guard<std::mutex> lock(g_tier_mutex);
    TierStreams* t = tier_streams();
    if (!t) return;
    cudaEventRecord(t->join[0], side);
    cudaStreamWaitEvent(st, t->join[0], 0);
}

template <class Long, class Warp, class Sub>
static void run_row_tiers(cudaStream_t st, Long run_long, Warp run_warp, Sub run_sub) {
    std::lock_guard<std::mutex> lock(g_tier_mutex);  // one host thread at a time forks and joins through the shared events
    TierStreams* t = tier_streams();
    if (!t || cudaEventRecord(t->fork, st) != cudaSuccess || cudaStreamWaitEvent(t->s[0], t->fork, 0) != cudaSuccess ||
        cudaStreamWaitEvent(t->s[1], t->fork, 0) != cudaSuccess) {
        (void)cudaGetLastError();
        run_long(st); run_warp(st); run_sub(st);
        return;
    }
    run_long(st);
    run_warp(t->s[0]);
    run_sub(t->s[1]);
    cudaEventRecord(t->join[0], t->s[0]);
    cudaEventRecord(t->join[1], t->s[1]);
    cudaStreamWaitEvent(st, t->join[0], 0);
    cudaStreamWaitEvent(st, t->join[1], 0);
}

gnn_status gat_alpha(const gnn_csr* g, const float* al, const float* ar, float slope, int H, float* alpha, cudaStream_t st) {
    if (g->N == 0 || g->E == 0) return GNN_OK;
    const int wg = row_grid_pl(g->N, false), lg = row_grid_pl(g->N, true), sg = row_grid_sub(g->N);
#define GNN_GA(HV)                                                                                                                       \
    run_row_tiers(                                                                                                                       \
        st, [&](cudaStream_t q) { gat_alpha_pl_kernel<HV, true><<<lg, PL_BLOCK, 0, q>>>(g->rowptr, g->col, g->N, al, ar, slope, alpha); }, \
        [&](cudaStream_t q) { gat_alpha_pl_kernel<HV, false><<<wg, SM_BLOCK, 0, q>>>(g->rowptr, g->col, g->N, al, ar, slope, alpha); },    \
        [&](cudaStream_t q) { gat_alpha_pl_kernel<HV, false, 8><<<sg, SM_BLOCK, 0, q>>>(g->rowptr, g->col, g->N, al, ar, slope, alpha); });
    if (H == 4) { GNN_GA(1) } else if (H == 8) { GNN_GA(2) } else if (H == 16) { GNN_GA(4) } else if (H == 32) { GNN_GA(8) } else {
        run_row_tiers(  // the two tiers write disjoint rows: side by side
            st, [&](cudaStream_t q) { gat_alpha_kernel<true><<<row_grid(g->N, true), SM_BLOCK, 0, q>>>(g->rowptr, g->col, g->N, H, al, ar, slope, alpha); },
            [&](cudaStream_t q) { gat_alpha_kernel<false><<<row_grid(g->N, false), SM_BLOCK, 0, q>>>(g->rowptr, g->col, g->N, H, al, ar, slope, alpha); },
            [&](cudaStream_t) {});
    }
#undef GNN_GA
    GNN_CHECK_LAUNCH("gnn_gat_fused (attention coefficients)");
    return GNN_OK;
}

// returns false if H is not handled here (caller falls back to its generic kernel)
bool gat_rows_backward_pl(const gnn_csr* g, const float* alpha, float* dalpha_dz, const float* al, const float* ar,
                          float slope, int H, float* dar, cudaStream_t st) {
    const int wg = row_grid_pl(g->N, false), lg = row_grid_pl(g->N, true), sg = row_grid_sub(g->N);
#define GNN_GB(HV)                                                                                                                                       \
    run_row_tiers(                                                                                                                                       \
        st, [&](cudaStream_t q) { gat_rows_bwd_pl_kernel<HV, true><<<lg, PL_BLOCK, 0, q>>>(g->rowptr, g->col, g->N, alpha, dalpha_dz, al, ar, slope, dar); }, \
        [&](cudaStream_t q) { gat_rows_bwd_pl_kernel<HV, false><<<wg, SM_BLOCK, 0, q>>>(g->rowptr, g->col, g->N, alpha, dalpha_dz, al, ar, slope, dar); },    \
        [&](cudaStream_t q) { gat_rows_bwd_pl_kernel<HV, false, 8><<<sg, SM_BLOCK, 0, q>>>(g->rowptr, g->col, g->N, alpha, dalpha_dz, al, ar, slope, dar); });
    if (H == 4) { GNN_GB(1) } else if (H == 8) { GNN_GB(2) } else if (H == 16) { GNN_GB(4) } else if (H == 32) { GNN_GB(8) } else return false;
#undef GNN_GB
    return true;
}

}  // namespace gnn

using namespace gnn;

extern "C" {

gnn_status gnn_edge_softmax(const gnn_csr* g, const void* logits_EH, int H, gnn_dtype dtype,
                            void* alpha_EH, float* rowmax, float* rowsum, gnn_stream stream) {
    const char* who = "gnn_edge_softmax";
    GNN_REQUIRE(g && g->rowptr && H >= 1, GNN_ERR_INVALID_ARG, "%s: bad argument", who);
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "%s: bad dtype", who);
    if (g->N == 0) return GNN_OK;
    GNN_REQUIRE(g->E == 0 || (logits_EH && alpha_EH), GNN_ERR_INVALID_ARG, "%s: null argument", who);
    cudaStream_t st = as_stream(stream);
    const int wgrid = row_grid(g->N, false), lgrid = row_grid_cluster(g->N);
    // the two row tiers write disjoint rows: side by side (the long rows' blocks beside the warps of the short ones)
    if (dtype == GNN_F32)
        run_row_tiers(
            st, [&](cudaStream_t q) { edge_softmax_long_kernel<float><<<lgrid, SM_BLOCK, 0, q>>>(g->rowptr, g->N, (const float*)logits_EH, H, (float*)alpha_EH, rowmax, rowsum); },
            [&](cudaStream_t q) { edge_softmax_kernel<float, false><<<wgrid, SM_BLOCK, 0, q>>>(g->rowptr, g->N, (const float*)logits_EH, H, (float*)alpha_EH, rowmax, rowsum); },
            [&](cudaStream_t) {});
    else
        run_row_tiers(
            st, [&](cudaStream_t q) { edge_softmax_long_kernel<__nv_bfloat16><<<lgrid, SM_BLOCK, 0, q>>>(g->rowptr, g->N, (const __nv_bfloat16*)logits_EH, H, (__nv_bfloat16*)alpha_EH, rowmax, rowsum); },
            [&](cudaStream_t q) { edge_softmax_kernel<__nv_bfloat16, false><<<wgrid, SM_BLOCK, 0, q>>>(g->rowptr, g->N, (const __nv_bfloat16*)logits_EH, H, (__nv_bfloat16*)alpha_EH, rowmax, rowsum); },
            [&](cudaStream_t) {});
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

gnn_status gnn_edge_softmax_backward(const gnn_csr* g, const void* alpha_EH, const void* dAlpha_EH,
                                     int H, gnn_dtype dtype, void* dLogits_EH, gnn_stream stream) {
    const char* who = "gnn_edge_softmax_backward";
    GNN_REQUIRE(g && g->rowptr && H >= 1, GNN_ERR_INVALID_ARG, "%s: bad argument", who);
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "%s: bad dtype", who);
    if (g->N == 0 || g->E == 0) return GNN_OK;
    GNN_REQUIRE(alpha_EH && dAlpha_EH && dLogits_EH, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    cudaStream_t st = as_stream(stream);
    const int wgrid = row_grid(g->N, false), lgrid = row_grid_cluster(g->N);
    if (dtype == GNN_F32)
        run_row_tiers(
            st, [&](cudaStream_t q) { edge_softmax_backward_long_kernel<float><<<lgrid, SM_BLOCK, 0, q>>>(g->rowptr, g->N, (const float*)alpha_EH, (const float*)dAlpha_EH, H, (float*)dLogits_EH); },
            [&](cudaStream_t q) { edge_softmax_backward_kernel<float, false><<<wgrid, SM_BLOCK, 0, q>>>(g->rowptr, g->N, (const float*)alpha_EH, (const float*)dAlpha_EH, H, (float*)dLogits_EH); },
            [&](cudaStream_t) {});
    else
        run_row_tiers(
            st, [&](cudaStream_t q) { edge_softmax_backward_long_kernel<__nv_bfloat16><<<lgrid, SM_BLOCK, 0, q>>>(g->rowptr, g->N, (const __nv_bfloat16*)alpha_EH, (const __nv_bfloat16*)dAlpha_EH, H, (__nv_bfloat16*)dLogits_EH); },
            [&](cudaStream_t q) { edge_softmax_backward_kernel<__nv_bfloat16, false><<<wgrid, SM_BLOCK, 0, q>>>(g->rowptr, g->N, (const __nv_bfloat16*)alpha_EH, (const __nv_bfloat16*)dAlpha_EH, H, (__nv_bfloat16*)dLogits_EH); },
            [&](cudaStream_t) {});
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

}  // extern "C"
