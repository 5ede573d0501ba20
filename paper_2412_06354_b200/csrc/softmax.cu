// Edge softmax over the incoming edges of each node, per head (the attention normalisation of
// the GAT layer named in Sec. 3 "Graph Convolutional Layers"), forward and backward.
// Logits and coefficients are [E,H] in CSR order, so a node's incoming edges are contiguous.
//
// One warp per row for ordinary rows; rows longer than SM_LONG_ROW positions are left to a
// second kernel that gives each of them a whole block.  Reductions use fixed shuffle / shared
// memory trees, so results are bit-reproducible.  All arithmetic is fp32.
#include "common.cuh"

namespace gnn {

constexpr int SM_LONG_ROW = 2048;  // positions
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

static __host__ __device__ inline bool head_pow2(int H) { return H >= 1 && H <= 32 && (H & (H - 1)) == 0; }

template <typename T, bool LONG>
__global__ void __launch_bounds__(SM_BLOCK)
edge_softmax_kernel(const int64_t* __restrict__ rowptr, int N, const T* __restrict__ s, int H,
                    T* __restrict__ alpha, float* __restrict__ rowmax, float* __restrict__ rowsum) {
    __shared__ float red[SM_BLOCK];
    const int row = LONG ? blockIdx.x : (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
    if (row >= N) return;
    const int64_t a = rowptr[row], b = rowptr[row + 1];
    const bool is_long = (b - a) > SM_LONG_ROW;
    if (is_long != LONG) return;  // uniform per warp (LONG = false) or per block (LONG = true)
    if (b == a) {
        if (!LONG && (threadIdx.x & 31) < H) {
            if (rowmax) rowmax[(size_t)row * H + (threadIdx.x & 31)] = 0.f;
            if (rowsum) rowsum[(size_t)row * H + (threadIdx.x & 31)] = 0.f;
        }
        return;
    }
    if (head_pow2(H)) softmax_row_pow2<T, LONG ? SM_BLOCK : 32>(s, alpha, a, b, H, row, rowmax, rowsum, red);
    else softmax_row_any<T, LONG ? SM_BLOCK : 32>(s, alpha, a, b, H, row, rowmax, rowsum, red);
}

template <typename T, bool LONG>
__global__ void __launch_bounds__(SM_BLOCK)
edge_softmax_backward_kernel(const int64_t* __restrict__ rowptr, int N, const T* __restrict__ alpha,
                             const T* __restrict__ dalpha, int H, T* __restrict__ ds) {
    __shared__ float red[SM_BLOCK];
    const int row = LONG ? blockIdx.x : (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
    if (row >= N) return;
    const int64_t a = rowptr[row], b = rowptr[row + 1];
    if (((b - a) > SM_LONG_ROW) != LONG || b == a) return;
    softmax_bwd_row<T, LONG ? SM_BLOCK : 32>(alpha, dalpha, ds, a, b, H, head_pow2(H), red);
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
    const int wgrid = (int)ceil_div((int64_t)g->N * 32, SM_BLOCK);
    if (dtype == GNN_F32) {
        edge_softmax_kernel<float, false><<<wgrid, SM_BLOCK, 0, st>>>(g->rowptr, g->N, (const float*)logits_EH, H, (float*)alpha_EH, rowmax, rowsum);
        edge_softmax_kernel<float, true><<<g->N, SM_BLOCK, 0, st>>>(g->rowptr, g->N, (const float*)logits_EH, H, (float*)alpha_EH, rowmax, rowsum);
    } else {
        edge_softmax_kernel<__nv_bfloat16, false><<<wgrid, SM_BLOCK, 0, st>>>(g->rowptr, g->N, (const __nv_bfloat16*)logits_EH, H, (__nv_bfloat16*)alpha_EH, rowmax, rowsum);
        edge_softmax_kernel<__nv_bfloat16, true><<<g->N, SM_BLOCK, 0, st>>>(g->rowptr, g->N, (const __nv_bfloat16*)logits_EH, H, (__nv_bfloat16*)alpha_EH, rowmax, rowsum);
    }
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
    const int wgrid = (int)ceil_div((int64_t)g->N * 32, SM_BLOCK);
    if (dtype == GNN_F32) {
        edge_softmax_backward_kernel<float, false><<<wgrid, SM_BLOCK, 0, st>>>(g->rowptr, g->N, (const float*)alpha_EH, (const float*)dAlpha_EH, H, (float*)dLogits_EH);
        edge_softmax_backward_kernel<float, true><<<g->N, SM_BLOCK, 0, st>>>(g->rowptr, g->N, (const float*)alpha_EH, (const float*)dAlpha_EH, H, (float*)dLogits_EH);
    } else {
        edge_softmax_backward_kernel<__nv_bfloat16, false><<<wgrid, SM_BLOCK, 0, st>>>(g->rowptr, g->N, (const __nv_bfloat16*)alpha_EH, (const __nv_bfloat16*)dAlpha_EH, H, (__nv_bfloat16*)dLogits_EH);
        edge_softmax_backward_kernel<__nv_bfloat16, true><<<g->N, SM_BLOCK, 0, st>>>(g->rowptr, g->N, (const __nv_bfloat16*)alpha_EH, (const __nv_bfloat16*)dAlpha_EH, H, (__nv_bfloat16*)dLogits_EH);
    }
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

}  // extern "C"
