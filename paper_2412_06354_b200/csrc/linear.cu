// Dense node-wise transform (the Dense layer / layer weight of the training example):
//   Y = X * W          X [N,K], W [K,M]
//   dX = dY * W^T      dY [N,M]
//   dW = X^T * dY      reduction over the N rows, split over row slabs and combined in slab order
//
// This file holds the entry points, their dispatch, and the fallback.  With K and M multiples of 16
// (16..256) the products run on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor
// memory): the pipelined kernels of linear_tma.cu (bf16: Y, dX, dW; fp32: Y, dX) or the
// single-buffered ones of linear_tc.cu (fp32 dW, fp32 weights too large for the pipeline, and bf16 when
// the tensor-map encoder is not available).  Everything else runs the shared-memory tiled FFMA kernel
// below with fp32 accumulation.  All sums have a fixed order.
#include "common.cuh"

namespace gnn {

// ------------------------------------------------------------------ FFMA path
// C[m,n] = sum_k A(m,k) * B(k,n) with arbitrary element strides, so transposed operands are
// stride swaps.  64x64 output tile per block, 16x16 threads, 4x4 outputs per thread, k in steps
// of 16.  k range [k0, k1) per blockIdx.z slab; slab results go to C + z*slab_stride.
constexpr int SG_TILE = 64, SG_K = 16;

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename TA, typename TB, typename TC>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const TA* __restrict__ A, int64_t sam, int64_t sak, const TB* __restrict__ B, int64_t sbk,
                 int64_t sbn, TC* __restrict__ C, int64_t Mr, int64_t Nc, int64_t Kd, int64_t k_per_slab,
                 int64_t slab_stride, const float* __restrict__ bias, int relu) {
    __shared__ float As[SG_K][SG_TILE + 1];
    __shared__ float Bs[SG_K][SG_TILE + 1];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int64_t m0 = (int64_t)blockIdx.y * SG_TILE, n0 = (int64_t)blockIdx.x * SG_TILE;
    const int64_t k0 = (int64_t)blockIdx.z * k_per_slab;
    const int64_t k1 = (k0 + k_per_slab < Kd) ? k0 + k_per_slab : Kd;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int64_t kb = k0; kb < k1; kb += SG_K) {
        for (int e = threadIdx.x; e < SG_K * SG_TILE; e += 256) {
            // A tile: consecutive threads walk the faster-varying of (m, k) in memory
            int kk, mm;
            if (sak <= sam) { kk = e % SG_K; mm = e / SG_K; } else { mm = e % SG_TILE; kk = e / SG_TILE; }
            const int64_t m = m0 + mm, k = kb + kk;
            As[kk][mm] = (m < Mr && k < k1) ? to_f32(A[m * sam + k * sak]) : 0.f;
            int kk2, nn;
            if (sbn <= sbk) { nn = e % SG_TILE; kk2 = e / SG_TILE; } else { kk2 = e % SG_K; nn = e / SG_K; }
            const int64_t n = n0 + nn, k2 = kb + kk2;
            Bs[kk2][nn] = (n < Nc && k2 < k1) ? to_f32(B[k2 * sbk + n * sbn]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < SG_K; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
    TC* Cz = C + (size_t)blockIdx.z * slab_stride;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty * 4 + i;
        if (m >= Mr) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t n = n0 + tx * 4 + j;
            if (n < Nc) {
                float y = acc[i][j];
                if (bias) y += bias[n];  // the element-wise tail of a layer, before the single rounding
                if (relu) y = fmaxf(y, 0.f);
                Cz[m * Nc + n] = from_f32<TC>(y);
            }
        }
    }
}

// out[i] = sum over slabs of part[s][i] in a fixed order: the slabs are cut into four contiguous
// groups, each summed in ascending order by one thread, and the four group sums are added in
// ascending group order.  64 elements x 4 groups per block.
template <typename TC>
__global__ void __launch_bounds__(256)
slab_sum_kernel(const float* __restrict__ part, int slabs, int64_t n, TC* __restrict__ out, int cols, int ld, int c0) {
    __shared__ float gsum[4][64];
    const int e = threadIdx.x & 63, g = threadIdx.x >> 6;
    const int64_t i = blockIdx.x * (int64_t)64 + e;
    const int per = (slabs + 3) / 4, z0 = g * per, z1 = min(slabs, z0 + per);
    float s = 0.f;
    if (i < n) {
        int z = z0;
        for (; z + 4 <= z1; z += 4) {
            const float a = part[(size_t)z * n + i], b = part[(size_t)(z + 1) * n + i], c = part[(size_t)(z + 2) * n + i],
                        d = part[(size_t)(z + 3) * n + i];
            s += a; s += b; s += c; s += d;
        }
        for (; z < z1; ++z) s += part[(size_t)z * n + i];
    }
    gsum[g][e] = s;
    __syncthreads();
    // the partials are [rows, cols]; the result may be a block of columns (c0 ..) of a matrix with rows ld apart
    if (g == 0 && i < n) out[(i / cols) * ld + c0 + (i % cols)] = from_f32<TC>(((gsum[0][e] + gsum[1][e]) + gsum[2][e]) + gsum[3][e]);
}

template <typename TA, typename TB, typename TC>
static void launch_simt(const TA* A, int64_t sam, int64_t sak, const TB* B, int64_t sbk, int64_t sbn, TC* C,
                        int64_t Mr, int64_t Nc, int64_t Kd, int64_t k_per_slab, int slabs, int64_t slab_stride,
                        cudaStream_t st, const float* bias = nullptr, int relu = 0) {
    dim3 grid((unsigned)ceil_div(Nc, SG_TILE), (unsigned)ceil_div(Mr, SG_TILE), (unsigned)slabs);
    gemm_simt_kernel<TA, TB, TC><<<grid, 256, 0, st>>>(A, sam, sak, B, sbk, sbn, C, Mr, Nc, Kd, k_per_slab, slab_stride, bias, relu);
}

// FFMA dW: rows of X / dY per partial.  128 rows while that gives at most 148 partials (small inputs
// still spread over many blocks), otherwise 4096.
static int dw_slab_rows(int64_t N) { return N <= 148 * 128 ? 128 : 4096; }
static int dw_slabs(int64_t N) { return (int)(N > 0 ? ceil_div(N, dw_slab_rows(N)) : 1); }

bool linear_tc_supported(int64_t N, int K, int M, gnn_dtype dtype);
gnn_status linear_tc_forward(const void* X, const void* W, int64_t N, int K, int M, int w_transposed, gnn_dtype dtype,
                             void* Y, int* d_flag, cudaStream_t st);
bool linear_tma_supported(int64_t N, int Kc, int Mo, int b_transposed, gnn_dtype dtype);
gnn_status linear_tma_forward(const void* X, const void* W, int64_t N, int Kc, int Mo, int b_transposed, void* Y, int* d_flag,
                              cudaStream_t st, const float* bias = nullptr, int relu = 0);
bool linear_tma_f32_supported(int64_t N, int Kc, int Mo, gnn_dtype dtype);
gnn_status linear_tma_f32_forward(const void* X, const void* W, int64_t N, int Kc, int Mo, int b_transposed, void* Y, int* d_flag,
                                  cudaStream_t st, const float* bias = nullptr, int relu = 0);
bool linear_tma_dw_supported(int64_t N, int K, int M, gnn_dtype dtype);
bool linear_tma_f32_dw_supported(int64_t N, int K, int M, gnn_dtype dtype);
int linear_tma_f32_dw_partials(int64_t N);
gnn_status linear_tma_f32_dw(const void* X, const void* dY, int64_t N, int K, int M, int ldd, float* part, int* d_flag, cudaStream_t st);
int linear_tma_dw_partials(int64_t N);
gnn_status linear_tma_dw(const void* X, const void* dY, int64_t N, int K, int M, int ldd, float* part, int* d_flag, cudaStream_t st);
bool linear_tc_dw_supported(int64_t N, int K, int M, gnn_dtype dtype);
int linear_tc_dw_partials(int64_t N);
gnn_status linear_tc_dw(const void* X, const void* dY, int64_t N, int K, int M, gnn_dtype dtype, float* part, int* d_flag,
                        cudaStream_t st);

}  // namespace gnn

using namespace gnn;

extern "C" {

size_t gnn_linear_workspace(int32_t N, int K, int M) {
    if (N < 0 || K <= 0 || M <= 0) return 0;
    const size_t parts = (size_t)(dw_slabs(N) > 148 ? dw_slabs(N) : 148);  // FFMA slabs or tensor-core CTA partials
    return 256 + up256(parts * K * M * 4);
}

gnn_status gnn_linear(const void* X, const void* W, int32_t N, int K, int M, gnn_dtype dtype, void* Y,
                      void* ws, size_t ws_bytes, gnn_stream stream) {
    return gnn_linear_bias_act(X, W, N, K, M, dtype, nullptr, 0, Y, ws, ws_bytes, stream);
}

gnn_status gnn_linear_bias_act(const void* X, const void* W, int32_t N, int K, int M, gnn_dtype dtype,
                               const float* bias, int relu, void* Y, void* ws, size_t ws_bytes,
                               gnn_stream stream) {
    const char* who = "gnn_linear";
    GNN_REQUIRE(N >= 0 && K > 0 && M > 0, GNN_ERR_INVALID_ARG, "%s: bad shape", who);
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "%s: bad dtype", who);
    if (N == 0) return GNN_OK;
    GNN_REQUIRE(X && W && Y, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(ws && ws_bytes >= 256, GNN_ERR_WORKSPACE_TOO_SMALL, "%s: workspace of %zu bytes needed", who, gnn_linear_workspace(N, K, M));
    cudaStream_t st = as_stream(stream);
    if (cudaMemsetAsync(ws, 0, sizeof(int), st) != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "%s: memset failed (is ws a device pointer?)", who);
    if (linear_tma_supported(N, K, M, 0, dtype)) return linear_tma_forward(X, W, N, K, M, 0, Y, (int*)ws, st, bias, relu);
    if (linear_tma_f32_supported(N, K, M, dtype)) return linear_tma_f32_forward(X, W, N, K, M, 0, Y, (int*)ws, st, bias, relu);
    // fp32 with weights too large for the pipelined kernel runs the single-buffered tensor-core kernel; with a
    // bias or relu it takes the FFMA kernel instead, whose epilogue applies them before the single rounding
    if (!bias && !relu && linear_tc_supported(N, K, M, dtype)) return linear_tc_forward(X, W, N, K, M, 0, dtype, Y, (int*)ws, st);
    if (dtype == GNN_F32) {
        launch_simt<float, float, float>((const float*)X, K, 1, (const float*)W, M, 1, (float*)Y, N, M, K, K, 1, 0, st, bias, relu);
    } else {
        launch_simt<__nv_bfloat16, __nv_bfloat16, __nv_bfloat16>((const __nv_bfloat16*)X, K, 1, (const __nv_bfloat16*)W, M, 1,
                                                               (__nv_bfloat16*)Y, N, M, K, K, 1, 0, st, bias, relu);
    }
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

gnn_status gnn_linear_backward(const void* X, const void* W, const void* dY, int32_t N, int K, int M,
                               gnn_dtype dtype, void* dX, void* dW, void* ws, size_t ws_bytes,
                               gnn_stream stream) {
    const char* who = "gnn_linear_backward";
    GNN_REQUIRE(N >= 0 && K > 0 && M > 0, GNN_ERR_INVALID_ARG, "%s: bad shape", who);
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "%s: bad dtype", who);
    GNN_REQUIRE(dY || N == 0, GNN_ERR_INVALID_ARG, "%s: null dY", who);
    const size_t need = gnn_linear_workspace(N, K, M);
    GNN_REQUIRE(ws && ws_bytes >= need, GNN_ERR_WORKSPACE_TOO_SMALL, "%s: workspace of %zu bytes needed", who, need);
    cudaStream_t st = as_stream(stream);
    if (cudaMemsetAsync(ws, 0, sizeof(int), st) != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "%s: memset failed (is ws a device pointer?)", who);
    if (dX && N > 0) {
        GNN_REQUIRE(W, GNN_ERR_INVALID_ARG, "%s: dX needs W", who);
        // dX[n,k] = sum_m dY[n,m] * W[k,m]
        if (linear_tma_supported(N, M, K, 1, dtype)) {
            gnn_status rc = linear_tma_forward(dY, W, N, M, K, 1, dX, (int*)ws, st);
            if (rc != GNN_OK) return rc;
        } else if (linear_tma_f32_supported(N, M, K, dtype)) {
            gnn_status rc = linear_tma_f32_forward(dY, W, N, M, K, 1, dX, (int*)ws, st);
            if (rc != GNN_OK) return rc;
        } else if (linear_tc_supported(N, M, K, dtype)) {
            gnn_status rc = linear_tc_forward(dY, W, N, M, K, 1, dtype, dX, (int*)ws, st);
            if (rc != GNN_OK) return rc;
        } else if (dtype == GNN_F32) {
            launch_simt<float, float, float>((const float*)dY, M, 1, (const float*)W, 1, M, (float*)dX, N, K, M, M, 1, 0, st);
        } else {
            launch_simt<__nv_bfloat16, __nv_bfloat16, __nv_bfloat16>((const __nv_bfloat16*)dY, M, 1, (const __nv_bfloat16*)W, 1, M,
                                                                   (__nv_bfloat16*)dX, N, K, M, M, 1, 0, st);
        }
        GNN_CHECK_LAUNCH(who);
    }
    if (dW) {
        GNN_REQUIRE(X || N == 0, GNN_ERR_INVALID_ARG, "%s: dW needs X", who);
        // dW[k,m] = sum_n X[n,k] * dY[n,m]: one fp32 partial per slab of rows, then summed in slab order
        float* part = (float*)((char*)ws + 256);
        int slabs = dw_slabs(N);
        const int64_t km = (int64_t)K * M;
        // more output columns than one pipelined launch takes (256, or fewer where K fills tensor memory): one launch
        // and one ordered sum per block of columns of dY, each through the same partial buffer
        int block = 0;
        if (N > 0 && M > 32) {
            const int step = dtype == GNN_F32 ? 32 : 16;
            for (int mc = (M < 256 ? M : 256) / step * step; mc >= step && !block; mc -= step)
                if (dtype == GNN_F32 ? linear_tma_f32_dw_supported(N, K, mc, dtype) : linear_tma_dw_supported(N, K, mc, dtype)) block = mc;
        }
        const bool whole = dtype == GNN_F32 ? linear_tma_f32_dw_supported(N, K, M, dtype) : linear_tma_dw_supported(N, K, M, dtype);
        if (!whole && block > 0 && M % (dtype == GNN_F32 ? 32 : 16) == 0) {
            const int s_el = dtype == GNN_F32 ? 4 : 2;
            for (int c0 = 0; c0 < M; c0 += block) {
                const int mc = M - c0 < block ? M - c0 : block;
                const void* dYb = (const char*)dY + (size_t)c0 * s_el;
                gnn_status rc;
                if (dtype == GNN_F32) {
                    slabs = linear_tma_f32_dw_partials(N);
                    rc = linear_tma_f32_dw(X, dYb, N, K, mc, M, part, (int*)ws, st);
                } else {
                    slabs = linear_tma_dw_partials(N);
                    rc = linear_tma_dw(X, dYb, N, K, mc, M, part, (int*)ws, st);
                }
                if (rc != GNN_OK) return rc;
                const int64_t kmc = (int64_t)K * mc;
                if (dtype == GNN_F32) slab_sum_kernel<float><<<(int)ceil_div(kmc, 64), 256, 0, st>>>(part, slabs, kmc, (float*)dW, mc, M, c0);
                else slab_sum_kernel<__nv_bfloat16><<<(int)ceil_div(kmc, 64), 256, 0, st>>>(part, slabs, kmc, (__nv_bfloat16*)dW, mc, M, c0);
                GNN_CHECK_LAUNCH(who);
            }
            return GNN_OK;
        }
        if (linear_tma_f32_dw_supported(N, K, M, dtype)) {
            slabs = linear_tma_f32_dw_partials(N);
            gnn_status rc = linear_tma_f32_dw(X, dY, N, K, M, M, part, (int*)ws, st);
            if (rc != GNN_OK) return rc;
        } else if (linear_tma_dw_supported(N, K, M, dtype)) {
            slabs = linear_tma_dw_partials(N);
            gnn_status rc = linear_tma_dw(X, dY, N, K, M, M, part, (int*)ws, st);
            if (rc != GNN_OK) return rc;
        } else if (linear_tc_dw_supported(N, K, M, dtype)) {
            slabs = linear_tc_dw_partials(N);
            gnn_status rc = linear_tc_dw(X, dY, N, K, M, dtype, part, (int*)ws, st);
            if (rc != GNN_OK) return rc;
        } else if (N == 0) {
            if (cudaMemsetAsync(part, 0, (size_t)km * 4, st) != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "%s: memset failed", who);
        } else if (dtype == GNN_F32) {
            launch_simt<float, float, float>((const float*)X, 1, K, (const float*)dY, M, 1, part, K, M, N, dw_slab_rows(N), slabs, km, st);
        } else {
            launch_simt<__nv_bfloat16, __nv_bfloat16, float>((const __nv_bfloat16*)X, 1, K, (const __nv_bfloat16*)dY, M, 1, part, K, M, N,
                                                           dw_slab_rows(N), slabs, km, st);
        }
        if (dtype == GNN_F32) slab_sum_kernel<float><<<(int)ceil_div(km, 64), 256, 0, st>>>(part, slabs, km, (float*)dW, M, M, 0);
        else slab_sum_kernel<__nv_bfloat16><<<(int)ceil_div(km, 64), 256, 0, st>>>(part, slabs, km, (__nv_bfloat16*)dW, M, M, 0);
        GNN_CHECK_LAUNCH(who);
    }
    return GNN_OK;
}

}  // extern "C"
