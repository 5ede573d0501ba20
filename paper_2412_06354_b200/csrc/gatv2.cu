// GATv2-style attention logits (Sec. 3 "Message Passing": apply_edges with the target and the source features;
// the attention layers of Sec. 3 "Graph Convolutional Layers"), forward and backward, without the E x F tensor:
//   s[p,h] = sum_c a[h,c] * LeakyReLU(Xl[col[p],h,c] + Xr[i,h,c])          for p in row i
// The nonlinearity sits between the sum of the two transformed endpoints and the attention vector, so the
// logit is not a sum of a source term and a target term as in gnn_gat_fused: both rows meet at every edge.
//
// Forward: every position is independent.  A warp takes 256 consecutive positions, keeps the target row's chunk
// in registers while the row lasts, gathers four source rows at a time and reduces over the lanes of a head.
// Backward: dXr[i] sums over the positions of row i, dXl[j] over the transposed row of j, each term
// ds * a * LeakyReLU'(z) needing both rows again.  A warp walks a row (four gathers in flight), rows over 256
// positions get a block whose warps take contiguous shares that are added in warp order; da is the column sum
// of per-row partials.  Every order is fixed: results are bit-reproducible.  Gathered rows stay in registers as
// loaded and are unpacked where they are used (bf16: 14-16 registers fewer, one more block per SM).
#include "common.cuh"

namespace gnn {

constexpr int V2_U = 4;           // gathers in flight per warp
constexpr int V2_CHUNK = 256;     // positions per warp in the forward kernel
constexpr int V2_LONG = 256;      // rows above this many positions get a block in the backward kernels
constexpr int V2_BLOCK = 512;     // threads of that block
constexpr int V2_SUM_BLOCKS = 592;

struct V2Params {
    const int64_t* rowptr;
    const int32_t* col;
    const int32_t* pos_index;  // factor row per position (transposed form: t2f), or nullptr: the position itself
    const void* Xself;         // rows of this sparse form
    const void* Xother;        // gathered rows
    const float* a;            // [F]
    const float* ds;           // [E,H]
    float* s_out;              // forward: [E,H]
    void* dX;                  // backward: [N,F]
    float* da_part;            // backward: [N,F] per-row partial of da, or nullptr
    int32_t N;
    int64_t E;
    int nvec, H, lph;          // 16-byte chunks per row (<= 32), heads, chunks per head
    float slope;
};

template <typename T>
__device__ __forceinline__ void v2_load(const void* base, int64_t row, int nvec, int li, bool on, float* x) {
    constexpr int EPC = Chunk<T>::N;
    if (on) {
        Chunk<T>::unpack(__ldg(reinterpret_cast<const uint4*>(base) + (size_t)row * nvec + li), x);
    } else {
#pragma unroll
        for (int j = 0; j < EPC; ++j) x[j] = 0.f;
    }
}

// the same chunk as it lies in memory: unpacked where it is used, so that a gather in flight holds four registers
__device__ __forceinline__ uint4 v2_load_raw(const void* base, int64_t row, int nvec, int li, bool on) {
    return on ? __ldg(reinterpret_cast<const uint4*>(base) + (size_t)row * nvec + li) : make_uint4(0u, 0u, 0u, 0u);
}

// ------------------------------------------------------------------ forward
template <typename T>
__global__ void __launch_bounds__(256) gatv2_logits_kernel(const V2Params P) {
    constexpr int EPC = Chunk<T>::N;
    const int lane = threadIdx.x & 31;
    const int64_t c = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int64_t cs = c * V2_CHUNK;
    if (cs >= P.E) return;
    const int64_t ce = cs + V2_CHUNK < P.E ? cs + V2_CHUNK : P.E;
    const bool on = lane < P.nvec;
    const int span = P.H > 1 ? P.lph : 32;  // lanes that share one result
    float av[EPC];
#pragma unroll
    for (int j = 0; j < EPC; ++j) av[j] = on ? P.a[lane * EPC + j] : 0.f;
    int r = lower_bound_i64(P.rowptr, P.N + 1, cs + 1) - 1;  // row holding position cs
    int64_t rend = P.rowptr[r + 1];
    float xs[EPC];
    v2_load<T>(P.Xself, r, P.nvec, lane, on, xs);
    for (int64_t p0 = cs; p0 < ce; p0 += V2_U) {
        uint4 raw[V2_U];
#pragma unroll
        for (int u = 0; u < V2_U; ++u)
            if (p0 + u < ce) raw[u] = v2_load_raw(P.Xother, P.col[p0 + u], P.nvec, lane, on);
#pragma unroll
        for (int u = 0; u < V2_U; ++u) {
            const int64_t p = p0 + u;
            if (p >= ce) break;
            if (p >= rend) {  // the row changed (rows without edges are passed over)
                do { ++r; rend = P.rowptr[r + 1]; } while (p >= rend);
                v2_load<T>(P.Xself, r, P.nvec, lane, on, xs);
            }
            float xo[EPC];
            Chunk<T>::unpack(raw[u], xo);
            float t = 0.f;
#pragma unroll
            for (int j = 0; j < EPC; ++j) {
                const float z = xo[j] + xs[j];
                t = fmaf(av[j], z > 0.f ? z : P.slope * z, t);
            }
            for (int o = span >> 1; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if (on && (lane % span) == 0) P.s_out[p * P.H + (P.H > 1 ? lane / P.lph : 0)] = t;
        }
    }
}

// ------------------------------------------------------------------ backward
// positions [pa, pb) of row `row` -> acc (gradient of the row's own matrix) and acc_a (this row's share of da)
template <typename T, bool DA>
__device__ __forceinline__ void v2_row_share(const V2Params& P, int row, int64_t pa, int64_t pb, int lane, bool on, const float* xs,
                                             const float* av, float* acc, float* acc_a) {
    constexpr int EPC = Chunk<T>::N;
    const int head = P.H > 1 ? lane / P.lph : 0;
    for (int64_t p0 = pa; p0 < pb; p0 += V2_U) {
        uint4 raw[V2_U];
        float dsv[V2_U];
#pragma unroll
        for (int u = 0; u < V2_U; ++u)
            if (p0 + u < pb) {
                raw[u] = v2_load_raw(P.Xother, P.col[p0 + u], P.nvec, lane, on);
                const int64_t q = P.pos_index ? (int64_t)P.pos_index[p0 + u] : p0 + u;
                dsv[u] = on ? __ldg(P.ds + q * P.H + head) : 0.f;
            }
#pragma unroll
        for (int u = 0; u < V2_U; ++u) {
            if (p0 + u >= pb) break;
            float xo[EPC];
            Chunk<T>::unpack(raw[u], xo);
#pragma unroll
            for (int j = 0; j < EPC; ++j) {
                const float z = xo[j] + xs[j];
                acc[j] = fmaf(dsv[u] * av[j], z > 0.f ? 1.0f : P.slope, acc[j]);
                if (DA) acc_a[j] = fmaf(dsv[u], z > 0.f ? z : P.slope * z, acc_a[j]);
            }
        }
    }
}

template <typename T>
__device__ __forceinline__ void v2_store(const V2Params& P, int row, int lane, bool on, const float* acc, const float* acc_a, bool da) {
    constexpr int EPC = Chunk<T>::N;
    if (!on) return;
    reinterpret_cast<uint4*>(P.dX)[(size_t)row * P.nvec + lane] = Chunk<T>::pack(acc);
    if (da) {
        float4* o = reinterpret_cast<float4*>(P.da_part + ((size_t)row * P.nvec + lane) * EPC);
#pragma unroll
        for (int j = 0; j < EPC; j += 4) o[j / 4] = make_float4(acc_a[j], acc_a[j + 1], acc_a[j + 2], acc_a[j + 3]);
    }
}

// rows of at most V2_LONG positions: a warp per row
template <typename T, bool DA>
__global__ void __launch_bounds__(256) gatv2_backward_rows_kernel(const V2Params P) {
    constexpr int EPC = Chunk<T>::N;
    const int lane = threadIdx.x & 31;
    const bool on = lane < P.nvec;
    float av[EPC];
#pragma unroll
    for (int j = 0; j < EPC; ++j) av[j] = on ? P.a[lane * EPC + j] : 0.f;
    const int64_t warps = (int64_t)gridDim.x * 8;
    for (int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); row < P.N; row += warps) {
        const int64_t a = P.rowptr[row], b = P.rowptr[row + 1];
        if (b - a > V2_LONG) continue;
        float xs[EPC], acc[EPC], acc_a[EPC];
        v2_load<T>(P.Xself, row, P.nvec, lane, on, xs);
#pragma unroll
        for (int j = 0; j < EPC; ++j) { acc[j] = 0.f; acc_a[j] = 0.f; }
        v2_row_share<T, DA>(P, (int)row, a, b, lane, on, xs, av, acc, acc_a);
        v2_store<T>(P, (int)row, lane, on, acc, acc_a, DA);
    }
}

// longer rows: a block per row, its warps take contiguous shares, added in warp order.  Block k owns the rows
// k, k + blocks, ... (hub rows of a power-law graph sit at neighbouring indices, the stride spreads them); its
// threads look at V2_BLOCK of them at once and list the long ones in shared memory, then the block works through
// the list.  The order of the list varies from run to run; no row's arithmetic depends on it.
template <typename T, bool DA>
__global__ void __launch_bounds__(V2_BLOCK, 2) gatv2_backward_long_kernel(const V2Params P) {
    constexpr int EPC = Chunk<T>::N, NW = V2_BLOCK / 32;
    __shared__ float part[2][NW][32 * EPC];
    __shared__ int list[V2_BLOCK];
    __shared__ int count;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const bool on = lane < P.nvec;
    float av[EPC];
#pragma unroll
    for (int j = 0; j < EPC; ++j) av[j] = on ? P.a[lane * EPC + j] : 0.f;
    for (int64_t k0 = 0; (int64_t)blockIdx.x + k0 * gridDim.x < P.N; k0 += V2_BLOCK) {
        __syncthreads();  // every thread is done with the previous list
        if (threadIdx.x == 0) count = 0;
        __syncthreads();
        const int64_t mine = (int64_t)blockIdx.x + (k0 + threadIdx.x) * gridDim.x;
        if (mine < P.N && P.rowptr[mine + 1] - P.rowptr[mine] > V2_LONG) list[atomicAdd(&count, 1)] = (int)mine;
        __syncthreads();
        const int n = count;
        for (int i = 0; i < n; ++i) {
            const int row = list[i];
            const int64_t a = P.rowptr[row], b = P.rowptr[row + 1];
            const int64_t per = (b - a + NW - 1) / NW;
            const int64_t pa = a + w * per, pb = pa + per < b ? pa + per : b;
            float xs[EPC], acc[EPC], acc_a[EPC];
            v2_load<T>(P.Xself, row, P.nvec, lane, on, xs);
#pragma unroll
            for (int j = 0; j < EPC; ++j) { acc[j] = 0.f; acc_a[j] = 0.f; }
            if (pa < pb) v2_row_share<T, DA>(P, row, pa, pb, lane, on, xs, av, acc, acc_a);
#pragma unroll
            for (int j = 0; j < EPC; ++j) { part[0][w][lane * EPC + j] = acc[j]; part[1][w][lane * EPC + j] = acc_a[j]; }
            __syncthreads();
            if (w == 0) {
#pragma unroll
                for (int j = 0; j < EPC; ++j) {
                    float s0 = part[0][0][lane * EPC + j], s1 = part[1][0][lane * EPC + j];
                    for (int q = 1; q < NW; ++q) { s0 += part[0][q][lane * EPC + j]; s1 += part[1][q][lane * EPC + j]; }
                    acc[j] = s0; acc_a[j] = s1;
                }
                v2_store<T>(P, row, lane, on, acc, acc_a, DA);
            }
            __syncthreads();
        }
    }
}

// da[f] = sum over rows of part[row, f]: per-block sums over a contiguous range of rows, then over the blocks
__global__ void __launch_bounds__(256) v2_colsum_partial_kernel(const float* __restrict__ part, int32_t N, int F, int rows_per_block,
                                                                float* __restrict__ bsum) {
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_block, r1 = r0 + rows_per_block < N ? r0 + rows_per_block : N;
    for (int f = threadIdx.x; f < F; f += blockDim.x) {
        float s = 0.f;
        for (int64_t r = r0; r < r1; ++r) s += part[(size_t)r * F + f];
        bsum[(size_t)blockIdx.x * F + f] = s;
    }
}
__global__ void v2_colsum_final_kernel(const float* __restrict__ bsum, int nb, int F, float* __restrict__ out) {
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= F) return;
    float s = 0.f;
    for (int b = 0; b < nb; ++b) s += bsum[(size_t)b * F + f];
    out[f] = s;
}

static gnn_status v2_check(const char* who, const gnn_csr* g, int H, int C, gnn_dtype dtype, int* nvec, int* lph) {
    GNN_REQUIRE(g && g->rowptr, GNN_ERR_INVALID_ARG, "%s: null graph", who);
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "%s: bad dtype", who);
    GNN_REQUIRE(H >= 1 && C >= 1, GNN_ERR_INVALID_ARG, "%s: bad H or C", who);
    const int s = elem_size(dtype);
    GNN_REQUIRE(((size_t)C * s) % 16 == 0, GNN_ERR_UNSUPPORTED, "%s: a head must be a multiple of 16 bytes wide", who);
    *lph = C * s / 16;
    *nvec = H * *lph;
    GNN_REQUIRE(*nvec <= 32, GNN_ERR_UNSUPPORTED, "%s: rows wider than 512 bytes are not supported (H*C=%d)", who, H * C);
    GNN_REQUIRE(H == 1 || (*lph & (*lph - 1)) == 0, GNN_ERR_UNSUPPORTED,
                "%s: with several heads a head must span a power-of-two number of 16-byte chunks (C=%d)", who, C);
    GNN_REQUIRE(g->E < ((int64_t)1 << 31), GNN_ERR_UNSUPPORTED, "%s: E must be below 2^31", who);
    return GNN_OK;
}

}  // namespace gnn

using namespace gnn;

extern "C" {

gnn_status gnn_gatv2_logits(const gnn_csr* g, const void* Xl, const void* Xr, const float* a, int H, int C,
                            gnn_dtype dtype, float slope, float* s_csr, gnn_stream stream) {
    const char* who = "gnn_gatv2_logits";
    int nvec, lph;
    gnn_status rc = v2_check(who, g, H, C, dtype, &nvec, &lph);
    if (rc != GNN_OK) return rc;
    if (g->E == 0) return GNN_OK;
    GNN_REQUIRE(Xl && Xr && a && s_csr && g->col, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(aligned16(Xl) && aligned16(Xr), GNN_ERR_INVALID_ARG, "%s: feature matrices must be 16-byte aligned", who);
    V2Params P = {};
    P.rowptr = g->rowptr; P.col = g->col; P.Xself = Xr; P.Xother = Xl; P.a = a; P.s_out = s_csr;
    P.N = g->N; P.E = g->E; P.nvec = nvec; P.H = H; P.lph = lph; P.slope = slope;
    const int grid = (int)ceil_div(ceil_div(g->E, V2_CHUNK), 8);
    if (dtype == GNN_F32) gatv2_logits_kernel<float><<<grid, 256, 0, as_stream(stream)>>>(P);
    else gatv2_logits_kernel<__nv_bfloat16><<<grid, 256, 0, as_stream(stream)>>>(P);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

size_t gnn_gatv2_logits_backward_workspace(int32_t N, int H, int C) {
    if (N < 0 || H <= 0 || C <= 0) return 0;
    return up256((size_t)(N > 0 ? N : 1) * H * C * 4) + up256((size_t)V2_SUM_BLOCKS * H * C * 4);
}

gnn_status gnn_gatv2_logits_backward(const gnn_csr* g, const void* Xl, const void* Xr, const float* a,
                                     const float* ds_csr, int H, int C, gnn_dtype dtype, float slope,
                                     void* dXl, void* dXr, float* da, void* ws, size_t ws_bytes,
                                     gnn_stream stream) {
    const char* who = "gnn_gatv2_logits_backward";
    int nvec, lph;
    gnn_status rc = v2_check(who, g, H, C, dtype, &nvec, &lph);
    if (rc != GNN_OK) return rc;
    GNN_REQUIRE(g->rowptrT && Xl && Xr && a && (ds_csr || g->E == 0), GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(g->E == 0 || (g->col && g->colT && g->t2f), GNN_ERR_INVALID_ARG, "%s: incomplete gnn_csr", who);
    GNN_REQUIRE(aligned16(Xl) && aligned16(Xr) && aligned16(dXl) && aligned16(dXr), GNN_ERR_INVALID_ARG,
                "%s: feature matrices must be 16-byte aligned", who);
    const int F = H * C;
    const size_t need = gnn_gatv2_logits_backward_workspace(g->N, H, C);
    GNN_REQUIRE(!da || (ws && ws_bytes >= need && aligned16(ws)), GNN_ERR_WORKSPACE_TOO_SMALL,
                "%s: workspace of %zu bytes needed for da, %zu given", who, need, ws_bytes);
    if (g->N == 0) return GNN_OK;
    cudaStream_t st = as_stream(stream);
    V2Params P = {};
    P.a = a; P.ds = ds_csr; P.N = g->N; P.E = g->E; P.nvec = nvec; P.H = H; P.lph = lph; P.slope = slope;
    const int wgrid = (int)(ceil_div(g->N, 8) < 148 * 16 ? ceil_div(g->N, 8) : 148 * 16);
    const int lgrid = g->N < 148 * 2 ? g->N : 148 * 2;
    float* part = da ? (float*)ws : nullptr;
    float* bsum = da ? (float*)((char*)ws + up256((size_t)g->N * F * 4)) : nullptr;
#define GNN_V2_BWD(TYPE, DAFLAG)                                        \
    gatv2_backward_rows_kernel<TYPE, DAFLAG><<<wgrid, 256, 0, st>>>(P); \
    gatv2_backward_long_kernel<TYPE, DAFLAG><<<lgrid, V2_BLOCK, 0, st>>>(P);
    if (dXr || da) {  // rows = targets: self = Xr, gathered = Xl, factors at the positions themselves
        GNN_REQUIRE(dXr, GNN_ERR_INVALID_ARG, "%s: da is computed with dXr; pass dXr as well", who);
        P.rowptr = g->rowptr; P.col = g->col; P.pos_index = nullptr; P.Xself = Xr; P.Xother = Xl; P.dX = dXr; P.da_part = part;
        if (dtype == GNN_F32) { if (da) { GNN_V2_BWD(float, true) } else { GNN_V2_BWD(float, false) } }
        else { if (da) { GNN_V2_BWD(__nv_bfloat16, true) } else { GNN_V2_BWD(__nv_bfloat16, false) } }
        GNN_CHECK_LAUNCH(who);
    }
    if (dXl) {  // rows = sources: self = Xl, gathered = Xr, factors through t2f
        P.rowptr = g->rowptrT; P.col = g->colT; P.pos_index = g->t2f; P.Xself = Xl; P.Xother = Xr; P.dX = dXl; P.da_part = nullptr;
        if (dtype == GNN_F32) { GNN_V2_BWD(float, false) } else { GNN_V2_BWD(__nv_bfloat16, false) }
        GNN_CHECK_LAUNCH(who);
    }
#undef GNN_V2_BWD
    if (da) {
        const int rpb = (int)ceil_div(g->N, V2_SUM_BLOCKS), nb = (int)ceil_div(g->N, rpb);
        v2_colsum_partial_kernel<<<nb, 256, 0, st>>>(part, g->N, F, rpb, bsum);
        v2_colsum_final_kernel<<<(int)ceil_div(F, 128), 128, 0, st>>>(bsum, nb, F, da);
        GNN_CHECK_LAUNCH(who);
    }
    return GNN_OK;
}

}  // extern "C"
