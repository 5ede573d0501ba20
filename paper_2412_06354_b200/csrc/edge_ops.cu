// Unfused message-passing primitives (Sec. 3 "Message Passing"): gather, apply_edges,
// aggregate_neighbors and their backward passes, on explicit E x F message tensors.  These are
// the building blocks custom layers are written with; the fused propagate avoids their E x F
// traffic.  Edge tensors are in CSR order unless stated.
#include "propagate.cuh"

namespace gnn {

// row of the sparse form that contains position p: last r with rowptr[r] <= p
__device__ __forceinline__ int row_of_position(const int64_t* rowptr, int N, int64_t p) {
    return lower_bound_i64(rowptr, N + 1, p + 1) - 1;
}

// Row of position p for a thread whose positions only grow: a block owns a contiguous span of (position, chunk) pairs,
// so from one step to the next a thread's position moves on by blockDim / chunks-per-position and its row by a step or
// two.  A full search per 16-byte chunk made the calls below run at a sixth of the memory rate; now there is one full
// search per thread, and another only where more than eight rows (a run of empty ones) are skipped at once.
__device__ __forceinline__ int advance_row(const int64_t* __restrict__ rowptr, int N, int row, int64_t p) {
    if (row < 0) return row_of_position(rowptr, N, p);
#pragma unroll 1
    for (int k = 0; k < 8; ++k) {
        if (rowptr[row + 1] > p) return row;  // rowptr[row] <= p holds throughout
        ++row;
    }
    return rowptr[row + 1] > p ? row : row_of_position(rowptr, N, p);
}
// first pair of this block's span and one past its last; spans are multiples of the block size
__device__ __forceinline__ void block_span(int64_t total, int64_t* t0, int64_t* t1) {
    const int64_t per = ((total + gridDim.x - 1) / gridDim.x + blockDim.x - 1) / blockDim.x * blockDim.x;
    *t0 = (int64_t)blockIdx.x * per;
    *t1 = *t0 + per < total ? *t0 + per : total;
}

// Grid-stride walk over (position, 16-byte chunk) pairs t = p*nvec + ci without a division per step:
// one 64-bit division when the thread starts, then p and ci advance by the quotient and remainder of
// the stride.
struct PosChunk {
    int64_t p, dp;
    int ci, dci, nvec;
    __device__ __forceinline__ PosChunk(int64_t t0, int64_t stride, int nv) : p(t0 / nv), dp(stride / nv), ci((int)(t0 % nv)), dci((int)(stride % nv)), nvec(nv) {}
    __device__ __forceinline__ void next() {
        p += dp;
        ci += dci;
        if (ci >= nvec) { ci -= nvec; ++p; }
    }
};

// out[k, chunk] = X[idx[k], chunk]; one thread per 16-byte chunk
__global__ void gather_rows_kernel(const int32_t* __restrict__ idx, int64_t E, const uint4* __restrict__ X,
                                   int nvec, uint4* __restrict__ out) {
    int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x, total = E * nvec;
    for (PosChunk q(t, stride, nvec); t < total; t += stride, q.next()) out[t] = X[(size_t)idx[q.p] * nvec + q.ci];
}

// m[p, f] = e[p, g(f)] * X[col[p], f]   (e == nullptr: plain copy of the source row)
template <typename T>
__global__ void apply_edges_mul_kernel(const int32_t* __restrict__ col, int64_t E, const uint4* __restrict__ X,
                                       int nvec, const float* __restrict__ e, int ew, int feats_per_e,
                                       uint4* __restrict__ m) {
    constexpr int EPC = Chunk<T>::N;
    int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x, total = E * nvec;
    const bool chunk_in_one = feats_per_e % EPC == 0;  // every 16-byte chunk lies under one multiplier
    for (PosChunk q(t, stride, nvec); t < total; t += stride, q.next()) {
        const int64_t p = q.p;
        const int ci = q.ci;
        float x[EPC];
        Chunk<T>::unpack(X[(size_t)col[p] * nvec + ci], x);
        if (e) {
            if (chunk_in_one) {
                const float f = e[p * ew + (ci * EPC) / feats_per_e];
#pragma unroll
                for (int j = 0; j < EPC; ++j) x[j] *= f;
            } else {
#pragma unroll
                for (int j = 0; j < EPC; ++j) x[j] *= e[p * ew + (ci * EPC + j) / feats_per_e];
            }
        }
        m[t] = Chunk<T>::pack(x);
    }
}

// s[p, h] = LeakyReLU_slope(al[col[p], h] + ar[row(p), h]), fp32
__global__ void gat_logit_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col, int N,
                                 int64_t E, int H, const float* __restrict__ al, const float* __restrict__ ar,
                                 float slope, float* __restrict__ s) {
    int64_t t0, t1;
    block_span(E * H, &t0, &t1);
    int i = -1;
    for (int64_t t = t0 + threadIdx.x; t < t1; t += blockDim.x) {
        const int64_t p = t / H;
        const int h = (int)(t - p * H);
        i = advance_row(rowptr, N, i, p);
        const float z = al[(size_t)col[p] * H + h] + ar[(size_t)i * H + h];
        s[t] = z > 0.f ? z : slope * z;
    }
}

// backward of aggregate w.r.t. the messages: dm[p, :] from dOut[row(p), :]
template <typename T>
__global__ void aggregate_backward_kernel(const int64_t* __restrict__ rowptr, int N, int64_t E, int op,
                                          const uint4* __restrict__ dOut, const int32_t* __restrict__ argmax,
                                          int nvec, uint4* __restrict__ dm) {
    constexpr int EPC = Chunk<T>::N;
    int64_t t0, t1;
    block_span(E * nvec, &t0, &t1);
    int i = -1;
    for (int64_t t = t0 + threadIdx.x; t < t1; t += blockDim.x) {
        const int64_t p = t / nvec;
        const int ci = (int)(t - p * nvec);
        i = advance_row(rowptr, N, i, p);
        uint4 raw = dOut[(size_t)i * nvec + ci];
        if (op == GNN_SUM) { dm[t] = raw; continue; }
        float x[EPC];
        Chunk<T>::unpack(raw, x);
        if (op == GNN_MEAN) {
            const float d = (float)(rowptr[i + 1] - rowptr[i]);
#pragma unroll
            for (int j = 0; j < EPC; ++j) x[j] = x[j] / d;
        } else {
            const int32_t* a = argmax + ((size_t)i * nvec + ci) * EPC;
#pragma unroll
            for (int j = 0; j < EPC; ++j) x[j] = (a[j] == (int32_t)p) ? x[j] : 0.f;
        }
        dm[t] = Chunk<T>::pack(x);
    }
}

static gnn_status check_rows(const char* who, int F, gnn_dtype dtype, int* nvec) {
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "%s: bad dtype", who);
    const int s = elem_size(dtype);
    GNN_REQUIRE(F > 0 && ((size_t)F * s) % 16 == 0, GNN_ERR_UNSUPPORTED,
                "%s: F*sizeof(element) = %d must be a multiple of 16 bytes", who, F * s);
    *nvec = F * s / 16;
    return GNN_OK;
}

// graph_ptr[g] = first node whose graph id is >= g; flag set if ids are unsorted or out of range
__global__ void graph_ptr_kernel(const int32_t* __restrict__ gid, int32_t N, int32_t G,
                                 int64_t* __restrict__ gptr, int* __restrict__ flag) {
    int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t n = t; n < N; n += stride) {
        const int a = gid[n];
        if (a < 0 || a >= G || (n + 1 < N && gid[n + 1] < a)) *flag = 1;
    }
    for (int64_t g = t; g <= G; g += stride) {
        int lo = 0, hi = N;
        while (lo < hi) {
            int mid = (lo + hi) >> 1;
            if (gid[mid] < (int32_t)g) lo = mid + 1; else hi = mid;
        }
        gptr[g] = lo;
    }
}

// out = alpha*a + beta*b, element-wise in fp32 (self terms of layers: W1*x_i + W2*agg, (1+eps)*x_i + sum)
template <typename T>
__global__ void axpby_kernel(float alpha, const uint4* __restrict__ a, float beta, const uint4* __restrict__ b,
                             int64_t nvec, uint4* __restrict__ out) {
    constexpr int EPC = Chunk<T>::N;
    int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; t < nvec; t += stride) {
        float x[EPC], y[EPC];
        Chunk<T>::unpack(a[t], x);
        Chunk<T>::unpack(b[t], y);
#pragma unroll
        for (int j = 0; j < EPC; ++j) x[j] = fmaf(alpha, x[j], beta * y[j]);
        out[t] = Chunk<T>::pack(x);
    }
}

}  // namespace gnn

using namespace gnn;

extern "C" {

gnn_status gnn_gather(const int32_t* idx, int64_t E, const void* X, int32_t N, int F,
                      gnn_dtype dtype, void* out, gnn_stream stream) {
    const char* who = "gnn_gather";
    int nvec;
    gnn_status rc = check_rows(who, F, dtype, &nvec);
    if (rc != GNN_OK) return rc;
    GNN_REQUIRE(E >= 0 && N >= 0, GNN_ERR_INVALID_ARG, "%s: negative size", who);
    if (E == 0) return GNN_OK;
    GNN_REQUIRE(idx && X && out && aligned16(X) && aligned16(out), GNN_ERR_INVALID_ARG,
                "%s: null or misaligned argument", who);
    gather_rows_kernel<<<grid_for(E * nvec, 256), 256, 0, as_stream(stream)>>>(idx, E, (const uint4*)X, nvec, (uint4*)out);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

gnn_status gnn_gather_backward(const gnn_csr* g, int by_src, const void* dOut_EF, int F,
                               gnn_dtype dtype, void* dX, void* ws, size_t ws_bytes,
                               gnn_stream stream) {
    const char* who = "gnn_gather_backward";
    GNN_REQUIRE(g && dOut_EF && dX, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    const int64_t* rp = by_src ? g->rowptrT : g->rowptr;
    const int32_t* rows = by_src ? g->eidT : g->eid;  // COO row of dOut for each position
    GNN_REQUIRE(rp && (g->E == 0 || rows), GNN_ERR_INVALID_ARG, "%s: incomplete gnn_csr", who);
    return run_chunked(who, MODE_SUM, g->N, g->E, rp, rows, nullptr, dOut_EF, dX, nullptr, nullptr,
                       nullptr, nullptr, 0, F, dtype, ws, ws_bytes, as_stream(stream));
}

gnn_status gnn_apply_edges(const gnn_csr* g, gnn_msg msg, const void* X_or_al, const void* ar,
                           const float* e, int e_width, int F, gnn_dtype dtype, float slope,
                           void* m_out, gnn_stream stream) {
    const char* who = "gnn_apply_edges";
    GNN_REQUIRE(g && g->rowptr && X_or_al && m_out, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    if (g->E == 0) return GNN_OK;
    GNN_REQUIRE(g->col, GNN_ERR_INVALID_ARG, "%s: null col", who);
    cudaStream_t st = as_stream(stream);
    if (msg == GNN_MSG_GAT_LOGIT) {
        GNN_REQUIRE(dtype == GNN_F32, GNN_ERR_UNSUPPORTED, "%s: GAT_LOGIT works on fp32 scores", who);
        GNN_REQUIRE(ar && F > 0, GNN_ERR_INVALID_ARG, "%s: GAT_LOGIT needs ar and F = heads", who);
        gat_logit_kernel<<<grid_for(g->E * F, 256), 256, 0, st>>>(g->rowptr, g->col, g->N, g->E, F, (const float*)X_or_al,
                                                                  (const float*)ar, slope, (float*)m_out);
        GNN_CHECK_LAUNCH(who);
        return GNN_OK;
    }
    GNN_REQUIRE(msg == GNN_MSG_COPY_XJ || msg == GNN_MSG_E_MUL_XJ, GNN_ERR_INVALID_ARG, "%s: bad message", who);
    int nvec;
    gnn_status rc = check_rows(who, F, dtype, &nvec);
    if (rc != GNN_OK) return rc;
    GNN_REQUIRE(aligned16(X_or_al) && aligned16(m_out), GNN_ERR_INVALID_ARG, "%s: misaligned matrix", who);
    const int epc = dtype == GNN_F32 ? 4 : 8;
    int feats_per_e = 1;
    if (msg == GNN_MSG_E_MUL_XJ) {
        GNN_REQUIRE(e && e_width >= 1 && F % e_width == 0, GNN_ERR_INVALID_ARG,
                    "%s: E_MUL_XJ needs e of width 1, H (dividing F) or F", who);
        feats_per_e = F / e_width;
        (void)epc;
    } else {
        e = nullptr;
        e_width = 1;
    }
    const int grid = grid_for(g->E * nvec, 256);
    if (dtype == GNN_F32)
        apply_edges_mul_kernel<float><<<grid, 256, 0, st>>>(g->col, g->E, (const uint4*)X_or_al, nvec, e, e_width, feats_per_e, (uint4*)m_out);
    else
        apply_edges_mul_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(g->col, g->E, (const uint4*)X_or_al, nvec, e, e_width, feats_per_e, (uint4*)m_out);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

gnn_status gnn_aggregate(const gnn_csr* g, gnn_op op, const void* m_EF, int F, gnn_dtype dtype,
                         void* out, int32_t* argmax, void* ws, size_t ws_bytes, gnn_stream stream) {
    const char* who = "gnn_aggregate";
    GNN_REQUIRE(g && g->rowptr && m_EF && out, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(op >= GNN_SUM && op <= GNN_MIN, GNN_ERR_INVALID_ARG, "%s: bad op", who);
    GNN_REQUIRE(!argmax || aligned16(argmax), GNN_ERR_INVALID_ARG, "%s: argmax must be 16-byte aligned", who);
    const int mode = op == GNN_MAX ? MODE_MAX : op == GNN_MIN ? MODE_MIN : MODE_SUM;
    // position p reads row p of the message tensor: the segmented reduction without a gather
    return run_chunked(who, mode, g->N, g->E, g->rowptr, nullptr, nullptr, m_EF, out, argmax, nullptr,
                       nullptr, nullptr, op == GNN_MEAN, F, dtype, ws, ws_bytes, as_stream(stream));
}

gnn_status gnn_aggregate_backward(const gnn_csr* g, gnn_op op, const void* dOut_NF,
                                  const int32_t* argmax, int F, gnn_dtype dtype, void* dm_EF,
                                  gnn_stream stream) {
    const char* who = "gnn_aggregate_backward";
    GNN_REQUIRE(g && g->rowptr && dOut_NF && dm_EF, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(op >= GNN_SUM && op <= GNN_MIN, GNN_ERR_INVALID_ARG, "%s: bad op", who);
    GNN_REQUIRE((op != GNN_MAX && op != GNN_MIN) || argmax, GNN_ERR_INVALID_ARG, "%s: MAX/MIN need the forward argmax", who);
    int nvec;
    gnn_status rc = check_rows(who, F, dtype, &nvec);
    if (rc != GNN_OK) return rc;
    if (g->E == 0) return GNN_OK;
    GNN_REQUIRE(aligned16(dOut_NF) && aligned16(dm_EF), GNN_ERR_INVALID_ARG, "%s: misaligned matrix", who);
    const int grid = grid_for(g->E * nvec, 256);
    cudaStream_t st = as_stream(stream);
    if (dtype == GNN_F32)
        aggregate_backward_kernel<float><<<grid, 256, 0, st>>>(g->rowptr, g->N, g->E, (int)op, (const uint4*)dOut_NF, argmax, nvec, (uint4*)dm_EF);
    else
        aggregate_backward_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(g->rowptr, g->N, g->E, (int)op, (const uint4*)dOut_NF, argmax, nvec, (uint4*)dm_EF);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

gnn_status gnn_graph_ptr_from_ids(const int32_t* graph_id, int32_t N, int32_t G, int64_t* graph_ptr,
                                  void* ws, size_t ws_bytes, gnn_stream stream) {
    const char* who = "gnn_graph_ptr_from_ids";
    GNN_REQUIRE(N >= 0 && G >= 0 && graph_ptr && (N == 0 || graph_id), GNN_ERR_INVALID_ARG, "%s: bad argument", who);
    GNN_REQUIRE(ws && ws_bytes >= 4, GNN_ERR_WORKSPACE_TOO_SMALL, "%s: 4 bytes of workspace needed", who);
    cudaStream_t st = as_stream(stream);
    int* flag = (int*)ws;
    if (cudaMemsetAsync(flag, 0, 4, st) != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "%s: memset failed", who);
    graph_ptr_kernel<<<grid_for((N > G ? N : G) + 1, 256), 256, 0, st>>>(graph_id, N, G, graph_ptr, flag);
    GNN_CHECK_LAUNCH(who);
    int h = 0;
    if (cudaMemcpyAsync(&h, flag, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
        GNN_FAIL(GNN_ERR_CUDA, "%s: reading the validation flag failed", who);
    GNN_REQUIRE(h == 0, GNN_ERR_NOT_SORTED, "%s: graph ids must be sorted and inside [0, %d)", who, G);
    return GNN_OK;
}

gnn_status gnn_reduce_nodes(const int64_t* graph_ptr, int32_t G, int32_t N, gnn_op op, const void* X,
                            int F, gnn_dtype dtype, void* out_GF, int32_t* argmax, void* ws,
                            size_t ws_bytes, gnn_stream stream) {
    const char* who = "gnn_reduce_nodes";
    GNN_REQUIRE(graph_ptr && X && out_GF && G >= 0 && N >= 0, GNN_ERR_INVALID_ARG, "%s: bad argument", who);
    GNN_REQUIRE(op >= GNN_SUM && op <= GNN_MIN, GNN_ERR_INVALID_ARG, "%s: bad op", who);
    GNN_REQUIRE(!argmax || aligned16(argmax), GNN_ERR_INVALID_ARG, "%s: argmax must be 16-byte aligned", who);
    const int mode = op == GNN_MAX ? MODE_MAX : op == GNN_MIN ? MODE_MIN : MODE_SUM;
    // graphs are the rows, nodes the positions: the same segmented reduction as aggregate
    return run_chunked(who, mode, G, N, graph_ptr, nullptr, nullptr, X, out_GF, argmax, nullptr, nullptr,
                       nullptr, op == GNN_MEAN, F, dtype, ws, ws_bytes, as_stream(stream));
}

gnn_status gnn_reduce_nodes_backward(const int64_t* graph_ptr, int32_t G, int32_t N, gnn_op op,
                                     const void* dOut_GF, const int32_t* argmax, int F,
                                     gnn_dtype dtype, void* dX_NF, gnn_stream stream) {
    const char* who = "gnn_reduce_nodes_backward";
    GNN_REQUIRE(graph_ptr && dOut_GF && dX_NF && G >= 0 && N >= 0, GNN_ERR_INVALID_ARG, "%s: bad argument", who);
    GNN_REQUIRE(op >= GNN_SUM && op <= GNN_MIN, GNN_ERR_INVALID_ARG, "%s: bad op", who);
    GNN_REQUIRE((op != GNN_MAX && op != GNN_MIN) || argmax, GNN_ERR_INVALID_ARG, "%s: MAX/MIN need the forward argmax", who);
    int nvec;
    gnn_status rc = check_rows(who, F, dtype, &nvec);
    if (rc != GNN_OK) return rc;
    if (N == 0) return GNN_OK;
    GNN_REQUIRE(aligned16(dOut_GF) && aligned16(dX_NF), GNN_ERR_INVALID_ARG, "%s: misaligned matrix", who);
    const int grid = grid_for((int64_t)N * nvec, 256);
    cudaStream_t st = as_stream(stream);
    if (dtype == GNN_F32)
        aggregate_backward_kernel<float><<<grid, 256, 0, st>>>(graph_ptr, G, N, (int)op, (const uint4*)dOut_GF, argmax, nvec, (uint4*)dX_NF);
    else
        aggregate_backward_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(graph_ptr, G, N, (int)op, (const uint4*)dOut_GF, argmax, nvec, (uint4*)dX_NF);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

gnn_status gnn_axpby(float alpha, const void* a, float beta, const void* b, int64_t n, gnn_dtype dtype,
                     void* out, gnn_stream stream) {
    const char* who = "gnn_axpby";
    GNN_REQUIRE(n >= 0 && (dtype == GNN_F32 || dtype == GNN_BF16), GNN_ERR_INVALID_ARG, "%s: bad argument", who);
    if (n == 0) return GNN_OK;
    const int epc = 16 / elem_size(dtype);
    GNN_REQUIRE(n % epc == 0, GNN_ERR_UNSUPPORTED, "%s: the element count must be a multiple of %d", who, epc);
    GNN_REQUIRE(a && b && out && aligned16(a) && aligned16(b) && aligned16(out), GNN_ERR_INVALID_ARG, "%s: null or misaligned argument", who);
    const int64_t nvec = n / epc;
    cudaStream_t st = as_stream(stream);
    if (dtype == GNN_F32) axpby_kernel<float><<<grid_for(nvec, 256), 256, 0, st>>>(alpha, (const uint4*)a, beta, (const uint4*)b, nvec, (uint4*)out);
    else axpby_kernel<__nv_bfloat16><<<grid_for(nvec, 256), 256, 0, st>>>(alpha, (const uint4*)a, beta, (const uint4*)b, nvec, (uint4*)out);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

}  // extern "C"
