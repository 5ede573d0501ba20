// Declarations shared by the kernels that reduce gathered rows over fixed edge chunks.
#pragma once
#include "common.cuh"

namespace gnn {

constexpr int PF_SLAB = 256;   // positions staged in shared memory at a time
constexpr int PF_WARPS = 8;    // warps per block

enum { MODE_SUM = 0, MODE_MAX = 1, MODE_MIN = 2, MODE_ROUTE = 3, MODE_HEADSUM = 4, MODE_EFSUM = 5 };

// MODE_HEADSUM extras: multipliers per (position, head) and an optional rank-1 row epilogue
//   out[r,f] += epi_l[r,h(f)] * epi_a[f] + epi_r[r,h(f)] * epi_b[f]
struct HeadExtra {
    const float* wh;  // [E,H]
    const int32_t* wh_index;  // nullptr: position p uses row p of wh; else row wh_index[p] (only where chunked_is_flat())
    int H;
    const float *epi_l, *epi_r;  // [rows,H] or nullptr
    const float *epi_a, *epi_b;  // [F]
};

// per-feature multipliers (MODE_EFSUM) and the optional row epilogue of run_chunked:
//   v = agg_c * v + self_c * c(r) * self_X[r,f] + bias[f], then max(v, 0) if relu
// c(r) = 1, the length of row r in self_rowptr, or [that length > 0] (gnn_self_mode)
struct RowExtra {
    const float* ef;  // MODE_EFSUM: [E, ef_ld] fp32, or nullptr
    int ef_ld;
    float agg_c;      // multiplier of the reduced value: 1 or -1
    const void* self_X;  // [rows, F] of the call's dtype, or nullptr
    float self_c;
    int self_mode;
    const int64_t* self_rowptr;
    const float* bias;  // [F] or nullptr
    int relu;
};

// lanes per row (4..32) and 16-byte vectors per lane (1, 2, 4) for rows of nvec 16-byte chunks
bool pick_shape(int nvec, int* lpr, int* vpl);

size_t chunked_workspace(int64_t E, int F, bool with_arg);

// does run_chunked use the position-first (flat) kernel for this problem?  (It honours HeadExtra::wh_index.)
bool chunked_is_flat(int64_t E, int F, gnn_dtype dtype);

// out[r,:] = reduce over positions p of row r of  w[p] * X[col[p],:]   (see propagate.cu)
gnn_status run_chunked(const char* who, int mode, int32_t N, int64_t E, const int64_t* rowptr,
                       const int32_t* col, const float* w, const void* X, void* out,
                       int32_t* argmax, const int64_t* gscale_rowptr, const int32_t* route_arg,
                       const int32_t* route_pos, int mean, int F, gnn_dtype dtype, void* ws,
                       size_t ws_bytes, cudaStream_t st, const HeadExtra* hx = nullptr, const RowExtra* rx = nullptr);

// dW[p,h] = <X[col[p],h,:], D[i,h,:]> for p in row i (H = 1, lph = 0: one dot product per edge, times 1/row length if mean)
gnn_status run_sddmm(const char* who, const gnn_csr* g, const void* X, const void* D, int H, int C, int mean,
                     gnn_dtype dtype, float* dW, cudaStream_t st);

}  // namespace gnn
