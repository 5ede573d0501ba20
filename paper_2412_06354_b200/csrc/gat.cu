// GAT layer core (the attention layer named in Sec. 3 "Graph Convolutional Layers"), forward
// and backward, on an already transformed node tensor Wx [N,H,C]:
//   al[n,h] = <a_src[h,:], Wx[n,h,:]>     ar[n,h] = <a_dst[h,:], Wx[n,h,:]>
//   s[p,h]  = LeakyReLU(al[col[p],h] + ar[i,h])   for position p in row i
//   alpha   = edge softmax of s over each row
//   out[i,h,:] = sum_p alpha[p,h] * Wx[col[p],h,:]
// The E x F message tensor is never formed: the weighted sum runs in the chunked gather kernel
// with one multiplier per (edge, head).  Scores and coefficients are fp32.
#include "propagate.cuh"

namespace gnn {

// thread per (node, head): the two score dot products (any C)
template <typename T>
__global__ void gat_scores_kernel(const T* __restrict__ Wx, const float* __restrict__ a_src,
                                  const float* __restrict__ a_dst, int64_t NH, int H, int C,
                                  float* __restrict__ al, float* __restrict__ ar) {
    int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (t >= NH) return;
    const int h = (int)(t % H);
    const T* x = Wx + t * C;  // (n*H + h)*C
    float sl = 0.f, sr = 0.f;
    for (int c = 0; c < C; ++c) {
        float v = (float)x[c];
        sl = fmaf(a_src[h * C + c], v, sl);
        sr = fmaf(a_dst[h * C + c], v, sr);
    }
    al[t] = sl;
    ar[t] = sr;
}

// Rows of at most 32 16-byte chunks whose heads span a power-of-two number of chunks: LPR lanes
// cover a node's row with one coalesced 16-byte load each (32/LPR nodes per warp), keep their slice
// of both attention vectors in registers, and the lanes of a head add up by xor-shuffles (fixed tree).
template <typename T, int LPR>
__global__ void __launch_bounds__(256)
gat_scores_rows_kernel(const T* __restrict__ Wx, const float* __restrict__ a_src, const float* __restrict__ a_dst,
                       int N, int H, int nvec, int lph, float* __restrict__ al, float* __restrict__ ar) {
    constexpr int EPC = Chunk<T>::N, NG = 32 / LPR;
    const int lane = threadIdx.x & 31, g = lane / LPR, li = lane % LPR;
    const bool on = li < nvec;
    float as[EPC], ad[EPC];
#pragma unroll
    for (int j = 0; j < EPC; ++j) {
        as[j] = on ? a_src[li * EPC + j] : 0.f;
        ad[j] = on ? a_dst[li * EPC + j] : 0.f;
    }
    const int64_t warp = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * (int64_t)blockDim.x) >> 5;
    for (int64_t n0 = warp * NG; n0 < N; n0 += nwarps * NG) {
        const int64_t n = n0 + g;
        float sl = 0.f, sr = 0.f;
        if (n < N && on) {
            float x[EPC];
            Chunk<T>::unpack(*reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(Wx) + ((size_t)n * nvec + li) * 16), x);
#pragma unroll
            for (int j = 0; j < EPC; ++j) { sl = fmaf(as[j], x[j], sl); sr = fmaf(ad[j], x[j], sr); }
        }
        for (int o = lph >> 1; o > 0; o >>= 1) {
            sl += __shfl_xor_sync(0xffffffffu, sl, o);
            sr += __shfl_xor_sync(0xffffffffu, sr, o);
        }
        if (n < N && on && (li % lph) == 0) {
            al[(size_t)n * H + li / lph] = sl;
            ar[(size_t)n * H + li / lph] = sr;
        }
    }
}

// Row-local part of the backward pass, one warp per row (a whole block for long rows):
//   d[h]   = sum_p alpha[p,h]*dalpha[p,h]
//   ds     = alpha*(dalpha - d);  dz = ds * (z > 0 ? 1 : slope),  z = al[col[p],h] + ar[i,h]
//   dz is written over dalpha; dar[i,h] = sum_p dz[p,h]
constexpr int GB_LONG_ROW = 2048;
constexpr int GB_BLOCK = 256;

template <int NT>
__device__ __forceinline__ float sum_same_head(float v, int H, float* red) {
    const int lane = threadIdx.x & 31;
    for (int o = 16; o >= H; o >>= 1) {
        float other = __shfl_xor_sync(0xffffffffu, v, o);
        v = ((lane & o) == 0) ? (v + other) : (other + v);
    }
    if (NT > 32) {
        __syncthreads();
        if (lane < H) red[(threadIdx.x >> 5) * 32 + lane] = v;
        __syncthreads();
        float r = 0.f;
        for (int w = 0; w < NT / 32; ++w) r += red[w * 32 + (lane % H)];
        v = r;
    }
    return v;
}

template <bool LONG>
__global__ void __launch_bounds__(GB_BLOCK)
gat_backward_rows_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col, int N, int H,
                         const float* __restrict__ alpha, float* __restrict__ dalpha_dz,
                         const float* __restrict__ al, const float* __restrict__ ar, float slope,
                         float* __restrict__ dar) {
    __shared__ float red[GB_BLOCK];
    constexpr int NT = LONG ? GB_BLOCK : 32;
    const int tid = LONG ? threadIdx.x : (threadIdx.x & 31);
    const int h = tid % H;  // H is a power of two <= 32: fixed per thread
    int row = LONG ? blockIdx.x : (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
    const int stride = LONG ? gridDim.x : (int)((gridDim.x * (int64_t)blockDim.x) >> 5);
    for (; row < N; row += stride) {
        const int64_t a = rowptr[row], b = rowptr[row + 1];
        if (((b - a) > GB_LONG_ROW) != LONG) continue;  // uniform per warp / per block
        if (b == a) {
            if (tid < H) dar[(size_t)row * H + tid] = 0.f;
            continue;
        }
        const size_t lo = (size_t)a * H, hi = (size_t)b * H;
        float d = 0.f;
        for (size_t t = lo + tid; t < hi; t += NT) d = fmaf(alpha[t], dalpha_dz[t], d);
        d = sum_same_head<NT>(d, H, red);
        const float arv = ar[(size_t)row * H + h];
        float sdz = 0.f;
        for (size_t t = lo + tid; t < hi; t += NT) {
            const int64_t p = (int64_t)(t / H);
            const float z = al[(size_t)col[p] * H + h] + arv;
            const float dz = alpha[t] * (dalpha_dz[t] - d) * (z > 0.f ? 1.f : slope);
            dalpha_dz[t] = dz;
            sdz += dz;
        }
        sdz = sum_same_head<NT>(sdz, H, red);
        if (tid < H) dar[(size_t)row * H + tid] = sdz;
    }
}

// da_src[f] = sum_n dal[n,h(f)] * Wx[n,f], da_dst likewise with dar: fixed two-stage reduction
constexpr int GA_BLOCKS = 1184;  // 8 per SM: short serial chains over the rows
template <typename T>
__global__ void gat_da_partial_kernel(const T* __restrict__ Wx, const float* __restrict__ dal,
                                      const float* __restrict__ dar, int N, int H, int C,
                                      float* __restrict__ partial) {
    const int F = H * C;
    const int n0 = (int)((int64_t)N * blockIdx.x / gridDim.x), n1 = (int)((int64_t)N * (blockIdx.x + 1) / gridDim.x);
    for (int f = threadIdx.x; f < F; f += blockDim.x) {
        const int h = f / C;
        float s0 = 0.f, s1 = 0.f;
        for (int n = n0; n < n1; ++n) {
            const float x = (float)Wx[(size_t)n * F + f];
            s0 = fmaf(dal[(size_t)n * H + h], x, s0);
            s1 = fmaf(dar[(size_t)n * H + h], x, s1);
        }
        partial[((size_t)blockIdx.x * 2) * F + f] = s0;
        partial[((size_t)blockIdx.x * 2 + 1) * F + f] = s1;
    }
}
// 16 features x 16 groups of partials per block; each group is summed in ascending order with
// independent loads in flight, then the group sums are added in ascending group order
__global__ void __launch_bounds__(256)
gat_da_final_kernel(const float* __restrict__ partial, int nblocks, int F,
                    float* __restrict__ da_src, float* __restrict__ da_dst) {
    __shared__ float sh[2][16][16];
    const int e = threadIdx.x & 15, gq = threadIdx.x >> 4;
    const int f = blockIdx.x * 16 + e;
    const int per = (nblocks + 15) / 16, b0 = gq * per, b1 = min(nblocks, b0 + per);
    float s0 = 0.f, s1 = 0.f;
    if (f < F) {
#pragma unroll 8
        for (int b = b0; b < b1; ++b) {
            s0 += partial[((size_t)b * 2) * F + f];
            s1 += partial[((size_t)b * 2 + 1) * F + f];
        }
    }
    sh[0][gq][e] = s0;
    sh[1][gq][e] = s1;
    __syncthreads();
    if (gq == 0 && f < F) {
        float t0 = sh[0][0][e], t1 = sh[1][0][e];
#pragma unroll
        for (int q = 1; q < 16; ++q) { t0 += sh[0][q][e]; t1 += sh[1][q][e]; }
        da_src[f] = t0;
        da_dst[f] = t1;
    }
}

// dal[j,h] = sum over transposed positions q of row j of dz[t2f[q],h]  (any H; H % 4 == 0 goes through the chunked
// kernel instead).  LONG = false: a warp per row of at most DAL_LONG positions, lanes stride over the positions,
// fixed shuffle tree.  LONG = true: block k owns the rows k, k + blocks, ...; its threads look at DAL_BLOCK of them
// at once and list the longer ones in shared memory (the order of the list enters no sum), then the whole block
// takes a listed row: threads stride over its positions, shuffle tree, the warps' sums added in warp order.
constexpr int DAL_LONG = 1024, DAL_BLOCK = 256;
template <bool LONG>
__global__ void __launch_bounds__(DAL_BLOCK) gat_dal_rows_kernel(const int64_t* __restrict__ rowptrT, const int32_t* __restrict__ t2f,
                                                                 int N, int H, const float* __restrict__ dz, float* __restrict__ dal) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (!LONG) {
        const int stride = (int)gridDim.x * (DAL_BLOCK / 32);
        for (int row = (int)blockIdx.x * (DAL_BLOCK / 32) + w; row < N; row += stride) {
            const int64_t a = rowptrT[row], b = rowptrT[row + 1];
            if (b - a > DAL_LONG) continue;  // uniform per warp
            for (int h = 0; h < H; ++h) {
                float s = 0.f;
                for (int64_t q = a + lane; q < b; q += 32) s += dz[(size_t)t2f[q] * H + h];
                for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                if (lane == 0) dal[(size_t)row * H + h] = s;
            }
        }
    } else {
        __shared__ float red[DAL_BLOCK / 32];
        __shared__ int list[DAL_BLOCK];
        __shared__ int count;
        for (int64_t k0 = 0; (int64_t)blockIdx.x + k0 * gridDim.x < N; k0 += DAL_BLOCK) {
            __syncthreads();  // every thread is done with the previous list
            if (threadIdx.x == 0) count = 0;
            __syncthreads();
            const int64_t mine = (int64_t)blockIdx.x + (k0 + threadIdx.x) * gridDim.x;
            if (mine < N && rowptrT[mine + 1] - rowptrT[mine] > DAL_LONG) list[atomicAdd(&count, 1)] = (int)mine;
            __syncthreads();
            const int n = count;
            for (int i = 0; i < n; ++i) {
                const int row = list[i];
                const int64_t a = rowptrT[row], b = rowptrT[row + 1];
                for (int h = 0; h < H; ++h) {
                    float s = 0.f;
                    for (int64_t q = a + threadIdx.x; q < b; q += DAL_BLOCK) s += dz[(size_t)t2f[q] * H + h];
                    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                    if (lane == 0) red[w] = s;
                    __syncthreads();
                    if (threadIdx.x == 0) {
                        float t = red[0];
                        for (int k = 1; k < DAL_BLOCK / 32; ++k) t += red[k];
                        dal[(size_t)row * H + h] = t;
                    }
                    __syncthreads();
                }
            }
        }
    }
}

static bool pow2_le32(int H) { return H >= 1 && H <= 32 && (H & (H - 1)) == 0; }

struct GatWs {
    float *alphaT, *dz, *dal, *dar, *partial;
    void* chunk_ws;
    size_t chunk_bytes, bytes;
};
static GatWs gat_carve(void* ws, int32_t N, int64_t E, int H, int C, int backward) {
    GatWs w;
    char* p = (char*)ws;
    size_t off = 0;
    const size_t EH = (size_t)(E > 0 ? E : 1) * H * 4, NH = (size_t)(N > 0 ? N : 1) * H * 4;
    w.alphaT = w.dz = w.dal = w.dar = w.partial = nullptr;
    if (backward) {
        w.alphaT = (float*)(p + off); off += up256(EH);
        w.dz = (float*)(p + off); off += up256(EH);
        w.dal = (float*)(p + off); off += up256(NH);
        w.dar = (float*)(p + off); off += up256(NH);
        w.partial = (float*)(p + off); off += up256((size_t)GA_BLOCKS * 2 * H * C * 4);
    }
    w.chunk_ws = p + off;
    size_t a = chunked_workspace(E, H * C, false), b = chunked_workspace(E, H, false);
    w.chunk_bytes = a > b ? a : b;
    off += up256(w.chunk_bytes);
    w.bytes = off;
    return w;
}

static gnn_status gat_check(const char* who, const gnn_csr* g, int H, int C, gnn_dtype dtype) {
    GNN_REQUIRE(g && g->rowptr && g->rowptrT, GNN_ERR_INVALID_ARG, "%s: null graph", who);
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "%s: bad dtype", who);
    GNN_REQUIRE(pow2_le32(H), GNN_ERR_UNSUPPORTED, "%s: the number of heads must be a power of two <= 32 (H=%d)", who, H);
    const int epc = 16 / elem_size(dtype);
    GNN_REQUIRE(C >= epc && C % epc == 0, GNN_ERR_UNSUPPORTED,
                "%s: features per head must be a multiple of %d (C=%d)", who, epc, C);
    // the per-head dot products of the backward pass reduce over a power-of-two number of lanes: the forward
    // call refuses the same shapes, so that a layer never runs forward and then fails backward
    GNN_REQUIRE(pow2_le32(C / epc), GNN_ERR_UNSUPPORTED,
                "%s: a head must span a power-of-two number (<= 32) of 16-byte chunks (C=%d)", who, C);
    return GNN_OK;
}

gnn_status gat_alpha(const gnn_csr* g, const float* al, const float* ar, float slope, int H, float* alpha, cudaStream_t st);
bool gat_rows_backward_pl(const gnn_csr* g, const float* alpha, float* dalpha_dz, const float* al, const float* ar,
                          float slope, int H, float* dar, cudaStream_t st);
gnn_status sddmm_heads(const char* who, const gnn_csr* g, const void* X, const void* dOut, int H, int C,
                       gnn_dtype dtype, float* dW_EH, cudaStream_t st, int mean);
cudaStream_t side_fork(cudaStream_t st);
void side_join(cudaStream_t st, cudaStream_t side);

}  // namespace gnn

using namespace gnn;

extern "C" {

size_t gnn_gat_fused_workspace(int32_t N, int64_t E, int H, int C, int backward) {
    if (N < 0 || E < 0 || H < 1 || C < 1) return 0;
    return gat_carve(nullptr, N, E, H, C, backward).bytes;
}

gnn_status gnn_gat_fused(const gnn_csr* g, const void* Wx, const float* a_src, const float* a_dst,
                         int H, int C, gnn_dtype dtype, float slope, void* out, float* alpha_csr,
                         float* al, float* ar, void* ws, size_t ws_bytes, gnn_stream stream) {
    const char* who = "gnn_gat_fused";
    gnn_status rc = gat_check(who, g, H, C, dtype);
    if (rc != GNN_OK) return rc;
    GNN_REQUIRE(Wx && a_src && a_dst && out && al && ar && (g->E == 0 || alpha_csr), GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GatWs w = gat_carve(ws, g->N, g->E, H, C, 0);
    GNN_REQUIRE(ws && ws_bytes >= w.bytes, GNN_ERR_WORKSPACE_TOO_SMALL, "%s: workspace of %zu bytes needed", who, w.bytes);
    if (g->N == 0) return GNN_OK;
    cudaStream_t st = as_stream(stream);
    const int64_t NH = (int64_t)g->N * H;
    const int s_el = elem_size(dtype), nvec = H * C * s_el / 16, lph = C * s_el / 16;  // chunks per row / per head
    int lpr = 0, vpl = 0;
    if (((size_t)C * s_el) % 16 == 0 && (lph & (lph - 1)) == 0 && pick_shape(nvec, &lpr, &vpl) && vpl == 1) {
        const int grid = grid_for(ceil_div(g->N, 32 / lpr) * 32, 256);
#define GNN_GS(T, L) gat_scores_rows_kernel<T, L><<<grid, 256, 0, st>>>((const T*)Wx, a_src, a_dst, g->N, H, nvec, lph, al, ar)
        if (dtype == GNN_F32) { if (lpr == 4) GNN_GS(float, 4); else if (lpr == 8) GNN_GS(float, 8); else if (lpr == 16) GNN_GS(float, 16); else GNN_GS(float, 32); }
        else { if (lpr == 4) GNN_GS(__nv_bfloat16, 4); else if (lpr == 8) GNN_GS(__nv_bfloat16, 8); else if (lpr == 16) GNN_GS(__nv_bfloat16, 16); else GNN_GS(__nv_bfloat16, 32); }
#undef GNN_GS
    } else if (dtype == GNN_F32)
        gat_scores_kernel<float><<<(int)ceil_div(NH, 256), 256, 0, st>>>((const float*)Wx, a_src, a_dst, NH, H, C, al, ar);
    else
        gat_scores_kernel<__nv_bfloat16><<<(int)ceil_div(NH, 256), 256, 0, st>>>((const __nv_bfloat16*)Wx, a_src, a_dst, NH, H, C, al, ar);
    GNN_CHECK_LAUNCH(who);
    // logits and their per-row softmax, written straight into alpha_csr
    GNN_REQUIRE(g->E == 0 || g->col, GNN_ERR_INVALID_ARG, "%s: null col", who);
    rc = gat_alpha(g, al, ar, slope, H, alpha_csr, st);
    if (rc != GNN_OK) return rc;
    HeadExtra hx = {alpha_csr, nullptr, H, nullptr, nullptr, nullptr, nullptr};
    return run_chunked(who, MODE_HEADSUM, g->N, g->E, g->rowptr, g->col, nullptr, Wx, out, nullptr, nullptr,
                       nullptr, nullptr, 0, H * C, dtype, w.chunk_ws, w.chunk_bytes, st, &hx);
}

gnn_status gnn_gat_fused_backward(const gnn_csr* g, const void* Wx, const float* a_src,
                                  const float* a_dst, const float* alpha_csr, const float* al,
                                  const float* ar, const void* dOut, int H, int C, gnn_dtype dtype,
                                  float slope, void* dWx, float* da_src, float* da_dst, void* ws,
                                  size_t ws_bytes, gnn_stream stream) {
    const char* who = "gnn_gat_fused_backward";
    gnn_status rc = gat_check(who, g, H, C, dtype);
    if (rc != GNN_OK) return rc;
    GNN_REQUIRE(Wx && a_src && a_dst && al && ar && dOut && dWx && da_src && da_dst && (g->E == 0 || alpha_csr),
                GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(g->E == 0 || (g->col && g->colT && g->t2f), GNN_ERR_INVALID_ARG, "%s: incomplete gnn_csr", who);
    GatWs w = gat_carve(ws, g->N, g->E, H, C, 1);
    GNN_REQUIRE(ws && ws_bytes >= w.bytes && aligned16(ws), GNN_ERR_WORKSPACE_TOO_SMALL, "%s: workspace of %zu bytes needed", who, w.bytes);
    cudaStream_t st = as_stream(stream);
    const int F = H * C;
    if (g->N == 0) {
        if (cudaMemsetAsync(da_src, 0, (size_t)F * 4, st) != cudaSuccess || cudaMemsetAsync(da_dst, 0, (size_t)F * 4, st) != cudaSuccess)
            GNN_FAIL(GNN_ERR_CUDA, "%s: memset failed", who);
        return GNN_OK;
    }
    // dalpha[p,h] = <dOut[i,h,:], Wx[col[p],h,:]>  -> w.dz
    rc = sddmm_heads(who, g, Wx, dOut, H, C, dtype, w.dz, st, 0);
    if (rc != GNN_OK) return rc;
    // softmax and LeakyReLU derivatives, dz over dalpha, dar per row
    if (!gat_rows_backward_pl(g, alpha_csr, w.dz, al, ar, slope, H, w.dar, st)) {
        const int64_t wwant = ceil_div((int64_t)g->N * 32, GB_BLOCK), cap = (int64_t)148 * 64;
        cudaStream_t beside = side_fork(st);  // the two tiers write disjoint rows: side by side
        gat_backward_rows_kernel<true><<<(int)(g->N < cap ? g->N : cap), GB_BLOCK, 0, st>>>(
            g->rowptr, g->col, g->N, H, alpha_csr, w.dz, al, ar, slope, w.dar);
        gat_backward_rows_kernel<false><<<(int)(wwant < cap ? wwant : cap), GB_BLOCK, 0, beside>>>(
            g->rowptr, g->col, g->N, H, alpha_csr, w.dz, al, ar, slope, w.dar);
        side_join(st, beside);
    }
    GNN_CHECK_LAUNCH(who);
    // dal[j,h] = sum over the out-edges of j of dz
    if (H % 4 == 0) {
        rc = run_chunked(who, MODE_SUM, g->N, g->E, g->rowptrT, g->t2f, nullptr, w.dz, w.dal, nullptr, nullptr,
                         nullptr, nullptr, 0, H, GNN_F32, w.chunk_ws, w.chunk_bytes, st);
        if (rc != GNN_OK) return rc;
    } else {
        const int64_t wblocks = ceil_div((int64_t)g->N, DAL_BLOCK / 32);
        gat_dal_rows_kernel<false><<<(int)(wblocks < 148 * 8 ? wblocks : 148 * 8), DAL_BLOCK, 0, st>>>(g->rowptrT, g->t2f, g->N, H, w.dz, w.dal);
        gat_dal_rows_kernel<true><<<g->N < 148 * 4 ? g->N : 148 * 4, DAL_BLOCK, 0, st>>>(g->rowptrT, g->t2f, g->N, H, w.dz, w.dal);
        GNN_CHECK_LAUNCH(who);
    }
    // attention-vector gradients: two small reductions that need dal and dar only, on a side branch of the stream
    // beside the transposed gather below (joined before the call returns its place in the stream)
    cudaStream_t side = side_fork(st);
    if (dtype == GNN_F32)
        gat_da_partial_kernel<float><<<GA_BLOCKS, 256, 0, side>>>((const float*)Wx, w.dal, w.dar, g->N, H, C, w.partial);
    else
        gat_da_partial_kernel<__nv_bfloat16><<<GA_BLOCKS, 256, 0, side>>>((const __nv_bfloat16*)Wx, w.dal, w.dar, g->N, H, C, w.partial);
    gat_da_final_kernel<<<(int)ceil_div(F, 16), 256, 0, side>>>(w.partial, GA_BLOCKS, F, da_src, da_dst);
    if (cudaGetLastError() != cudaSuccess) {
        side_join(st, side);
        GNN_FAIL(GNN_ERR_CUDA, "%s: launch failed", who);
    }
    // dWx[j,h,:] = sum_q alpha[t2f[q],h]*dOut[colT[q],h,:] + dal[j,h]*a_src[h,:] + dar[j,h]*a_dst[h,:]
    // the flat kernel reads alpha through t2f; the row-walking one wants it permuted to transposed order first
    const bool indexed = chunked_is_flat(g->E, F, dtype);
    if (g->E > 0 && !indexed) {
        rc = gnn_permute_edge_data(g->t2f, g->E, H, 4, alpha_csr, w.alphaT, stream);
        if (rc != GNN_OK) {
            side_join(st, side);
            return rc;
        }
    }
    HeadExtra hx = {indexed ? alpha_csr : w.alphaT, indexed ? g->t2f : nullptr, H, w.dal, w.dar, a_src, a_dst};
    rc = run_chunked(who, MODE_HEADSUM, g->N, g->E, g->rowptrT, g->colT, nullptr, dOut, dWx, nullptr, nullptr,
                     nullptr, nullptr, 0, F, dtype, w.chunk_ws, w.chunk_bytes, st, &hx);
    side_join(st, side);  // the call's work is complete in the caller's stream only once the side branch is
    return rc;
}

}  // extern "C"
