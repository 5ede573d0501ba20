// Graph set-up: COO -> sparse forms (stable LSD radix sort), degrees, GCN normalisation,
// self-loops, edge-data permutation.  Integer results are unique and bit-exact.
#include <stdarg.h>

#include "common.cuh"

namespace gnn {

static thread_local char g_err[512] = "";
void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

// ------------------------------------------------------------------ validation
__global__ void validate_coo_kernel(int32_t N, int64_t E, const int32_t* __restrict__ src,
                                    const int32_t* __restrict__ dst, int* __restrict__ flag) {
    int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (; k < E; k += stride) {
        int s = src[k], d = dst[k];
        bad |= (s < 0) | (s >= N) | (d < 0) | (d >= N);
    }
    if (bad) *flag = 1;  // benign race: every writer stores the same value
}

// ------------------------------------------------------------------ validation of a caller-built sparse form
// Bits of the result word; every read stays in bounds whatever the arrays hold (an index is used only after its
// range check, row look-ups search rowptr[0..N] by position).
enum : int {
    CSR_BAD_ROWPTR = 1,     // rowptr / rowptrT: first entry 0, last entry E, non-decreasing
    CSR_BAD_NODE = 2,       // col / colT outside [0, N)
    CSR_BAD_EDGE = 4,       // eid / eidT / t2f outside [0, E)
    CSR_BAD_PERM = 8,       // eid, eidT or t2f holds a value twice
    CSR_BAD_ORDER = 16,     // edge ids not ascending inside a row (the order that makes the forms unique)
    CSR_BAD_CROSS = 32,     // the two forms disagree: position t2f[q] is not the same edge as transposed position q
};

__device__ __forceinline__ int csr_row_of(const int64_t* __restrict__ rowptr, int32_t N, int64_t p) {
    int lo = 0, hi = N;  // largest i in [0, N) with rowptr[i] <= p (rowptr[0] = 0 <= p when the pointers are sound)
    while (hi - lo > 1) {
        const int mid = lo + (hi - lo) / 2;
        if (rowptr[mid] <= p) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void csr_validate_pointers_kernel(int32_t N, int64_t E, const int64_t* __restrict__ rowptr,
                                             const int64_t* __restrict__ rowptrT, int* __restrict__ flag) {
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i > N) return;
    bool bad = false;
    const int64_t a = rowptr[i], b = rowptrT[i];
    bad |= a < 0 || a > E || b < 0 || b > E;
    if (i == 0) bad |= a != 0 || b != 0;
    if (i == N) bad |= a != E || b != E;
    if (i < N) bad |= rowptr[i + 1] < a || rowptrT[i + 1] < b;
    if (bad) atomicOr(flag, CSR_BAD_ROWPTR);
}

// runs only when the pointers passed: one thread per position of either form
__global__ void csr_validate_positions_kernel(int32_t N, int64_t E, const int64_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                                              const int32_t* __restrict__ eid, const int64_t* __restrict__ rowptrT,
                                              const int32_t* __restrict__ colT, const int32_t* __restrict__ eidT,
                                              const int32_t* __restrict__ t2f, unsigned* __restrict__ seen, int64_t words,
                                              int* __restrict__ flag) {
    const int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (p >= E) return;
    int bad = 0;
    const int32_t c = col[p], cT = colT[p], e = eid[p], eT = eidT[p], f = t2f[p];
    if (c < 0 || c >= N || cT < 0 || cT >= N) bad |= CSR_BAD_NODE;
    const bool e_ok = e >= 0 && e < E, eT_ok = eT >= 0 && eT < E, f_ok = f >= 0 && f < E;
    if (!e_ok || !eT_ok || !f_ok) bad |= CSR_BAD_EDGE;
    // each of the three arrays must hold every value once: a bit per value and array
    if (e_ok && (atomicOr(seen + (e >> 5), 1u << (e & 31)) >> (e & 31)) & 1u) bad |= CSR_BAD_PERM;
    if (eT_ok && (atomicOr(seen + words + (eT >> 5), 1u << (eT & 31)) >> (eT & 31)) & 1u) bad |= CSR_BAD_PERM;
    if (f_ok && (atomicOr(seen + 2 * words + (f >> 5), 1u << (f & 31)) >> (f & 31)) & 1u) bad |= CSR_BAD_PERM;
    // ascending edge ids inside a row, in both forms
    const int i = csr_row_of(rowptr, N, p), j = csr_row_of(rowptrT, N, p);
    if (p + 1 < rowptr[i + 1] && e_ok && eid[p + 1] <= e) bad |= CSR_BAD_ORDER;
    if (p + 1 < rowptrT[j + 1] && eT_ok && eidT[p + 1] <= eT) bad |= CSR_BAD_ORDER;
    // transposed position p (row j = the edge's source, colT = its target) and position t2f[p] are one edge
    if (f_ok && eT_ok) {
        if (eid[f] != eT || col[f] != j || csr_row_of(rowptr, N, f) != cT) bad |= CSR_BAD_CROSS;
    }
    if (bad) atomicOr(flag, bad);
}

// ------------------------------------------------------------------ exclusive scan (uint32)
// three launches: per-tile sums, scan of the tile sums by one block, per-tile scan + offset
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

// exclusive scan of one value per thread over a 256-thread block; *total = block sum
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* total) {
    __shared__ uint32_t warp_sums[SCAN_THREADS / 32];
    __shared__ uint32_t block_total;
    int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_sums[wid] = inc;
    __syncthreads();
    if (wid == 0) {
        uint32_t s = lane < SCAN_THREADS / 32 ? warp_sums[lane] : 0;
        uint32_t si = s;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t t = __shfl_up_sync(0xffffffffu, si, o);
            if (lane >= o) si += t;
        }
        if (lane < SCAN_THREADS / 32) warp_sums[lane] = si - s;
        if (lane == 31) block_total = si;
    }
    __syncthreads();
    uint32_t r = warp_sums[wid] + inc - v;
    *total = block_total;
    __syncthreads();
    return r;
}

__global__ void scan_tile_sums_kernel(const uint32_t* __restrict__ in, int64_t n,
                                      uint32_t* __restrict__ tile_sums) {
    int64_t base = (int64_t)blockIdx.x * SCAN_TILE + threadIdx.x * SCAN_ITEMS;
    uint32_t s = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i)
        if (base + i < n) s += in[base + i];
    uint32_t total;
    block_exclusive_scan(s, &total);
    if (threadIdx.x == 0) tile_sums[blockIdx.x] = total;
}

__global__ void scan_single_block_kernel(uint32_t* __restrict__ data, int64_t n) {
    uint32_t carry = 0;
    for (int64_t base = 0; base < n; base += SCAN_THREADS) {
        int64_t i = base + threadIdx.x;
        uint32_t v = i < n ? data[i] : 0, total;
        uint32_t ex = block_exclusive_scan(v, &total);
        if (i < n) data[i] = carry + ex;
        carry += total;
    }
}

__global__ void scan_apply_kernel(const uint32_t* __restrict__ in, int64_t n,
                                  const uint32_t* __restrict__ tile_offsets,
                                  uint32_t* __restrict__ out) {
    int64_t base = (int64_t)blockIdx.x * SCAN_TILE + threadIdx.x * SCAN_ITEMS;
    uint32_t v[SCAN_ITEMS], s = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        v[i] = base + i < n ? in[base + i] : 0;
        s += v[i];
    }
    uint32_t total;
    uint32_t ex = block_exclusive_scan(s, &total) + tile_offsets[blockIdx.x];
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        if (base + i < n) out[base + i] = ex;
        ex += v[i];
    }
}

// ------------------------------------------------------------------ stable LSD radix sort
constexpr int RS_THREADS = 256;
constexpr int RS_WARPS = RS_THREADS / 32;
constexpr int RS_ROUNDS = 16;
constexpr int RS_TILE = RS_THREADS * RS_ROUNDS;  // 4096 keys per block
constexpr int RS_BINS = 256;

// element order inside a tile: warp-major, then round, then lane
__device__ __forceinline__ int64_t rs_index(int64_t tile0, int warp, int round, int lane) {
    return tile0 + (int64_t)warp * (32 * RS_ROUNDS) + round * 32 + lane;
}

__global__ void __launch_bounds__(RS_THREADS)
radix_hist_kernel(const int32_t* __restrict__ keys, int64_t E, int shift, uint32_t nblocks,
                  uint32_t* __restrict__ table) {
    __shared__ uint32_t cnt[RS_BINS];
    cnt[threadIdx.x] = 0;
    __syncthreads();
    int64_t tile0 = (int64_t)blockIdx.x * RS_TILE;
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll 4
    for (int r = 0; r < RS_ROUNDS; ++r) {
        int64_t i = rs_index(tile0, warp, r, lane);
        if (i < E) atomicAdd(&cnt[(keys[i] >> shift) & 0xFF], 1u);
    }
    __syncthreads();
    table[(size_t)threadIdx.x * nblocks + blockIdx.x] = cnt[threadIdx.x];
}

// vals_in == nullptr means "value = index" (first pass)
__global__ void __launch_bounds__(RS_THREADS)
radix_scatter_kernel(const int32_t* __restrict__ keys_in, const int32_t* __restrict__ vals_in,
                     int64_t E, int shift, uint32_t nblocks, const uint32_t* __restrict__ base,
                     int32_t* __restrict__ keys_out, int32_t* __restrict__ vals_out) {
    __shared__ uint32_t wcnt[RS_WARPS][RS_BINS];
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int w = 0; w < RS_WARPS; ++w) wcnt[w][threadIdx.x] = 0;
    __syncthreads();
    int64_t tile0 = (int64_t)blockIdx.x * RS_TILE;
    const uint32_t lt = (1u << lane) - 1u;
    int32_t key[RS_ROUNDS];
    // (i) per-warp digit totals
#pragma unroll
    for (int r = 0; r < RS_ROUNDS; ++r) {
        int64_t i = rs_index(tile0, warp, r, lane);
        bool ok = i < E;
        key[r] = ok ? keys_in[i] : 0;
        int d = ok ? ((key[r] >> shift) & 0xFF) : RS_BINS;  // invalid lanes form their own group
        uint32_t peers = __match_any_sync(0xffffffffu, d);
        if (ok && (peers & lt) == 0) wcnt[warp][d] += __popc(peers);  // one leader per digit
        __syncwarp();
    }
    __syncthreads();
    // (ii) digit d: global base, then exclusive prefix over the warps of this block
    {
        int d = threadIdx.x;
        uint32_t run = base[(size_t)d * nblocks + blockIdx.x];
#pragma unroll
        for (int w = 0; w < RS_WARPS; ++w) {
            uint32_t t = wcnt[w][d];
            wcnt[w][d] = run;
            run += t;
        }
    }
    __syncthreads();
    // (iii) stable ranks and scatter
#pragma unroll
    for (int r = 0; r < RS_ROUNDS; ++r) {
        int64_t i = rs_index(tile0, warp, r, lane);
        bool ok = i < E;
        int d = ok ? ((key[r] >> shift) & 0xFF) : RS_BINS;
        uint32_t peers = __match_any_sync(0xffffffffu, d);
        if (ok) {
            uint32_t pos = wcnt[warp][d] + __popc(peers & lt);
            keys_out[pos] = key[r];
            vals_out[pos] = vals_in ? vals_in[i] : (int32_t)i;
        }
        __syncwarp();
        if (ok && (peers & lt) == 0) wcnt[warp][d] += __popc(peers);
        __syncwarp();
    }
}

__global__ void csr_finalize_kernel(int32_t N, int64_t E, const int32_t* __restrict__ sorted_keys,
                                    const int32_t* __restrict__ sorted_vals,
                                    const int32_t* __restrict__ other, int64_t* __restrict__ rowptr,
                                    int32_t* __restrict__ col, int32_t* __restrict__ eid) {
    int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t p = t; p < E; p += stride) {
        int32_t k = sorted_vals[p];
        eid[p] = k;
        col[p] = other[k];
    }
    // rowptr[i] = first position whose key is >= i
    for (int64_t i = t; i <= N; i += stride) {
        int64_t lo = 0, hi = E;
        while (lo < hi) {
            int64_t mid = (lo + hi) >> 1;
            if (sorted_keys[mid] < (int32_t)i) lo = mid + 1; else hi = mid;
        }
        rowptr[i] = lo;
    }
}

__global__ void invert_perm_kernel(int64_t E, const int32_t* __restrict__ eid,
                                   int32_t* __restrict__ pos) {
    int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; p < E; p += stride) pos[eid[p]] = (int32_t)p;
}
__global__ void compose_perm_kernel(int64_t E, const int32_t* __restrict__ pos,
                                    const int32_t* __restrict__ eidT, int32_t* __restrict__ t2f) {
    int64_t q = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; q < E; q += stride) t2f[q] = pos[eidT[q]];
}

struct SortWs {
    int32_t *kA, *vA, *kB, *vB;
    uint32_t *table, *tile_sums;
    int* flag;
    size_t bytes;
};

static SortWs carve(void* ws, int64_t E) {
    SortWs s;
    size_t nblocks = (size_t)ceil_div(E > 0 ? E : 1, RS_TILE);
    size_t table_n = nblocks * RS_BINS;
    size_t tiles = (size_t)ceil_div((int64_t)table_n, SCAN_TILE);
    size_t eb = up256((size_t)(E > 0 ? E : 1) * 4);
    char* p = (char*)ws;
    size_t off = 0;
    s.flag = (int*)(p + off); off += 256;
    s.kA = (int32_t*)(p + off); off += eb;
    s.vA = (int32_t*)(p + off); off += eb;
    s.kB = (int32_t*)(p + off); off += eb;
    s.vB = (int32_t*)(p + off); off += eb;
    s.table = (uint32_t*)(p + off); off += up256(table_n * 4);
    s.tile_sums = (uint32_t*)(p + off); off += up256(tiles * 4);
    s.bytes = off;
    return s;
}

// stable sort of (key[k], k) by key; result left in *sk, *sv (pointers into ws)
static gnn_status sort_by_key(int32_t N, int64_t E, const int32_t* keys, const SortWs& w,
                              cudaStream_t st, const int32_t** sk, const int32_t** sv) {
    int bits = 0;
    while (bits < 31 && ((int64_t)1 << bits) < (int64_t)N) ++bits;
    int passes = bits == 0 ? 1 : (bits + 7) / 8;
    uint32_t nblocks = (uint32_t)ceil_div(E > 0 ? E : 1, RS_TILE);
    int64_t table_n = (int64_t)nblocks * RS_BINS;
    int tiles = (int)ceil_div(table_n, SCAN_TILE);
    const int32_t* kin = keys;
    const int32_t* vin = nullptr;
    int32_t* kout = w.kA;
    int32_t* vout = w.vA;
    for (int p = 0; p < passes; ++p) {
        int shift = 8 * p;
        radix_hist_kernel<<<nblocks, RS_THREADS, 0, st>>>(kin, E, shift, nblocks, w.table);
        scan_tile_sums_kernel<<<tiles, SCAN_THREADS, 0, st>>>(w.table, table_n, w.tile_sums);
        scan_single_block_kernel<<<1, SCAN_THREADS, 0, st>>>(w.tile_sums, tiles);
        scan_apply_kernel<<<tiles, SCAN_THREADS, 0, st>>>(w.table, table_n, w.tile_sums, w.table);
        radix_scatter_kernel<<<nblocks, RS_THREADS, 0, st>>>(kin, vin, E, shift, nblocks, w.table,
                                                            kout, vout);
        GNN_CHECK_LAUNCH("radix sort pass");
        kin = kout;
        vin = vout;
        kout = (kout == w.kA) ? w.kB : w.kA;
        vout = (vout == w.vA) ? w.vB : w.vA;
    }
    *sk = kin;
    *sv = vin;
    return GNN_OK;
}

// ------------------------------------------------------------------ degrees / GCN coefficients
__global__ void degree_count_kernel(int32_t N, const int64_t* __restrict__ rowptr,
                                    int32_t* __restrict__ deg) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i < N) deg[i] = (int32_t)(rowptr[i + 1] - rowptr[i]);
}

// one warp per row; lane-strided partial sums combined by a fixed shuffle tree
__global__ void degree_weighted_kernel(int32_t N, const int64_t* __restrict__ rowptr,
                                       const float* __restrict__ w, float* __restrict__ deg) {
    int64_t row = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (row >= N) return;
    int64_t a = rowptr[row], b = rowptr[row + 1];
    float s = 0.f;
    for (int64_t p = a + lane; p < b; p += 32) s += w[p];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) deg[row] = s;
}

__global__ void degree_unit_kernel(int32_t N, const int64_t* __restrict__ rowptr,
                                   float* __restrict__ deg) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i < N) deg[i] = (float)(rowptr[i + 1] - rowptr[i]);
}

// coef[p] = w[p] / sqrt(deg[row(p)] * deg[col[p]]).  LONG = false: a warp per row of at most GC_LONG positions.
// LONG = true: block k owns the rows k, k + blocks, ...; its threads look at 256 of them at once, list the longer ones
// in shared memory, and the whole block takes a listed row (a single warp would walk a hub of 10^5 positions alone).
constexpr int GC_LONG = 1024;
__device__ __forceinline__ float gcn_coef(float wp, float di, float dj) {
    // IEEE sqrt and division (no approximate rsqrt): ~1e-7 relative
    return (di > 0.f && dj > 0.f) ? __fdiv_rn(wp, __fsqrt_rn(di * dj)) : 0.f;
}
template <bool LONG>
__global__ void __launch_bounds__(256) gcn_coef_kernel(int32_t N, const int64_t* __restrict__ rowptr,
                                                       const int32_t* __restrict__ col, const float* __restrict__ w,
                                                       const float* __restrict__ deg, float* __restrict__ coef) {
    if (!LONG) {
        int64_t row = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
        int lane = threadIdx.x & 31;
        if (row >= N) return;
        int64_t a = rowptr[row], b = rowptr[row + 1];
        if (b - a > GC_LONG) return;
        float di = deg[row];
        for (int64_t p = a + lane; p < b; p += 32) coef[p] = gcn_coef(w ? w[p] : 1.0f, di, deg[col[p]]);
    } else {
        __shared__ int list[256];
        __shared__ int count;
        for (int64_t k0 = 0; (int64_t)blockIdx.x + k0 * gridDim.x < N; k0 += 256) {
            __syncthreads();  // every thread is done with the previous list
            if (threadIdx.x == 0) count = 0;
            __syncthreads();
            const int64_t mine = (int64_t)blockIdx.x + (k0 + threadIdx.x) * gridDim.x;
            if (mine < N && rowptr[mine + 1] - rowptr[mine] > GC_LONG) list[atomicAdd(&count, 1)] = (int)mine;
            __syncthreads();
            const int n = count;
            for (int i = 0; i < n; ++i) {  // the order of the list does not matter: every position is written once
                const int row = list[i];
                const int64_t a = rowptr[row], b = rowptr[row + 1];
                const float di = deg[row];
                for (int64_t p = a + threadIdx.x; p < b; p += 256) coef[p] = gcn_coef(w ? w[p] : 1.0f, di, deg[col[p]]);
            }
        }
    }
}

__global__ void permute_f32_kernel(int64_t E, const int32_t* __restrict__ perm,
                                   const float* __restrict__ in, float* __restrict__ out) {
    int64_t p = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; p < E; p += stride) out[p] = in[perm[p]];
}

template <typename T>
__global__ void permute_rows_kernel(int64_t E, int width, const int32_t* __restrict__ perm,
                                    const T* __restrict__ in, T* __restrict__ out) {
    int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t total = E * width;
    for (; t < total; t += stride) {
        int64_t p = t / width;
        int c = (int)(t - p * width);
        out[t] = in[(int64_t)perm[p] * width + c];
    }
}

__global__ void add_self_loops_kernel(int32_t N, int64_t E, const int32_t* __restrict__ src,
                                      const int32_t* __restrict__ dst, int32_t* __restrict__ so,
                                      int32_t* __restrict__ dout) {
    int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; k < E + N; k += stride) {
        if (k < E) { so[k] = src[k]; dout[k] = dst[k]; }
        else { so[k] = (int32_t)(k - E); dout[k] = (int32_t)(k - E); }
    }
}

}  // namespace gnn

using namespace gnn;

extern "C" {

const char* gnn_status_string(gnn_status s) {
    switch (s) {
        case GNN_OK: return "ok";
        case GNN_ERR_INVALID_ARG: return "invalid argument";
        case GNN_ERR_INDEX_OUT_OF_RANGE: return "index out of range";
        case GNN_ERR_NOT_SORTED: return "not sorted";
        case GNN_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case GNN_ERR_UNSUPPORTED: return "unsupported";
        case GNN_ERR_CUDA: return "CUDA error";
        case GNN_ERR_TIMEOUT: return "timeout";
    }
    return "unknown status";
}
const char* gnn_last_error_string(void) { return g_err; }
int gnn_version(void) { return 100; }

size_t gnn_coo_to_csr_workspace(int32_t N, int64_t E) {
    (void)N;
    if (E < 0) return 0;
    return carve(nullptr, E).bytes;
}

gnn_status gnn_coo_to_csr(int32_t N, int64_t E, const int32_t* src, const int32_t* dst,
                          gnn_csr* out, void* ws, size_t ws_bytes, gnn_stream stream) {
    GNN_REQUIRE(N >= 0 && E >= 0, GNN_ERR_INVALID_ARG, "gnn_coo_to_csr: negative size");
    GNN_REQUIRE(E <= 0x7FFFFFFFLL - 1, GNN_ERR_UNSUPPORTED, "gnn_coo_to_csr: E must be < 2^31");
    GNN_REQUIRE(out && out->rowptr && out->rowptrT, GNN_ERR_INVALID_ARG, "gnn_coo_to_csr: null output");
    GNN_REQUIRE(E == 0 || (src && dst && out->col && out->eid && out->colT && out->eidT && out->t2f),
                GNN_ERR_INVALID_ARG, "gnn_coo_to_csr: null edge array");
    GNN_REQUIRE(ws && ws_bytes >= gnn_coo_to_csr_workspace(N, E), GNN_ERR_WORKSPACE_TOO_SMALL,
                "gnn_coo_to_csr: workspace of %zu bytes needed", gnn_coo_to_csr_workspace(N, E));
    cudaStream_t st = as_stream(stream);
    SortWs w = carve(ws, E);
    out->N = N;
    out->E = E;

    if (cudaMemsetAsync(w.flag, 0, sizeof(int), st) != cudaSuccess)
        GNN_FAIL(GNN_ERR_CUDA, "gnn_coo_to_csr: memset failed (is ws a device pointer?)");
    if (E > 0) validate_coo_kernel<<<grid_for(E, 256), 256, 0, st>>>(N, E, src, dst, w.flag);
    GNN_CHECK_LAUNCH("validate_coo");
    int h_flag = 0;
    if (cudaMemcpyAsync(&h_flag, w.flag, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        GNN_FAIL(GNN_ERR_CUDA, "gnn_coo_to_csr: reading the validation flag failed: %s",
                 cudaGetErrorString(cudaGetLastError()));
    GNN_REQUIRE(h_flag == 0, GNN_ERR_INDEX_OUT_OF_RANGE,
                "gnn_coo_to_csr: an edge endpoint is outside [0, %d)", N);

    const int32_t *sk, *sv;
    gnn_status rc;
    const int fgrid = grid_for(E > N ? E : (int64_t)N + 1, 256);
    // by target
    if ((rc = sort_by_key(N, E, dst, w, st, &sk, &sv)) != GNN_OK) return rc;
    csr_finalize_kernel<<<fgrid, 256, 0, st>>>(N, E, sk, sv, src, out->rowptr, out->col, out->eid);
    GNN_CHECK_LAUNCH("csr_finalize");
    // by source
    if ((rc = sort_by_key(N, E, src, w, st, &sk, &sv)) != GNN_OK) return rc;
    csr_finalize_kernel<<<fgrid, 256, 0, st>>>(N, E, sk, sv, dst, out->rowptrT, out->colT, out->eidT);
    GNN_CHECK_LAUNCH("csr_finalize (transposed)");
    if (E > 0) {
        invert_perm_kernel<<<grid_for(E, 256), 256, 0, st>>>(E, out->eid, w.kA);
        compose_perm_kernel<<<grid_for(E, 256), 256, 0, st>>>(E, w.kA, out->eidT, out->t2f);
        GNN_CHECK_LAUNCH("t2f");
    }
    return GNN_OK;
}

size_t gnn_csr_validate_workspace(int64_t E) {
    if (E < 0) return 0;
    return 256 + up256((size_t)3 * (size_t)((E + 31) / 32) * 4);
}

gnn_status gnn_csr_validate(const gnn_csr* g, void* ws, size_t ws_bytes, gnn_stream stream) {
    GNN_REQUIRE(g, GNN_ERR_INVALID_ARG, "gnn_csr_validate: null graph");
    GNN_REQUIRE(g->N >= 0 && g->E >= 0 && g->E <= 0x7FFFFFFFLL - 1, GNN_ERR_INVALID_ARG, "gnn_csr_validate: bad sizes (N=%d, E=%lld)", g->N, (long long)g->E);
    GNN_REQUIRE(g->rowptr && g->rowptrT, GNN_ERR_INVALID_ARG, "gnn_csr_validate: null row pointers");
    GNN_REQUIRE(g->E == 0 || (g->col && g->eid && g->colT && g->eidT && g->t2f), GNN_ERR_INVALID_ARG, "gnn_csr_validate: null edge array");
    const size_t need = gnn_csr_validate_workspace(g->E);
    GNN_REQUIRE(ws && ws_bytes >= need, GNN_ERR_WORKSPACE_TOO_SMALL, "gnn_csr_validate: workspace of %zu bytes needed", need);
    cudaStream_t st = as_stream(stream);
    int* flag = (int*)ws;
    unsigned* seen = (unsigned*)((char*)ws + 256);
    const int64_t words = (g->E + 31) / 32;
    if (cudaMemsetAsync(ws, 0, need, st) != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "gnn_csr_validate: memset failed (is ws a device pointer?)");
    auto read_flag = [&](int* h) {
        return cudaMemcpyAsync(h, flag, sizeof(int), cudaMemcpyDeviceToHost, st) == cudaSuccess && cudaStreamSynchronize(st) == cudaSuccess;
    };
    csr_validate_pointers_kernel<<<(int)ceil_div((int64_t)g->N + 1, 256), 256, 0, st>>>(g->N, g->E, g->rowptr, g->rowptrT, flag);
    GNN_CHECK_LAUNCH("csr_validate_pointers");
    int h = 0;
    if (!read_flag(&h)) GNN_FAIL(GNN_ERR_CUDA, "gnn_csr_validate: reading the result failed: %s", cudaGetErrorString(cudaGetLastError()));
    if (h == 0 && g->E > 0 && g->N > 0) {  // the position checks look rows up through the pointers: only once those are sound
        csr_validate_positions_kernel<<<(int)ceil_div(g->E, 256), 256, 0, st>>>(g->N, g->E, g->rowptr, g->col, g->eid, g->rowptrT, g->colT,
                                                                           g->eidT, g->t2f, seen, words, flag);
        GNN_CHECK_LAUNCH("csr_validate_positions");
        if (!read_flag(&h)) GNN_FAIL(GNN_ERR_CUDA, "gnn_csr_validate: reading the result failed: %s", cudaGetErrorString(cudaGetLastError()));
    }
    GNN_REQUIRE(h == 0, GNN_ERR_INVALID_ARG, "gnn_csr_validate: not a sparse form of one edge list:%s%s%s%s%s%s",
                (h & CSR_BAD_ROWPTR) ? " row pointers (0 .. E, non-decreasing);" : "", (h & CSR_BAD_NODE) ? " node index outside [0, N);" : "",
                (h & CSR_BAD_EDGE) ? " edge index outside [0, E);" : "", (h & CSR_BAD_PERM) ? " eid / eidT / t2f not a permutation;" : "",
                (h & CSR_BAD_ORDER) ? " edge ids not ascending inside a row;" : "", (h & CSR_BAD_CROSS) ? " the two forms describe different edges;" : "");
    return GNN_OK;
}

gnn_status gnn_degree(const gnn_csr* g, int transposed, const float* w, void* deg_out,
                      gnn_stream stream) {
    GNN_REQUIRE(g && deg_out, GNN_ERR_INVALID_ARG, "gnn_degree: null argument");
    const int64_t* rp = transposed ? g->rowptrT : g->rowptr;
    GNN_REQUIRE(rp, GNN_ERR_INVALID_ARG, "gnn_degree: null rowptr");
    if (g->N == 0) return GNN_OK;
    cudaStream_t st = as_stream(stream);
    if (!w)
        degree_count_kernel<<<(int)ceil_div(g->N, 256), 256, 0, st>>>(g->N, rp, (int32_t*)deg_out);
    else
        degree_weighted_kernel<<<(int)ceil_div((int64_t)g->N * 32, 256), 256, 0, st>>>(g->N, rp, w, (float*)deg_out);
    GNN_CHECK_LAUNCH("gnn_degree");
    return GNN_OK;
}

gnn_status gnn_add_self_loops(int32_t N, int64_t E, const int32_t* src, const int32_t* dst,
                              int32_t* src_out, int32_t* dst_out, gnn_stream stream) {
    GNN_REQUIRE(N >= 0 && E >= 0, GNN_ERR_INVALID_ARG, "gnn_add_self_loops: negative size");
    GNN_REQUIRE(E + N <= 0x7FFFFFFFLL - 1, GNN_ERR_UNSUPPORTED, "gnn_add_self_loops: E+N must be < 2^31");
    if (E + N == 0) return GNN_OK;
    GNN_REQUIRE(src_out && dst_out && (E == 0 || (src && dst)), GNN_ERR_INVALID_ARG,
                "gnn_add_self_loops: null argument");
    add_self_loops_kernel<<<grid_for(E + N, 256), 256, 0, as_stream(stream)>>>(N, E, src, dst, src_out, dst_out);
    GNN_CHECK_LAUNCH("gnn_add_self_loops");
    return GNN_OK;
}

gnn_status gnn_gcn_norm(const gnn_csr* g, const float* w_csr, float* deg_out, float* coef_csr,
                        float* coef_csrT, gnn_stream stream) {
    GNN_REQUIRE(g && g->rowptr && deg_out, GNN_ERR_INVALID_ARG, "gnn_gcn_norm: null argument");
    GNN_REQUIRE(!coef_csrT || coef_csr, GNN_ERR_INVALID_ARG,
                "gnn_gcn_norm: coef_csrT is derived from coef_csr, which is NULL");
    if (g->N == 0) return GNN_OK;
    cudaStream_t st = as_stream(stream);
    if (w_csr)
        degree_weighted_kernel<<<(int)ceil_div((int64_t)g->N * 32, 256), 256, 0, st>>>(g->N, g->rowptr, w_csr, deg_out);
    else
        degree_unit_kernel<<<(int)ceil_div(g->N, 256), 256, 0, st>>>(g->N, g->rowptr, deg_out);
    if (coef_csr && g->E > 0) {
        GNN_REQUIRE(g->col, GNN_ERR_INVALID_ARG, "gnn_gcn_norm: null col");
        gcn_coef_kernel<false><<<(int)ceil_div((int64_t)g->N * 32, 256), 256, 0, st>>>(g->N, g->rowptr, g->col, w_csr, deg_out, coef_csr);
        gcn_coef_kernel<true><<<g->N < 148 * 8 ? g->N : 148 * 8, 256, 0, st>>>(g->N, g->rowptr, g->col, w_csr, deg_out, coef_csr);
        if (coef_csrT) {
            GNN_REQUIRE(g->t2f, GNN_ERR_INVALID_ARG, "gnn_gcn_norm: null t2f");
            permute_f32_kernel<<<grid_for(g->E, 256), 256, 0, st>>>(g->E, g->t2f, coef_csr, coef_csrT);
        }
    }
    GNN_CHECK_LAUNCH("gnn_gcn_norm");
    return GNN_OK;
}

gnn_status gnn_permute_edge_data(const int32_t* perm, int64_t E, int width, int elem_bytes,
                                 const void* in, void* out, gnn_stream stream) {
    GNN_REQUIRE(E >= 0 && width >= 1, GNN_ERR_INVALID_ARG, "gnn_permute_edge_data: bad size");
    if (E == 0) return GNN_OK;
    GNN_REQUIRE(perm && in && out && in != out, GNN_ERR_INVALID_ARG, "gnn_permute_edge_data: null or aliased argument");
    cudaStream_t st = as_stream(stream);
    int grid = grid_for(E * width, 256);
    switch (elem_bytes) {
        case 1: permute_rows_kernel<uint8_t><<<grid, 256, 0, st>>>(E, width, perm, (const uint8_t*)in, (uint8_t*)out); break;
        case 2: permute_rows_kernel<uint16_t><<<grid, 256, 0, st>>>(E, width, perm, (const uint16_t*)in, (uint16_t*)out); break;
        case 4: permute_rows_kernel<uint32_t><<<grid, 256, 0, st>>>(E, width, perm, (const uint32_t*)in, (uint32_t*)out); break;
        case 8: permute_rows_kernel<uint64_t><<<grid, 256, 0, st>>>(E, width, perm, (const uint64_t*)in, (uint64_t*)out); break;
        default: GNN_FAIL(GNN_ERR_UNSUPPORTED, "gnn_permute_edge_data: elem_bytes must be 1, 2, 4 or 8");
    }
    GNN_CHECK_LAUNCH("gnn_permute_edge_data");
    return GNN_OK;
}

}  // extern "C"
