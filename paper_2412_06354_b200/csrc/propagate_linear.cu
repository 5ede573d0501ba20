// Aggregate -> transform fusion: Y = epilogue( (op over the incoming edges of w * X[source,:]) * W ), the
// propagate of Sec. 3 "Message Passing" followed by the weight of a conv layer (the GCNConv of the training
// example), without writing the aggregated [N,K] matrix to memory.
//
// One persistent CTA per SM works on tiles of 128 target rows:
//   gather warps   reduce the rows of the tile (fp32 accumulation in a fixed order) and write them, rounded to
//                  bf16 (fp32 input: split exactly into three bf16 terms), straight into the shared-memory
//                  operand tile in the tensor core's K-major 128-byte-swizzled layout.  A lane group owns
//                  whole rows, taken from a per-tile counter, and keeps eight row gathers in flight across the
//                  rows it owns (most rows have a handful of edges); rows longer than PL_LONG positions are
//                  left to a second phase in which all gather warps split each such row and add their partial
//                  sums in warp order (a 1000-position row walked by one lane group, eight gathers at a time,
//                  would hold its tile for a hundred load latencies).  Which group reduces a row does not change the order of its additions, so
//                  results are bit-reproducible.
//   warp 0         issues tcgen05.mma (128 x M x 16, fp32 accumulator in tensor memory; fp32 input: the six
//                  products of the three-term split with i + j <= 4) on the tile and the resident weights.
//   warps 1..4     epilogue: accumulator -> bias / relu -> staging block -> bulk tensor store to Y.
// Every wait is bounded: on expiry a status word reports GNN_ERR_TIMEOUT and the roles leave their loops.
#include <cuda.h>

#include "propagate.cuh"
#include "tc_common.cuh"

namespace gnn {

bool make_map(CUtensorMap* m, const void* ptr, int64_t rows, int cols, int box_rows);      // bf16, 64-column boxes
bool make_map_f32(CUtensorMap* m, const void* ptr, int64_t rows, int cols, int box_rows);  // fp32, 32-column boxes
bool tensor_map_encoder_available();

#ifndef PL_GATHER_WARPS_N
#define PL_GATHER_WARPS_N 11
#endif
constexpr int PL_GATHER_WARPS = PL_GATHER_WARPS_N;
constexpr int PL_EPI_WARPS = 4;
constexpr int PL_THREADS = 32 * (1 + PL_EPI_WARPS + PL_GATHER_WARPS);
#ifndef PL_U_N
#define PL_U_N 8
#endif
constexpr int PL_U = PL_U_N;         // row gathers a lane group keeps in flight
#ifndef PL_LONG_N
#define PL_LONG_N 128
#endif
#ifndef PL_LONG_WARPS_N
#define PL_LONG_WARPS_N 11
#endif
constexpr int PL_LONG = PL_LONG_N;   // rows longer than this are split over PL_LONG_WARPS warps
constexpr int PL_LONG_WARPS = PL_LONG_WARPS_N;
static_assert(PL_LONG_WARPS <= PL_GATHER_WARPS, "the second phase runs on gather warps");
constexpr int PL_WINDOW = 2048;      // positions of a tile whose indices (and multipliers) are staged in shared memory
constexpr int PL_MAX_STAGES = 2;
constexpr uint32_t PL_SLICE_BYTES = TC_ROWS * 128;  // 64 bf16 columns of the 128-row operand tile
constexpr size_t PL_SMEM_MAX = 222 * 1024;  // dynamic shared memory per CTA (227 KB less the static part)
constexpr uint32_t PL_SW128 = 2;

__device__ __constant__ unsigned char kPlPairA[6] = {2, 0, 1, 1, 0, 0};  // levels of A and B per product, small terms first
__device__ __constant__ unsigned char kPlPairB[6] = {0, 2, 1, 0, 1, 0};

struct PlParams {
    const int64_t* rowptr;
    const int32_t* col;
    const float* w;     // per-position multiplier or nullptr
    const int64_t* gscale_rowptr;  // if set: a gathered row c is divided by max(1, length of row c in this other form)
    const void* X;      // [*, K] gathered rows
    const void* W;      // [K,M] (b_transposed = 0) or [M,K] (b_transposed = 1), same dtype as X
    const float* bias;  // [M] or nullptr
    int relu;
    int32_t N;
    int K, M;
    int mean;
    int b_transposed;
    int stages;
    int window;         // positions of a tile whose indices and multipliers are staged in shared memory (per stage)
    int acc_stride, tmem_cols;
    int* status;
};

__device__ __forceinline__ void pl_st16(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void pl_st8(uint32_t addr, uint32_t a, uint32_t b) {
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "r"(a), "r"(b) : "memory");
}
__device__ __forceinline__ void pl_named_barrier(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// x = x1 + x2 + x3 exactly, each term a bf16 (the remainders are exact in fp32)
__device__ __forceinline__ void pl_split3(float x, uint32_t* t) {
#pragma unroll
    for (int l = 0; l < 3; ++l) {
        const __nv_bfloat16 b = __float2bfloat16_rn(x);
        t[l] = (uint32_t)__bfloat16_as_ushort(b);
        x -= __bfloat162float(b);
    }
}

// Finished row r of the tile (EPC fp32 values of 16-byte input chunk ci) -> operand tile(s).
// bf16 input: one 16-byte chunk of 8 columns.  fp32 input: 4 columns = half a chunk, three levels.
template <typename T>
__device__ __forceinline__ void pl_store_row(uint32_t stage, uint32_t level_bytes, int r, int ci, const float* v) {
    if (sizeof(T) == 2) {
        const int j = ci >> 3, c = ci & 7;  // 64-column slice, 16-byte chunk inside its 128-byte row
        pl_st16(stage + (uint32_t)j * PL_SLICE_BYTES + (uint32_t)r * 128u + (uint32_t)((c ^ (r & 7)) << 4), Chunk<__nv_bfloat16>::pack(v));
    } else {
        const int k0 = ci * 4, j = k0 >> 6, c = (k0 & 63) >> 3, half = (k0 >> 2) & 1;
        uint32_t t[4][3];
#pragma unroll
        for (int q = 0; q < 4; ++q) pl_split3(v[q], t[q]);
        const uint32_t a = stage + (uint32_t)j * PL_SLICE_BYTES + (uint32_t)r * 128u + (uint32_t)((c ^ (r & 7)) << 4) + (uint32_t)half * 8u;
#pragma unroll
        for (int l = 0; l < 3; ++l) pl_st8(a + (uint32_t)l * level_bytes, t[0][l] | (t[1][l] << 16), t[2][l] | (t[3][l] << 16));
    }
}

// shared-memory bookkeeping of one operand-tile stage
struct PlStageCtl {
    int next_row;                 // next row of the tile nobody has taken yet
    int n_long;                   // rows left to the second phase
    int long_rows[TC_ROWS];
    int rp[TC_ROWS + 1];         // row pointers of the tile's rows (clamped past the last row); E < 2^31
};

// Phase 1 of a tile for one lane group: row r of the tile, at most PL_LONG positions, PL_U gathers in flight.
// Out of line so that the registers of this loop are not shared with the rest of the kernel (a spilled
// register here costs a trip to L2: the kernel's shared memory leaves the L1 almost no room).
template <typename T, bool WEIGHTED>
__device__ __noinline__ void pl_take_row(const PlParams& P, int rs, int len, int r, uint32_t stage, uint32_t level_bytes,
                                         const char* Xl, uint32_t row_bytes, int li, bool col_lane, uint64_t pol_keep,
                                         const int* scol, const float* sw) {
    constexpr int EPC = Chunk<T>::N;
    float acc[EPC];
#pragma unroll
    for (int j = 0; j < EPC; ++j) acc[j] = 0.f;
    const int32_t* const colp = P.col + rs;
    if (scol) {  // the row lies inside the staged window: indices and multipliers come from shared memory
        for (int q0 = 0; q0 < len; q0 += PL_U) {
            uint4 buf[PL_U];
#pragma unroll
            for (int u = 0; u < PL_U; ++u)
                if (q0 + u < len) buf[u] = ld_hint16(Xl + (size_t)(uint32_t)scol[q0 + u] * row_bytes, pol_keep);
#pragma unroll
            for (int u = 0; u < PL_U; ++u) {
                if (q0 + u >= len) break;
                float x[EPC];
                Chunk<T>::unpack(buf[u], x);
                const float wq = WEIGHTED ? sw[q0 + u] : 1.0f;
#pragma unroll
                for (int j = 0; j < EPC; ++j) acc[j] = WEIGHTED ? fmaf(wq, x[j], acc[j]) : acc[j] + x[j];
            }
        }
    } else
    for (int q0 = 0; q0 < len; q0 += PL_U) {
        int cols[PL_U];
        uint4 buf[PL_U];
        float wv[WEIGHTED ? PL_U : 1];
#pragma unroll
        for (int u = 0; u < PL_U; ++u) cols[u] = q0 + u < len ? __ldg(colp + q0 + u) : 0;
#pragma unroll
        for (int u = 0; u < PL_U; ++u)
            if (q0 + u < len) {
                buf[u] = ld_hint16(Xl + (size_t)(uint32_t)cols[u] * row_bytes, pol_keep);
                if (WEIGHTED) {
                    float wq = P.w ? __ldg(P.w + rs + q0 + u) : 1.0f;
                    if (P.gscale_rowptr) {
                        const int64_t d = P.gscale_rowptr[cols[u] + 1] - P.gscale_rowptr[cols[u]];
                        wq = wq / (float)(d > 1 ? d : 1);
                    }
                    wv[WEIGHTED ? u : 0] = wq;
                }
            }
#pragma unroll
        for (int u = 0; u < PL_U; ++u) {
            if (q0 + u >= len) break;
            float x[EPC];
            Chunk<T>::unpack(buf[u], x);
#pragma unroll
            for (int j = 0; j < EPC; ++j) acc[j] = WEIGHTED ? fmaf(wv[WEIGHTED ? u : 0], x[j], acc[j]) : acc[j] + x[j];
        }
    }
    if (!col_lane) return;
    if (P.mean) {
        const float d = (float)(len > 1 ? len : 1);
#pragma unroll
        for (int j = 0; j < EPC; ++j) acc[j] = acc[j] / d;
    }
    pl_store_row<T>(stage, level_bytes, r, li, acc);
}

// Phase 2: this warp's share of one long row (positions rs + gw * per ...), lane groups interleaved, combined by
// a fixed shuffle tree; lanes of group 0 leave the partial sum in part[gw][...]
template <typename T, bool WEIGHTED>
__device__ __noinline__ void pl_long_share(const PlParams& P, int rs, int len, int gw, float* part, const char* Xl, uint32_t row_bytes,
                                           int lane, int lpr, bool col_lane, uint64_t pol_keep) {
    constexpr int EPC = Chunk<T>::N;
    const int K = P.K, g = lane / lpr, li = lane % lpr, ng = 32 / lpr, re = rs + len;
    const int per = (len + PL_LONG_WARPS - 1) / PL_LONG_WARPS;
    const int pa = rs + gw * per, pb = (pa + per < re) ? pa + per : re;
    float acc[EPC];
#pragma unroll
    for (int j = 0; j < EPC; ++j) acc[j] = 0.f;
    for (int p0 = pa + g; p0 < pb; p0 += ng * PL_U) {
        uint4 buf[PL_U];
        float wv[WEIGHTED ? PL_U : 1];
#pragma unroll
        for (int u = 0; u < PL_U; ++u) {
            const int p = p0 + u * ng;
            if (p < pb) {
                const int cc = __ldg(P.col + p);
                buf[u] = ld_hint16(Xl + (size_t)(uint32_t)cc * row_bytes, pol_keep);
                if (WEIGHTED) {
                    float wq = P.w ? __ldg(P.w + p) : 1.0f;
                    if (P.gscale_rowptr) {
                        const int64_t d = P.gscale_rowptr[cc + 1] - P.gscale_rowptr[cc];
                        wq = wq / (float)(d > 1 ? d : 1);
                    }
                    wv[WEIGHTED ? u : 0] = wq;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < PL_U; ++u) {
            if (p0 + u * ng >= pb) break;
            float x[EPC];
            Chunk<T>::unpack(buf[u], x);
#pragma unroll
            for (int j = 0; j < EPC; ++j) acc[j] = WEIGHTED ? fmaf(wv[WEIGHTED ? u : 0], x[j], acc[j]) : acc[j] + x[j];
        }
    }
    __syncwarp();
    for (int o = lpr; o < 32; o <<= 1) {  // combine the lane groups: both partners add in the same operand order
        const bool low = (lane & o) == 0;
#pragma unroll
        for (int j = 0; j < EPC; ++j) {
            const float ov = __shfl_xor_sync(0xffffffffu, acc[j], o);
            acc[j] = low ? (acc[j] + ov) : (ov + acc[j]);
        }
    }
    if (lane < lpr && col_lane) {
#pragma unroll
        for (int j = 0; j < EPC; ++j) part[(size_t)gw * K + li * EPC + j] = acc[j];
    }
}

template <typename T, bool WEIGHTED>
__global__ void __launch_bounds__(PL_THREADS, 1)
propagate_linear_kernel(const __grid_constant__ CUtensorMap mapY, const __grid_constant__ PlParams P) {
    constexpr int EPC = Chunk<T>::N;
    constexpr int LEVELS = sizeof(T) == 2 ? 1 : 3, PAIRS = sizeof(T) == 2 ? 1 : 6;
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * PL_MAX_STAGES + 4];  // a_full[S], a_empty[S], acc_full[2], acc_empty[2]
    __shared__ uint32_t tmem_base_slot;
    __shared__ PlStageCtl ctl[PL_MAX_STAGES];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = P.K, M = P.M, S = P.stages;
    const int kblocks = (K + 63) / 64, kchunks = K / 8;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t b_level = (uint32_t)M * K * 2, b_sbo = (uint32_t)kchunks * 128;
    const uint32_t level_bytes = (uint32_t)kblocks * PL_SLICE_BYTES, stage_bytes = level_bytes * LEVELS;
    const uint32_t w0 = base;
    const uint32_t a0 = base + (((uint32_t)LEVELS * b_level + 1023u) & ~1023u);
    const uint32_t stg0 = a0 + (uint32_t)S * stage_bytes;                  // per epilogue warp: 32 rows x 128 bytes
    const uint32_t part0 = stg0 + PL_EPI_WARPS * 4096u;                    // PL_LONG_WARPS partial rows of K floats
    const uint32_t win0 = part0 + (uint32_t)PL_LONG_WARPS * (uint32_t)K * 4u;           // per stage: window ints + window floats
    const uint32_t bar0 = smem_u32(bars);
    auto a_full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto a_empty = [&](int s) { return bar0 + 8u * (uint32_t)(PL_MAX_STAGES + s); };
    auto acc_full = [&](int a) { return bar0 + 8u * (uint32_t)(2 * PL_MAX_STAGES + a); };
    auto acc_empty = [&](int a) { return bar0 + 8u * (uint32_t)(2 * PL_MAX_STAGES + 2 + a); };

    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(a_full(s), PL_GATHER_WARPS); mbar_init(a_empty(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(acc_full(a), 1); mbar_init(acc_empty(a), PL_EPI_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapY)) : "memory");
    }
    if (tid < PL_MAX_STAGES) { ctl[tid].next_row = 0; ctl[tid].n_long = 0; }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)P.tmem_cols);
    // Weights -> shared memory in the canonical no-swizzle layout (core matrix = 8 rows x 16 bytes), once per CTA.
    // 16-byte chunk c of stored row r:
    //   stored [K,M] (MN-major B): r = k, c = 8 output columns: offset c*sbo + (k/8)*128 + (k%8)*16
    //   stored [M,K] (K-major  B): r = n, c = 8 k's:            offset (n/8)*sbo + c*128 + (n%8)*16
    {
        const int rows = P.b_transposed ? M : K, chunks = (P.b_transposed ? K : M) / 8;
        for (int e = tid; e < rows * chunks; e += PL_THREADS) {
            const int q = e >> 3, rg = q / chunks, c = q - rg * chunks, r = rg * 8 + (e & 7);
            const uint32_t off = P.b_transposed ? (uint32_t)(r >> 3) * b_sbo + (uint32_t)c * 128 + (uint32_t)(r & 7) * 16
                                                : (uint32_t)c * b_sbo + (uint32_t)(r >> 3) * 128 + (uint32_t)(r & 7) * 16;
            if (sizeof(T) == 2) {
                pl_st16(w0 + off, __ldg(reinterpret_cast<const uint4*>(P.W) + (size_t)r * chunks + c));
            } else {
                const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(P.W) + ((size_t)r * chunks + c) * 8);
                const float4 lo = __ldg(src), hi = __ldg(src + 1);
                const float x[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
                uint32_t t[8][3];
#pragma unroll
                for (int q8 = 0; q8 < 8; ++q8) pl_split3(x[q8], t[q8]);
#pragma unroll
                for (int l = 0; l < 3; ++l)
                    pl_st16(w0 + (uint32_t)l * b_level + off, make_uint4(t[0][l] | (t[1][l] << 16), t[2][l] | (t[3][l] << 16),
                                                                          t[4][l] | (t[5][l] << 16), t[6][l] | (t[7][l] << 16)));
            }
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    const int64_t ntiles = ((int64_t)P.N + TC_ROWS - 1) / TC_ROWS;
    bool failed = false;

    if (warp == 0) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc(M, P.b_transposed ? 0 : 1);
            uint32_t lt = 0;
            for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x, ++lt) {
                const uint32_t a = lt & 1u;
                const int s = (int)(lt % (uint32_t)S);
                if (!mbar_wait_bounded(acc_empty((int)a), ((lt >> 1) & 1u) ^ 1u)) { failed = true; break; }
                if (!mbar_wait_bounded(a_full(s), (lt / (uint32_t)S) & 1u)) { failed = true; break; }
                tc_fence_after();
                const uint32_t dacc = tmem_base + a * (uint32_t)P.acc_stride;
                const uint32_t stage = a0 + (uint32_t)s * stage_bytes;
                for (int j = 0; j < kblocks; ++j) {
                    const int ksteps = (K - j * 64) >= 64 ? 4 : (K - j * 64) / 16;
                    for (int kk = 0; kk < ksteps; ++kk)
                        for (int q = 0; q < PAIRS; ++q) {
                            const uint32_t la = PAIRS == 1 ? 0u : kPlPairA[q], lb = PAIRS == 1 ? 0u : kPlPairB[q];
                            // A: rows 128 bytes apart, groups of 8 rows 1024 bytes apart; a k-step is 32 bytes along the row
                            const uint64_t adesc = make_smem_desc(stage + la * level_bytes + (uint32_t)j * PL_SLICE_BYTES + (uint32_t)kk * 32u, 16, 1024, PL_SW128);
                            const uint64_t bdesc = make_smem_desc(w0 + lb * b_level + (uint32_t)(j * 4 + kk) * 256u, 128, b_sbo);
                            mma_bf16_ss(dacc, adesc, bdesc, idesc, (j > 0 || kk > 0 || q > 0) ? 1u : 0u);
                        }
                }
                mma_commit(a_empty(s));
                mma_commit(acc_full((int)a));
            }
        }
    } else if (warp <= PL_EPI_WARPS) {
        // ------------------------------------------------------------ epilogue (tensor-memory lanes 32*(warp % 4)..)
        const int quarter = warp & 3;
        const uint32_t stg = stg0 + (uint32_t)(warp - 1) * 4096u;
        constexpr int CB = sizeof(T) == 2 ? 64 : 32;  // columns per 128-byte staging row
        uint32_t lt = 0;
        for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x, ++lt) {
            const uint32_t a = lt & 1u;
            if (!mbar_wait_bounded(acc_full((int)a), (lt >> 1) & 1u)) { failed = true; break; }
            tc_fence_after();
            const int64_t row0 = t * TC_ROWS + quarter * 32;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + a * (uint32_t)P.acc_stride;
            for (int cb = 0; cb * CB < M; ++cb) {
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // staging block free again
                __syncwarp();
                const int groups = (M - cb * CB >= CB ? CB : M - cb * CB) / 16;
                for (int g16 = 0; g16 < groups; ++g16) {
                    uint32_t r[16];
                    tmem_ld16(taddr + (uint32_t)(cb * CB + g16 * 16), r);
                    tmem_ld_wait();
                    float f[16];
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        f[q] = __uint_as_float(r[q]);
                        if (P.bias) f[q] += __ldg(P.bias + cb * CB + g16 * 16 + q);
                        if (P.relu) f[q] = fmaxf(f[q], 0.f);
                    }
                    // row = lane, 128 bytes per row; 16-byte chunk c sits at position c ^ (row % 8)
                    if (sizeof(T) == 2) {
#pragma unroll
                        for (int h2 = 0; h2 < 2; ++h2)
                            pl_st16(stg + (uint32_t)lane * 128u + ((uint32_t)((2 * g16 + h2) ^ (lane & 7)) << 4), Chunk<__nv_bfloat16>::pack(f + 8 * h2));
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            pl_st16(stg + (uint32_t)lane * 128u + ((uint32_t)((4 * g16 + q) ^ (lane & 7)) << 4),
                                    make_uint4(__float_as_uint(f[4 * q]), __float_as_uint(f[4 * q + 1]), __float_as_uint(f[4 * q + 2]), __float_as_uint(f[4 * q + 3])));
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0 && row0 < P.N) {  // rows past N are clipped by the copy engine
                    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                                     reinterpret_cast<uint64_t>(&mapY)),
                                 "r"(cb * CB), "r"((int)row0), "r"(stg)
                                 : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty((int)a));
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    } else {
        // ------------------------------------------------------------ gather warps
        constexpr int GT = 32 * PL_GATHER_WARPS;
        const int gw = warp - (1 + PL_EPI_WARPS), gt = tid - 32 * (1 + PL_EPI_WARPS);
        const int nvec = K * (int)sizeof(T) / 16;              // 16-byte chunks per gathered row (<= 32)
        const int lpr = nvec <= 4 ? 4 : nvec <= 8 ? 8 : nvec <= 16 ? 16 : 32;
        const int g = lane / lpr, li = lane % lpr, ng = 32 / lpr;
        const unsigned gmask = lpr == 32 ? 0xffffffffu : (((1u << lpr) - 1u) << (g * lpr));
        const bool col_lane = li < nvec;
        const uint32_t row_bytes = (uint32_t)nvec * 16u;
        const char* const Xl = reinterpret_cast<const char*>(P.X) + (size_t)(col_lane ? li : 0) * 16;
        const uint64_t pol_keep = policy_evict_last();
        uint32_t lt = 0;
        for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x, ++lt) {
            const int s = (int)(lt % (uint32_t)S);
            PlStageCtl& C = ctl[s];
            const uint32_t stage = a0 + (uint32_t)s * stage_bytes;
            int* const ecol = reinterpret_cast<int*>(smem_raw + (win0 - smem_u32(smem_raw)) + (size_t)s * P.window * 8);
            float* const ew = reinterpret_cast<float*>(ecol + P.window);
            // the tensor core has read the previous contents of this stage (first uses: passes at once)
            int ok = 1;
            if (lane == 0) ok = mbar_wait_bounded(a_empty(s), ((lt / (uint32_t)S) & 1u) ^ 1u) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            {   // every gather warp takes the same decision: a warp that left alone would hang the others' barriers
                int any_failed;
                asm volatile("{\n\t.reg .pred p, q;\n\tsetp.eq.s32 q, %1, 0;\n\tbar.red.or.pred p, 1, %2, q;\n\tselp.s32 %0, 1, 0, p;\n\t}\n"
                             : "=r"(any_failed) : "r"(ok), "r"(GT) : "memory");
                if (any_failed) { failed = true; break; }
            }
            const int64_t row0 = t * TC_ROWS;
            if (gt <= TC_ROWS) {
                const int64_t r = row0 + gt < P.N ? row0 + gt : P.N;
                C.rp[gt] = (int)P.rowptr[r];
            }
            if (gt == 0) { C.next_row = 0; C.n_long = 0; }
            pl_named_barrier(1, GT);
            {   // stage the indices (and multipliers, rescaled once) of the tile's first PL_WINDOW positions
                const int p0 = C.rp[0], nw = min(C.rp[TC_ROWS] - p0, P.window);
                for (int i = gt; i < nw; i += GT) {
                    const int cc = __ldg(P.col + p0 + i);
                    ecol[i] = cc;
                    if (WEIGHTED) {
                        float wq = P.w ? __ldg(P.w + p0 + i) : 1.0f;
                        if (P.gscale_rowptr) {
                            const int64_t d = P.gscale_rowptr[cc + 1] - P.gscale_rowptr[cc];
                            wq = wq / (float)(d > 1 ? d : 1);
                        }
                        ew[i] = wq;
                    }
                }
            }
            pl_named_barrier(1, GT);

            // ---- phase 1: a lane group takes one row at a time from the tile's counter
            for (;;) {
                int r = 0;
                if (li == 0) r = atomicAdd(&C.next_row, 1);
                r = __shfl_sync(gmask, r, g * lpr);
                if (r >= TC_ROWS) break;
                const int rs = C.rp[r], len = C.rp[r + 1] - rs;
                if (len > PL_LONG) {
                    if (li == 0) C.long_rows[atomicAdd(&C.n_long, 1)] = r;
                    continue;
                }
                const int off = rs - C.rp[0];
                const bool staged = off + len <= P.window;
                pl_take_row<T, WEIGHTED>(P, rs, len, r, stage, level_bytes, Xl, row_bytes, li, col_lane, pol_keep,
                                         staged ? ecol + off : nullptr, staged ? ew + off : nullptr);
            }
            __syncwarp();
            pl_named_barrier(1, GT);

            // ---- phase 2: long rows, each split over PL_LONG_WARPS warps whose partial sums are added in warp order
            const int nl = C.n_long;
            if (nl > 0 && gw < PL_LONG_WARPS) {
                for (int k = 0; k < nl; ++k) {
                    const int r = C.long_rows[k];
                    const int len = C.rp[r + 1] - C.rp[r];
                    float* part = reinterpret_cast<float*>(smem_raw + (part0 - smem_u32(smem_raw)));
                    pl_long_share<T, WEIGHTED>(P, C.rp[r], len, gw, part, Xl, row_bytes, lane, lpr, col_lane, pol_keep);
                    pl_named_barrier(2, 32 * PL_LONG_WARPS);
                    if (gw == 0 && lane < lpr && col_lane) {
                        float v[EPC];
#pragma unroll
                        for (int j = 0; j < EPC; ++j) {
                            float sum = part[li * EPC + j];
                            for (int q = 1; q < PL_LONG_WARPS; ++q) sum += part[(size_t)q * K + li * EPC + j];
                            v[j] = P.mean ? sum / (float)len : sum;
                        }
                        pl_store_row<T>(stage, level_bytes, r, li, v);
                    }
                    pl_named_barrier(2, 32 * PL_LONG_WARPS);
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(a_full(s));
        }
    }
    if (failed) atomicExch(P.status, 7);  // GNN_ERR_TIMEOUT
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols);
}

// ------------------------------------------------------------------ host side
static size_t pl_fixed_bytes(int K, int M, int levels) {
    return 1024 + (((size_t)levels * M * K * 2 + 1023) & ~(size_t)1023) + (size_t)PL_EPI_WARPS * 4096 + (size_t)PL_LONG_WARPS * K * 4;
}
static size_t pl_stage_bytes(int K, int levels) { return (size_t)levels * ((K + 63) / 64) * PL_SLICE_BYTES; }

// can the fused kernel take this product?  Kc = contraction length (width of the gathered rows), Mo = output columns
static bool pl_supported(int32_t N, int Kc, int Mo, gnn_dtype dtype) {
    if (N <= 0 || N >= 2147483647 - TC_ROWS) return false;
    if (Kc % 16 != 0 || Kc < 16 || Kc > 256 || Mo % 16 != 0 || Mo < 16 || Mo > 256) return false;
    if (Kc * elem_size(dtype) > 512) return false;  // a gathered row fills at most one warp
    const int levels = dtype == GNN_F32 ? 3 : 1;
    if (pl_fixed_bytes(Kc, Mo, levels) + pl_stage_bytes(Kc, levels) > PL_SMEM_MAX) return false;
    return tensor_map_encoder_available();
}

static gnn_status pl_launch(const char* who, const int64_t* rowptr, const int32_t* col, const float* w, const int64_t* gscale_rowptr,
                            const void* X, const void* W, int32_t N, int Kc, int Mo, int mean, int b_transposed, gnn_dtype dtype,
                            const float* bias, int relu, void* Y, int* d_status, cudaStream_t st) {
    GNN_REQUIRE(aligned16(X) && aligned16(W) && aligned16(Y), GNN_ERR_INVALID_ARG, "%s: matrices must be 16-byte aligned", who);
    CUtensorMap mapY;
    const bool ok = dtype == GNN_F32 ? make_map_f32(&mapY, Y, N, Mo, 32) : make_map(&mapY, Y, N, Mo, 32);
    if (!ok) GNN_FAIL(GNN_ERR_CUDA, "%s: tensor map encoding failed", who);
    const int levels = dtype == GNN_F32 ? 3 : 1;
    PlParams P;
    P.rowptr = rowptr; P.col = col; P.w = w; P.gscale_rowptr = gscale_rowptr; P.X = X; P.W = W; P.bias = bias; P.relu = relu;
    P.N = N; P.K = Kc; P.M = Mo; P.mean = mean; P.b_transposed = b_transposed; P.status = d_status;
    const size_t fixed = pl_fixed_bytes(Kc, Mo, levels), stage = pl_stage_bytes(Kc, levels);
    int stages = (int)((PL_SMEM_MAX - fixed) / stage);
    P.stages = stages > PL_MAX_STAGES ? PL_MAX_STAGES : stages;
    const size_t left = PL_SMEM_MAX - fixed - (size_t)P.stages * stage;
    int window = (int)(left / ((size_t)P.stages * 8)) & ~31;
    P.window = window > PL_WINDOW ? PL_WINDOW : window;
    P.acc_stride = (Mo + 31) & ~31;
    int cols = 32;
    while (cols < 2 * P.acc_stride) cols <<= 1;
    P.tmem_cols = cols;
    const size_t smem = fixed + (size_t)P.stages * stage + (size_t)P.stages * P.window * 8;
    const int64_t ntiles = ((int64_t)N + TC_ROWS - 1) / TC_ROWS;
    const int grid = (int)(ntiles < 148 ? ntiles : 148);
    gnn_status rc;
    const bool weighted = w != nullptr || gscale_rowptr != nullptr;
#define GNN_PL_CASE(TYPE, WFLAG, SLOT)                                                                  \
    {                                                                                                   \
        rc = allow_big_smem(who, (const void*)propagate_linear_kernel<TYPE, WFLAG>, SLOT, PL_SMEM_MAX); \
        if (rc != GNN_OK) return rc;                                                                    \
        propagate_linear_kernel<TYPE, WFLAG><<<grid, PL_THREADS, smem, st>>>(mapY, P);                  \
    }
    if (dtype == GNN_F32) {
        if (weighted) GNN_PL_CASE(float, true, 8) else GNN_PL_CASE(float, false, 9)
    } else {
        if (weighted) GNN_PL_CASE(__nv_bfloat16, true, 10) else GNN_PL_CASE(__nv_bfloat16, false, 11)
    }
#undef GNN_PL_CASE
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

}  // namespace gnn

using namespace gnn;

extern "C" {

size_t gnn_propagate_linear_workspace(int32_t N, int64_t E, int K, int M) {
    if (N < 0 || E < 0 || K <= 0 || M <= 0) return 0;
    const int F = K > M ? K : M;
    // status word + the aggregated matrix of the unfused path (backward with dW, shapes the fused kernel does not take)
    return 256 + up256((size_t)N * F * 4) + chunked_workspace(E, F, false) + gnn_linear_workspace(N, K, M);
}

gnn_status gnn_propagate_linear(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* X, const float* w_csr,
                                const void* W, int K, int M, gnn_dtype dtype, const float* bias, int relu,
                                void* Y, void* ws, size_t ws_bytes, gnn_stream stream) {
    const char* who = "gnn_propagate_linear";
    GNN_REQUIRE(g && g->rowptr && X && W && Y, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(g->E == 0 || g->col, GNN_ERR_INVALID_ARG, "%s: null col", who);
    GNN_REQUIRE(msg == GNN_MSG_COPY_XJ || msg == GNN_MSG_E_MUL_XJ, GNN_ERR_UNSUPPORTED, "%s: message must be COPY_XJ or E_MUL_XJ", who);
    GNN_REQUIRE(msg == GNN_MSG_COPY_XJ || w_csr, GNN_ERR_INVALID_ARG, "%s: E_MUL_XJ needs w_csr", who);
    GNN_REQUIRE(op == GNN_SUM || op == GNN_MEAN, GNN_ERR_UNSUPPORTED, "%s: op must be SUM or MEAN", who);
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "%s: bad dtype", who);
    GNN_REQUIRE(K > 0 && M > 0, GNN_ERR_INVALID_ARG, "%s: bad K or M", who);
    const size_t need = gnn_propagate_linear_workspace(g->N, g->E, K, M);
    GNN_REQUIRE(ws && ws_bytes >= need && aligned16(ws), GNN_ERR_WORKSPACE_TOO_SMALL, "%s: workspace of %zu bytes needed, %zu given", who, need, ws_bytes);
    if (g->N == 0) return GNN_OK;
    cudaStream_t st = as_stream(stream);
    const float* w = msg == GNN_MSG_E_MUL_XJ ? w_csr : nullptr;
    if (cudaMemsetAsync(ws, 0, sizeof(int), st) != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "%s: memset failed (is ws a device pointer?)", who);
    if (pl_supported(g->N, K, M, dtype))
        return pl_launch(who, g->rowptr, g->col, w, nullptr, X, W, g->N, K, M, op == GNN_MEAN, 0, dtype, bias, relu, Y, (int*)ws, st);
    // shapes the fused kernel does not take: aggregate into the workspace, then the dense transform with the same epilogue
    const int F = K > M ? K : M;
    char* H = (char*)ws + 256;
    char* pws = H + up256((size_t)g->N * F * 4);
    const size_t pbytes = chunked_workspace(g->E, F, false);
    gnn_status rc = run_chunked(who, MODE_SUM, g->N, g->E, g->rowptr, g->col, w, X, H, nullptr, nullptr, nullptr, nullptr,
                                op == GNN_MEAN, K, dtype, pws, pbytes, st);
    if (rc != GNN_OK) return rc;
    return gnn_linear_bias_act(H, W, g->N, K, M, dtype, bias, relu, Y, pws + pbytes, gnn_linear_workspace(g->N, K, M), stream);
}

gnn_status gnn_propagate_linear_backward(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* dY, const void* X,
                                         const float* w_csrT, const void* W, int K, int M, gnn_dtype dtype,
                                         void* dX, void* dW, void* ws, size_t ws_bytes, gnn_stream stream) {
    const char* who = "gnn_propagate_linear_backward";
    GNN_REQUIRE(g && g->rowptr && g->rowptrT && dY, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(g->E == 0 || g->colT, GNN_ERR_INVALID_ARG, "%s: null colT", who);
    GNN_REQUIRE(msg == GNN_MSG_COPY_XJ || msg == GNN_MSG_E_MUL_XJ, GNN_ERR_UNSUPPORTED, "%s: message must be COPY_XJ or E_MUL_XJ", who);
    GNN_REQUIRE(msg == GNN_MSG_COPY_XJ || w_csrT, GNN_ERR_INVALID_ARG, "%s: E_MUL_XJ needs w_csrT", who);
    GNN_REQUIRE(op == GNN_SUM || op == GNN_MEAN, GNN_ERR_UNSUPPORTED, "%s: op must be SUM or MEAN", who);
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "%s: bad dtype", who);
    GNN_REQUIRE(K > 0 && M > 0, GNN_ERR_INVALID_ARG, "%s: bad K or M", who);
    const size_t need = gnn_propagate_linear_workspace(g->N, g->E, K, M);
    GNN_REQUIRE(ws && ws_bytes >= need && aligned16(ws), GNN_ERR_WORKSPACE_TOO_SMALL, "%s: workspace of %zu bytes needed, %zu given", who, need, ws_bytes);
    if (g->N == 0 || (!dX && !dW)) return GNN_OK;
    cudaStream_t st = as_stream(stream);
    const float* w = msg == GNN_MSG_E_MUL_XJ ? w_csrT : nullptr;
    const int64_t* gscale = op == GNN_MEAN ? g->rowptr : nullptr;
    if (cudaMemsetAsync(ws, 0, sizeof(int), st) != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "%s: memset failed (is ws a device pointer?)", who);
    if (!dW && pl_supported(g->N, M, K, dtype)) {
        // dX = (A^T dY) * W^T: the same fused kernel on the transposed form, contraction over M
        GNN_REQUIRE(W, GNN_ERR_INVALID_ARG, "%s: dX needs W", who);
        return pl_launch(who, g->rowptrT, g->colT, w, gscale, dY, W, g->N, M, K, 0, 1, dtype, nullptr, 0, dX, (int*)ws, st);
    }
    // with dW wanted the transposed aggregate G = A^T dY is needed in memory anyway (dW = X^T G, dX = G W^T)
    const int F = K > M ? K : M;
    char* G = (char*)ws + 256;
    char* pws = G + up256((size_t)g->N * F * 4);
    const size_t pbytes = chunked_workspace(g->E, F, false);
    gnn_status rc = run_chunked(who, MODE_SUM, g->N, g->E, g->rowptrT, g->colT, w, dY, G, nullptr, gscale, nullptr, nullptr, 0, M,
                                dtype, pws, pbytes, st);
    if (rc != GNN_OK) return rc;
    return gnn_linear_backward(X, W, G, g->N, K, M, dtype, dX, dW, pws + pbytes, gnn_linear_workspace(g->N, K, M), stream);
}

}  // extern "C"
