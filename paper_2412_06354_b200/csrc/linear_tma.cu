// Pipelined tensor-core path of the dense node-wise transform for bf16: Y[N,Mo] = X[N,Kc] * B with
// B = W[Kc,Mo] as stored (b_transposed = 0: Y = X*W) or the transpose of W[Mo,Kc] (b_transposed = 1:
// dX = dY*W^T), and dW = X^T * dY.
//
// One persistent CTA per SM, three roles:
//   warp 0   loader: one thread issues bulk tensor copies (TMA).  The weight matrix is fetched once
//            per CTA; X arrives as slices of 128 rows x 64 contraction elements (128 bytes per row,
//            128-byte swizzle, 16 KB) into a ring of shared-memory slots, each copy signalling the
//            slot's "full" mbarrier with its byte count.
//   warp 1   MMA issuer: one thread waits for a slice, issues its four tcgen05.mma (128 x Mo x 16,
//            fp32 accumulator in tensor memory) and commits them to the slot's "empty" barrier, so the
//            loader can refill the slot as soon as the tensor core has read it.  Two accumulators
//            alternate between tiles.
//   warps 2..9  epilogue: wait for a tile's accumulator, read it back (tcgen05.ld), round to bf16,
//            write 32 rows x 64 columns at a time into a swizzled staging block that one bulk tensor
//            store sends to Y (rows past N are clipped by the copy engine), and hand the accumulator back.
// The contraction is short (Kc <= 256), so the kernel is bound by reading X and writing Y; the ring
// keeps 64-100 KB of loads in flight per SM.
//
// Every wait has an iteration limit: on expiry the role raises a status word and leaves its loop, the
// other roles run into their own limits, the loader waits (bounded) for copies still in flight, and
// the CTA frees its tensor memory and returns.
#include <cuda.h>  // CUtensorMap and its enums; the encoder itself is looked up through the runtime

#include <mutex>

#include "tc_common.cuh"

namespace gnn {

constexpr int TM_EPI_WARPS = 8;
constexpr int TM_THREADS = 32 * (2 + TM_EPI_WARPS);
constexpr int TM_KB = 64;                                    // contraction elements per slice = one 128-byte swizzle row
constexpr uint32_t TM_SLICE_BYTES = TC_ROWS * TM_KB * 2;     // 16 KB
constexpr uint32_t TM_STAGING_BYTES = 32 * 128;              // per epilogue warp: 32 rows x 64 bf16 columns of Y
constexpr int TM_MAX_STAGES = 8;
constexpr size_t TM_SMEM_MAX = 225 * 1024;                   // dynamic shared memory per CTA (227 KB less the static part)
constexpr uint32_t SW128 = 2;                                // descriptor layout code of the 128-byte swizzle

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}

struct TmaParams {
    int64_t N;
    int Kc, Mo;        // contraction length, output columns
    int b_transposed;
    int w_box_rows;    // rows of one weight box (a box has at most 256 rows: taller blocks arrive as two boxes)
    int stages;        // ring slots
    int acc_stride;    // tensor-memory columns between the two accumulators
    int tmem_cols;
    int* status;
    const float* bias;  // [Mo] added to every output row, or nullptr
    int relu;           // max(y, 0) after the bias
};

__global__ void __launch_bounds__(TM_THREADS, 1)
linear_tma_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW,
                  const __grid_constant__ CUtensorMap mapY, const TmaParams P) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * TM_MAX_STAGES + 5];  // full[S], empty[S], wfull, acc_full[2], acc_empty[2]
    __shared__ uint32_t tmem_base_slot;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Kc = P.Kc, Mo = P.Mo, S = P.stages;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms are 1024-byte aligned
    const int kblocks = (Kc + TM_KB - 1) / TM_KB;
    // weight blocks: one per 64 elements of the stored matrix's contiguous dimension
    const int wblocks = P.b_transposed ? kblocks : (Mo + 63) / 64;
    const uint32_t wblock_bytes = (uint32_t)(P.b_transposed ? Mo : Kc) * 128u;
    const uint32_t w0 = base, stage0 = base + (uint32_t)wblocks * wblock_bytes;
    const uint32_t ring0 = stage0 + TM_EPI_WARPS * TM_STAGING_BYTES;
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty = [&](int s) { return bar0 + 8u * (uint32_t)(TM_MAX_STAGES + s); };
    const uint32_t wfull = bar0 + 8u * (2 * TM_MAX_STAGES);
    auto acc_full = [&](int a) { return bar0 + 8u * (uint32_t)(2 * TM_MAX_STAGES + 1 + a); };
    auto acc_empty = [&](int a) { return bar0 + 8u * (uint32_t)(2 * TM_MAX_STAGES + 3 + a); };

    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        mbar_init(wfull, 1);
        for (int a = 0; a < 2; ++a) { mbar_init(acc_full(a), 1); mbar_init(acc_empty(a), TM_EPI_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapX)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapW)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapY)) : "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)P.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    const int64_t ntiles = (P.N + TC_ROWS - 1) / TC_ROWS;
    bool failed = false;

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t keep = policy_evict_last(), stream = policy_evict_first();
            mbar_arrive_expect_tx(wfull, (uint32_t)wblocks * wblock_bytes);
            const int w_rows = P.b_transposed ? Mo : Kc;
            for (int b = 0; b < wblocks; ++b)
                for (int r0 = 0; r0 < w_rows; r0 += P.w_box_rows)  // rows are 128 bytes apart: stacked boxes lie as one taller box would
                    tma_load_2d(w0 + (uint32_t)b * wblock_bytes + (uint32_t)r0 * 128u, &mapW, b * 64, r0, wfull, keep);
            uint32_t it = 0;
            for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x)
                for (int j = 0; j < kblocks; ++j, ++it) {
                    const int s = (int)(it % (uint32_t)S);
                    const uint32_t use = it / (uint32_t)S;
                    // the slot's previous contents have been consumed (first use: passes at once)
                    if (!mbar_wait_bounded(empty(s), (use & 1u) ^ 1u)) { failed = true; break; }
                    mbar_arrive_expect_tx(full(s), TM_SLICE_BYTES);
                    tma_load_2d(ring0 + (uint32_t)s * TM_SLICE_BYTES, &mapX, j * TM_KB, (int)(t * TC_ROWS), full(s), stream);
                }
            if (failed) {
                // do not leave while copies into this CTA's shared memory may still be in flight
                const uint32_t first = it > (uint32_t)S ? it - (uint32_t)S : 0u;
                for (uint32_t i = first; i < it; ++i) mbar_wait_bounded(full((int)(i % (uint32_t)S)), (i / (uint32_t)S) & 1u);
                mbar_wait_bounded(wfull, 0);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc(Mo, P.b_transposed ? 0 : 1);
            failed = !mbar_wait_bounded(wfull, 0);
            uint32_t it = 0, lt = 0;
            for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x, ++lt) {
                const uint32_t a = lt & 1u;
                // the epilogue has drained this accumulator (first two tiles: passes at once)
                if (!mbar_wait_bounded(acc_empty((int)a), ((lt >> 1) & 1u) ^ 1u)) { failed = true; break; }
                tc_fence_after();
                const uint32_t dacc = tmem_base + a * (uint32_t)P.acc_stride;
                for (int j = 0; j < kblocks; ++j, ++it) {
                    const int s = (int)(it % (uint32_t)S);
                    if (!mbar_wait_bounded(full(s), (it / (uint32_t)S) & 1u)) { failed = true; break; }
                    tc_fence_after();
                    const uint32_t a_slice = ring0 + (uint32_t)s * TM_SLICE_BYTES;
                    const int ksteps = (Kc - j * TM_KB) >= TM_KB ? TM_KB / 16 : (Kc - j * TM_KB) / 16;
                    for (int kk = 0; kk < ksteps; ++kk) {
                        // A: rows 128 bytes apart, groups of 8 rows 1024 bytes apart; a k-step is 32 bytes along the row
                        const uint64_t adesc = make_smem_desc(a_slice + (uint32_t)kk * 32u, 16, 1024, SW128);
                        uint64_t bdesc;
                        if (P.b_transposed)  // K-major: block j holds Mo rows (output columns) of 64 contraction elements
                            bdesc = make_smem_desc(w0 + (uint32_t)j * wblock_bytes + (uint32_t)kk * 32u, 16, 1024, SW128);
                        else  // MN-major: block m holds Kc rows (contraction) of 64 output columns; blocks LBO apart
                            bdesc = make_smem_desc(w0 + (uint32_t)(j * TM_KB + kk * 16) * 128u, wblock_bytes, 1024, SW128);
                        mma_bf16_ss(dacc, adesc, bdesc, idesc, (j > 0 || kk > 0) ? 1u : 0u);
                    }
                    mma_commit(empty(s));  // slot reusable once these MMAs have read it
                }
                if (failed) break;
                mma_commit(acc_full((int)a));
            }
        }
    } else {
        const int ew = warp - 2, quarter = warp & 3, half = ew >> 2;  // tensor-memory lanes 32*(warp % 4)..: hardware rule
        const uint32_t stg = stage0 + (uint32_t)ew * TM_STAGING_BYTES;
        uint32_t lt = 0;
        for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x, ++lt) {
            const uint32_t a = lt & 1u;
            if (!mbar_wait_bounded(acc_full((int)a), (lt >> 1) & 1u)) { failed = true; break; }
            tc_fence_after();
            const int64_t row0 = t * TC_ROWS + quarter * 32;  // first of this warp's 32 rows
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + a * (uint32_t)P.acc_stride;
            for (int cb = half; cb * 64 < Mo; cb += 2) {
                // the previous bulk store has finished reading the staging block
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                __syncwarp();
                const int groups = (Mo - cb * 64 >= 64 ? 64 : Mo - cb * 64) / 16;
                for (int g = 0; g < groups; ++g) {
                    uint32_t r[16];
                    tmem_ld16(taddr + (uint32_t)(cb * 64 + g * 16), r);
                    tmem_ld_wait();
                    float f[16];
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        f[q] = __uint_as_float(r[q]);
                        if (P.bias) f[q] += __ldg(P.bias + cb * 64 + g * 16 + q);
                        if (P.relu) f[q] = fmaxf(f[q], 0.f);
                    }
                    // row = lane, 128 bytes per row; 16-byte chunk c sits at position c ^ (row % 8)
#pragma unroll
                    for (int h2 = 0; h2 < 2; ++h2) {
                        const uint4 v = Chunk<__nv_bfloat16>::pack(f + 8 * h2);
                        const uint32_t dst = stg + (uint32_t)lane * 128u + ((uint32_t)((2 * g + h2) ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0 && row0 < P.N) {  // rows past N are clipped by the copy engine
                    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                                     reinterpret_cast<uint64_t>(&mapY)),
                                 "r"(cb * 64), "r"((int)row0), "r"(stg)
                                 : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty((int)a));
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // staging block is read, rows are written
    }
    if (failed) atomicExch(P.status, 7);  // GNN_ERR_TIMEOUT
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols);
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encoder() {
    static std::once_flag once;
    static EncodeTiledFn fn = nullptr;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

// row-major bf16 matrix [rows, cols]; box = 64 columns (128 bytes, swizzled) x box_rows rows; out-of-range reads give zeros
bool tensor_map_encoder_available() { return encoder() != nullptr; }

static bool make_map_ld(CUtensorMap* m, const void* ptr, int64_t rows, int cols, int ld, int box_rows);
bool make_map(CUtensorMap* m, const void* ptr, int64_t rows, int cols, int box_rows) { return make_map_ld(m, ptr, rows, cols, cols, box_rows); }
// a block of columns of a wider matrix: rows ld elements apart
static bool make_map_ld(CUtensorMap* m, const void* ptr, int64_t rows, int cols, int ld, int box_rows) {
    EncodeTiledFn enc = encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static size_t tma_w_bytes(int Kc, int Mo, int b_transposed) {
    return b_transposed ? (size_t)((Kc + 63) / 64) * Mo * 128 : (size_t)((Mo + 63) / 64) * Kc * 128;
}

// widest block of output columns whose weights fit shared memory beside the staging blocks and two slices; the MMA
// takes at most 256 columns and two accumulators of them fill tensor memory
static int tma_column_block(int Kc, int Mo, int b_transposed) {
    int mc = Mo < 256 ? Mo : 256;
    while (mc >= 16 && tma_w_bytes(Kc, mc, b_transposed) + TM_EPI_WARPS * TM_STAGING_BYTES + 2 * TM_SLICE_BYTES + 1024 > TM_SMEM_MAX) mc -= 16;
    return mc >= 16 ? mc : 0;
}

bool linear_tma_supported(int64_t N, int Kc, int Mo, int b_transposed, gnn_dtype dtype) {
    if (dtype != GNN_BF16 || N <= 0 || N >= ((int64_t)1 << 31) - TC_ROWS) return false;
    if (Kc % 16 != 0 || Kc < 16 || Kc > 512 || Mo % 16 != 0 || Mo < 16 || Mo > 1024) return false;
    if (Kc > 256 && Kc % 32 != 0) return false;  // a weight block taller than 256 rows arrives as two boxes of Kc / 2 rows
    if (tma_column_block(Kc, Mo, b_transposed) == 0) return false;
    return encoder() != nullptr;
}

// More than 256 output columns, or weights too large for shared memory, run as one launch per block of output columns.
gnn_status linear_tma_forward(const void* X, const void* W, int64_t N, int Kc, int Mo, int b_transposed, void* Y, int* d_flag,
                              cudaStream_t st, const float* bias, int relu) {
    const char* who = "gnn_linear (pipelined tensor-core path)";
    GNN_REQUIRE(aligned16(X) && aligned16(W) && aligned16(Y), GNN_ERR_INVALID_ARG, "%s: matrices must be 16-byte aligned", who);
    const int block = tma_column_block(Kc, Mo, b_transposed);
    GNN_REQUIRE(block > 0, GNN_ERR_UNSUPPORTED, "%s: weights do not fit shared memory", who);
    CUtensorMap mapX;
    if (!make_map(&mapX, X, N, Kc, TC_ROWS)) GNN_FAIL(GNN_ERR_CUDA, "%s: tensor map encoding failed", who);
    gnn_status rc = allow_big_smem(who, (const void*)linear_tma_kernel, 4, TM_SMEM_MAX);
    if (rc != GNN_OK) return rc;
    const int64_t ntiles = (N + TC_ROWS - 1) / TC_ROWS;
    const __nv_bfloat16* Wb = (const __nv_bfloat16*)W;
    for (int c0 = 0; c0 < Mo; c0 += block) {
        const int mc = Mo - c0 < block ? Mo - c0 : block;
        // stored [Kc,Mo]: a block of columns (rows Mo apart); stored [Mo,Kc]: a block of rows
        const int w_rows = b_transposed ? mc : Kc, w_cols = b_transposed ? Kc : mc;
        const int box_rows = w_rows > 256 ? w_rows / 2 : w_rows;
        CUtensorMap mapW, mapY;
        if (!make_map_ld(&mapW, b_transposed ? Wb + (size_t)c0 * Kc : Wb + c0, w_rows, w_cols, b_transposed ? Kc : Mo, box_rows) ||
            !make_map_ld(&mapY, (const __nv_bfloat16*)Y + c0, N, mc, Mo, 32))
            GNN_FAIL(GNN_ERR_CUDA, "%s: tensor map encoding failed", who);
        TmaParams P;
        P.N = N; P.Kc = Kc; P.Mo = mc; P.b_transposed = b_transposed; P.w_box_rows = box_rows; P.status = d_flag;
        P.bias = bias ? bias + c0 : nullptr; P.relu = relu;
        const size_t wbytes = tma_w_bytes(Kc, mc, b_transposed);
        const size_t fixed = 1024 + wbytes + (size_t)TM_EPI_WARPS * TM_STAGING_BYTES;
        int stages = (int)((TM_SMEM_MAX - fixed) / TM_SLICE_BYTES);
        P.stages = stages > TM_MAX_STAGES ? TM_MAX_STAGES : stages;
        P.acc_stride = (mc + 31) & ~31;
        int cols = 32;
        while (cols < 2 * P.acc_stride) cols <<= 1;
        P.tmem_cols = cols;
        const size_t smem = fixed + (size_t)P.stages * TM_SLICE_BYTES;
        linear_tma_kernel<<<(int)(ntiles < 148 ? ntiles : 148), TM_THREADS, smem, st>>>(mapX, mapW, mapY, P);
        GNN_CHECK_LAUNCH(who);
    }
    return GNN_OK;
}

// ------------------------------------------------------------------ fp32: Y = X * B on the bf16 tensor cores
// Every fp32 value is split exactly into three bf16 terms (x = x1 + x2 + x3, 8 mantissa bits each) and the
// six products with i + j <= 4 are accumulated (the dropped ones are below 2^-23 of a product), which keeps
// the fp32 tolerance.  Roles of the persistent CTA:
//   warp 0      loader: X arrives as fp32 slices of 128 rows x 32 columns (128-byte rows, 128-byte swizzle)
//               in a ring of shared-memory slots;
//   warps 2..9  converters: read a slice, split it, and write the three bf16 levels into one of two operand
//               buffers in the tensor core's canonical no-swizzle layout (8 rows x 16 bytes per core matrix);
//   warp 1      MMA issuer: 2 k-steps x 6 level pairs per slice into one of two accumulators;
//   warps 10..17 epilogue: accumulator -> swizzled staging blocks of 32 rows x 32 columns -> bulk tensor stores to Y.
// The weight matrix is split once per CTA by all warps before the roles start.
constexpr int TF_CONV_WARPS = 8, TF_EPI_WARPS = 8;
constexpr int TF_THREADS = 32 * (2 + TF_CONV_WARPS + TF_EPI_WARPS);
constexpr int TF_KB = 32;                                  // contraction elements per slice
constexpr uint32_t TF_SLICE_BYTES = TC_ROWS * TF_KB * 4;   // 16 KB of fp32
constexpr uint32_t TF_LEVEL_BYTES = TC_ROWS * TF_KB * 2;   // 8 KB: one bf16 level of a slice
constexpr int TF_MAX_STAGES = 6;

__device__ __constant__ unsigned char kPairA3[6] = {2, 0, 1, 1, 0, 0};  // levels of A and B per product, small terms first
__device__ __constant__ unsigned char kPairB3[6] = {0, 2, 1, 0, 1, 0};

// 8 fp32 values -> three 16-byte chunks of bf16 (x = x1 + x2 + x3 exactly)
__device__ __forceinline__ void split8(const float* xin, uint4* lv) {
    float x[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) x[j] = xin[j];
#pragma unroll
    for (int l = 0; l < 3; ++l) {
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            __nv_bfloat162 b = __floats2bfloat162_rn(x[j], x[j + 1]);
            w[j / 2] = *reinterpret_cast<uint32_t*>(&b);
            // remainders are exact in fp32: the rounded term shares the leading bits of x
            x[j] -= __uint_as_float(w[j / 2] << 16);
            x[j + 1] -= __uint_as_float(w[j / 2] & 0xFFFF0000u);
        }
        lv[l] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}
__device__ __forceinline__ void st_shared16(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 ld_shared16(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

struct TmaF32Params {
    const float* W;  // [Kc,Mo] (b_transposed = 0) or [Mo,Kc] (b_transposed = 1), rows ldw elements apart
    int ldw;
    int64_t N;
    int Kc, Mo;
    int b_transposed;
    int stages;
    int acc_stride, tmem_cols;
    int* status;
    const float* bias;  // [Mo] added to every output row, or nullptr
    int relu;           // max(y, 0) after the bias
};

__global__ void __launch_bounds__(TF_THREADS, 1)
linear_tma_f32_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY, const TmaF32Params P) {
    extern __shared__ unsigned char smem_raw[];
    // f_full[S], f_empty[S], o_full[2], o_empty[2], acc_full[2], acc_empty[2]
    __shared__ __align__(8) uint64_t bars[2 * TF_MAX_STAGES + 8];
    __shared__ uint32_t tmem_base_slot;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Kc = P.Kc, Mo = P.Mo, S = P.stages;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int kchunks = Kc / 8;                    // 16-byte chunks of bf16 along the whole contraction
    const uint32_t b_sbo = (uint32_t)kchunks * 128;  // weight levels: same layout as a whole-K operand
    const uint32_t b_level = (uint32_t)Mo * Kc * 2;
    const uint32_t w0 = base, ring0 = base + ((3 * b_level + 1023u) & ~1023u), op0 = ring0 + (uint32_t)S * TF_SLICE_BYTES;
    const uint32_t stage0 = op0 + 2u * 3u * TF_LEVEL_BYTES;  // per epilogue warp: 32 rows x 32 fp32 columns of Y
    const int nslices = (Kc + TF_KB - 1) / TF_KB;
    const uint32_t bar0 = smem_u32(bars);
    auto f_full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto f_empty = [&](int s) { return bar0 + 8u * (uint32_t)(TF_MAX_STAGES + s); };
    auto o_full = [&](int o) { return bar0 + 8u * (uint32_t)(2 * TF_MAX_STAGES + o); };
    auto o_empty = [&](int o) { return bar0 + 8u * (uint32_t)(2 * TF_MAX_STAGES + 2 + o); };
    auto acc_full = [&](int a) { return bar0 + 8u * (uint32_t)(2 * TF_MAX_STAGES + 4 + a); };
    auto acc_empty = [&](int a) { return bar0 + 8u * (uint32_t)(2 * TF_MAX_STAGES + 6 + a); };

    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(f_full(s), 1); mbar_init(f_empty(s), TF_CONV_WARPS); }
        for (int o = 0; o < 2; ++o) {
            mbar_init(o_full(o), TF_CONV_WARPS); mbar_init(o_empty(o), 1);
            mbar_init(acc_full(o), 1); mbar_init(acc_empty(o), TF_EPI_WARPS);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapX)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapY)) : "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)P.tmem_cols);
    // weight levels.  16-byte chunk c of stored row r:
    //   stored [Kc,Mo] (MN-major B): r = k, c = 8 output columns: offset c*sbo + (k/8)*128 + (k%8)*16
    //   stored [Mo,Kc] (K-major  B): r = n, c = 8 k's:            offset (n/8)*sbo + c*128 + (n%8)*16
    // eight consecutive threads take the eight rows of one core matrix: contiguous 16-byte stores
    {
        const int rows = P.b_transposed ? Mo : Kc, chunks = (P.b_transposed ? Kc : Mo) / 8;
        for (int e = tid; e < rows * chunks; e += TF_THREADS) {
            const int q = e >> 3, rg = q / chunks, c = q - rg * chunks, r = rg * 8 + (e & 7);
            const float4* src = reinterpret_cast<const float4*>(P.W + (size_t)r * P.ldw + (size_t)c * 8);
            const float4 lo = __ldg(src), hi = __ldg(src + 1);
            const float x[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
            uint4 lv[3];
            split8(x, lv);
            const uint32_t off = P.b_transposed ? (uint32_t)(r >> 3) * b_sbo + (uint32_t)c * 128 + (uint32_t)(r & 7) * 16
                                                : (uint32_t)c * b_sbo + (uint32_t)(r >> 3) * 128 + (uint32_t)(r & 7) * 16;
#pragma unroll
            for (int l = 0; l < 3; ++l) st_shared16(w0 + (uint32_t)l * b_level + off, lv[l]);
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    const int64_t ntiles = (P.N + TC_ROWS - 1) / TC_ROWS;
    bool failed = false;

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t stream = policy_evict_first();
            uint32_t it = 0;
            for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x)
                for (int j = 0; j < nslices; ++j, ++it) {
                    const int s = (int)(it % (uint32_t)S);
                    if (!mbar_wait_bounded(f_empty(s), ((it / (uint32_t)S) & 1u) ^ 1u)) { failed = true; break; }
                    mbar_arrive_expect_tx(f_full(s), TF_SLICE_BYTES);
                    tma_load_2d(ring0 + (uint32_t)s * TF_SLICE_BYTES, &mapX, j * TF_KB, (int)(t * TC_ROWS), f_full(s), stream);
                }
            if (failed) {
                const uint32_t first = it > (uint32_t)S ? it - (uint32_t)S : 0u;
                for (uint32_t i = first; i < it; ++i) mbar_wait_bounded(f_full((int)(i % (uint32_t)S)), (i / (uint32_t)S) & 1u);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc(Mo, P.b_transposed ? 0 : 1);
            uint32_t it = 0, lt = 0;
            for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x, ++lt) {
                const uint32_t a = lt & 1u;
                if (!mbar_wait_bounded(acc_empty((int)a), ((lt >> 1) & 1u) ^ 1u)) { failed = true; break; }
                tc_fence_after();
                const uint32_t dacc = tmem_base + a * (uint32_t)P.acc_stride;
                for (int j = 0; j < nslices; ++j, ++it) {
                    const uint32_t o = it & 1u;
                    if (!mbar_wait_bounded(o_full((int)o), (it >> 1) & 1u)) { failed = true; break; }
                    tc_fence_after();
                    const uint32_t abuf = op0 + o * 3u * TF_LEVEL_BYTES;
                    const int ksteps = (Kc - j * TF_KB) >= TF_KB ? TF_KB / 16 : (Kc - j * TF_KB) / 16;
                    for (int kk = 0; kk < ksteps; ++kk)
                        for (int q = 0; q < 6; ++q) {
                            // A slice: 4 chunks along k, core matrices 128 bytes apart, groups of 8 rows 512 bytes apart
                            const uint64_t adesc = make_smem_desc(abuf + (uint32_t)kPairA3[q] * TF_LEVEL_BYTES + (uint32_t)kk * 256u, 128, 512);
                            const uint64_t bdesc = make_smem_desc(w0 + (uint32_t)kPairB3[q] * b_level + (uint32_t)(j * (TF_KB / 16) + kk) * 256u, 128, b_sbo);
                            mma_bf16_ss(dacc, adesc, bdesc, idesc, (j > 0 || kk > 0 || q > 0) ? 1u : 0u);
                        }
                    mma_commit(o_empty((int)o));
                }
                if (failed) break;
                mma_commit(acc_full((int)a));
            }
        }
    } else if (warp < 2 + TF_CONV_WARPS) {
        // Every converter warp works on every slice, in order: a waiter that skipped uses of a slot would
        // find the parity of an older completed phase and run ahead of the copy (parity waits only tell
        // the last two phases apart), so the slices are not divided among groups of warps.
        constexpr int GT = 32 * TF_CONV_WARPS;
        const int ct = tid - 64;
        uint32_t it = 0;
        for (int64_t t = blockIdx.x; t < ntiles && !failed; t += gridDim.x)
            for (int j = 0; j < nslices; ++j, ++it) {
                const int s = (int)(it % (uint32_t)S);
                const uint32_t o = it & 1u;
                if (!mbar_wait_bounded(f_full(s), (it / (uint32_t)S) & 1u)) { failed = true; break; }
                if (!mbar_wait_bounded(o_empty((int)o), ((it >> 1) & 1u) ^ 1u)) { failed = true; break; }
                tc_fence_after();
                const uint32_t src = ring0 + (uint32_t)s * TF_SLICE_BYTES, dst = op0 + o * 3u * TF_LEVEL_BYTES;
#pragma unroll
                for (int rep = 0; rep < (TC_ROWS * (TF_KB / 8)) / GT; ++rep) {
                    const int e = ct + rep * GT;
                    const int q = e >> 3, rg = q >> 2, kc = q & 3, r = rg * 8 + (e & 7);
                    // fp32 row r: 128 bytes, 16-byte chunk c at position c ^ (r % 8)
                    const uint4 c0 = ld_shared16(src + (uint32_t)r * 128u + (uint32_t)(((2 * kc) ^ (r & 7)) << 4));
                    const uint4 c1 = ld_shared16(src + (uint32_t)r * 128u + (uint32_t)(((2 * kc + 1) ^ (r & 7)) << 4));
                    const float x[8] = {__uint_as_float(c0.x), __uint_as_float(c0.y), __uint_as_float(c0.z), __uint_as_float(c0.w),
                                        __uint_as_float(c1.x), __uint_as_float(c1.y), __uint_as_float(c1.z), __uint_as_float(c1.w)};
                    uint4 lv[3];
                    split8(x, lv);
                    const uint32_t off = (uint32_t)(r >> 3) * 512u + (uint32_t)kc * 128u + (uint32_t)(r & 7) * 16u;
#pragma unroll
                    for (int l = 0; l < 3; ++l) st_shared16(dst + (uint32_t)l * TF_LEVEL_BYTES + off, lv[l]);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
                __syncwarp();
                if (lane == 0) { mbar_arrive(f_empty(s)); mbar_arrive(o_full((int)o)); }
            }
    } else {
        const int ew = warp - (2 + TF_CONV_WARPS), quarter = warp & 3, half = ew >> 2;
        const uint32_t stg = stage0 + (uint32_t)ew * 4096u;
        uint32_t lt = 0;
        for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x, ++lt) {
            const uint32_t a = lt & 1u;
            if (!mbar_wait_bounded(acc_full((int)a), (lt >> 1) & 1u)) { failed = true; break; }
            tc_fence_after();
            const int64_t row0 = t * TC_ROWS + quarter * 32;  // first of this warp's 32 rows
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + a * (uint32_t)P.acc_stride;
            for (int cb = half; cb * 32 < Mo; cb += 2) {  // blocks of 32 columns = 128-byte rows
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // staging block free again
                __syncwarp();
                const int groups = (Mo - cb * 32 >= 32 ? 32 : Mo - cb * 32) / 16;
                for (int g16 = 0; g16 < groups; ++g16) {
                    uint32_t r[16];
                    tmem_ld16(taddr + (uint32_t)(cb * 32 + g16 * 16), r);
                    tmem_ld_wait();
                    if (P.bias || P.relu) {
#pragma unroll
                        for (int q = 0; q < 16; ++q) {
                            float y = __uint_as_float(r[q]);
                            if (P.bias) y += __ldg(P.bias + cb * 32 + g16 * 16 + q);
                            if (P.relu) y = fmaxf(y, 0.f);
                            r[q] = __float_as_uint(y);
                        }
                    }
                    // row = lane, 128 bytes per row; 16-byte chunk c sits at position c ^ (row % 8)
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        st_shared16(stg + (uint32_t)lane * 128u + ((uint32_t)((4 * g16 + q) ^ (lane & 7)) << 4),
                                    make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]));
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0 && row0 < P.N) {  // rows past N are clipped by the copy engine
                    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                                     reinterpret_cast<uint64_t>(&mapY)),
                                 "r"(cb * 32), "r"((int)row0), "r"(stg)
                                 : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty((int)a));
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
    if (failed) atomicExch(P.status, 7);  // GNN_ERR_TIMEOUT
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols);
}

// ------------------------------------------------------------------ dW = X^T * dY
// Contraction over the N rows.  A = X^T (features x rows) and B = dY (rows x columns) are both
// MN-major as stored, so the same 64-column x 64-row swizzled boxes serve: a pipeline slot holds 64
// rows of X (K/64 boxes) and of dY (M/64 boxes).  The MMA warp issues, per slot, four k-steps of 16
// rows for each half of 128 features (MMA shape 128 x M x 16) into per-CTA accumulators that stay in
// tensor memory for the whole kernel; at the end the epilogue warps write one fp32 partial [K,M] per
// CTA, and the partials are summed in CTA order by the caller (fixed order: deterministic).
constexpr int DW_ROWS = 64;                         // rows of X / dY per slot
constexpr uint32_t DW_BOX_BYTES = DW_ROWS * 128;    // one 64 x 64 bf16 box

struct TmaDwParams {
    float* part;  // [gridDim.x][K][M]
    int64_t N;
    int K, M;
    int stages;
    int tmem_cols;
    int* status;
};

__global__ void __launch_bounds__(TM_THREADS, 1)
linear_tma_dw_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapD,
                     const __grid_constant__ CUtensorMap mapP, const TmaDwParams P) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * TM_MAX_STAGES + 1];  // full[S], empty[S], acc_full
    __shared__ uint32_t tmem_base_slot;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = P.K, M = P.M, S = P.stages;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // whole blocks of the MMA's 128 feature rows: boxes that start past column K arrive as zeros
    const int halves = (K + 127) / 128, xboxes = 2 * halves, dboxes = (M + 63) / 64;
    const uint32_t slot_bytes = (uint32_t)(xboxes + dboxes) * DW_BOX_BYTES;
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty = [&](int s) { return bar0 + 8u * (uint32_t)(TM_MAX_STAGES + s); };
    const uint32_t acc_full = bar0 + 8u * (2 * TM_MAX_STAGES);

    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        mbar_init(acc_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapX)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapD)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapP)) : "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)P.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    const int64_t nchunks = (P.N + DW_ROWS - 1) / DW_ROWS;  // gridDim.x <= nchunks: every CTA has work
    bool failed = false;

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t stream = policy_evict_first();
            uint32_t it = 0;
            for (int64_t c = blockIdx.x; c < nchunks; c += gridDim.x, ++it) {
                const int s = (int)(it % (uint32_t)S);
                if (!mbar_wait_bounded(empty(s), ((it / (uint32_t)S) & 1u) ^ 1u)) { failed = true; break; }
                mbar_arrive_expect_tx(full(s), slot_bytes);
                const uint32_t slot = base + (uint32_t)s * slot_bytes;
                for (int b = 0; b < xboxes; ++b) tma_load_2d(slot + (uint32_t)b * DW_BOX_BYTES, &mapX, b * 64, (int)(c * DW_ROWS), full(s), stream);
                for (int b = 0; b < dboxes; ++b)
                    tma_load_2d(slot + (uint32_t)(xboxes + b) * DW_BOX_BYTES, &mapD, b * 64, (int)(c * DW_ROWS), full(s), stream);
            }
            if (failed) {
                const uint32_t first = it > (uint32_t)S ? it - (uint32_t)S : 0u;
                for (uint32_t i = first; i < it; ++i) mbar_wait_bounded(full((int)(i % (uint32_t)S)), (i / (uint32_t)S) & 1u);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc(M, 1, 1);  // A and B both MN-major
            uint32_t it = 0;
            for (int64_t c = blockIdx.x; c < nchunks; c += gridDim.x, ++it) {
                const int s = (int)(it % (uint32_t)S);
                if (!mbar_wait_bounded(full(s), (it / (uint32_t)S) & 1u)) { failed = true; break; }
                tc_fence_after();
                const uint32_t sa = base + (uint32_t)s * slot_bytes, sb = sa + (uint32_t)xboxes * DW_BOX_BYTES;
                for (int h = 0; h < halves; ++h)
                    for (int kk = 0; kk < DW_ROWS / 16; ++kk) {
                        // rows (contraction) are 128 bytes apart, groups of 8 rows 1024 bytes, blocks of 64 features / columns one box
                        const uint64_t adesc = make_smem_desc(sa + (uint32_t)(2 * h) * DW_BOX_BYTES + (uint32_t)kk * 2048u, DW_BOX_BYTES, 1024, SW128);
                        const uint64_t bdesc = make_smem_desc(sb + (uint32_t)kk * 2048u, DW_BOX_BYTES, 1024, SW128);
                        mma_bf16_ss(tmem_base + (uint32_t)(h * M), adesc, bdesc, idesc, (it > 0 || kk > 0) ? 1u : 0u);
                    }
                mma_commit(empty(s));
            }
            if (!failed) mma_commit(acc_full);
        }
    } else {
        const int ew = warp - 2, quarter = warp & 3, half = ew >> 2;
        if (!mbar_wait_bounded(acc_full, 0)) {
            failed = true;
        } else {
            tc_fence_after();
            // the pipeline slots are idle now (every load was consumed before the last commit): each warp
            // stages 32 feature rows x 32 columns of fp32 there and sends them with a bulk tensor store
            const uint32_t stg = base + (uint32_t)ew * 4096u;
            for (int h = 0; h < halves; ++h) {
                if (h * 128 + quarter * 32 >= K) break;  // feature rows past K (K is a multiple of 32): the next CTA's rows of the partial matrix
                const int prow0 = (int)blockIdx.x * K + h * 128 + quarter * 32;  // row of the [parts*K, M] partial matrix
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(h * M);
                for (int cb = half; cb * 32 < M; cb += 2) {
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    __syncwarp();
                    const int groups = (M - cb * 32 >= 32 ? 32 : M - cb * 32) / 16;
                    for (int g16 = 0; g16 < groups; ++g16) {
                        uint32_t r[16];
                        tmem_ld16(taddr + (uint32_t)(cb * 32 + g16 * 16), r);
                        tmem_ld_wait();
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            st_shared16(stg + (uint32_t)lane * 128u + ((uint32_t)((4 * g16 + q) ^ (lane & 7)) << 4),
                                        make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]));
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                                         reinterpret_cast<uint64_t>(&mapP)),
                                     "r"(cb * 32), "r"(prow0), "r"(stg)
                                     : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
            }
            if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        }
    }
    if (failed) atomicExch(P.status, 7);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols);
}

bool linear_tma_dw_supported(int64_t N, int K, int M, gnn_dtype dtype) {
    if (dtype != GNN_BF16 || N <= 0 || N >= ((int64_t)1 << 31) - TC_ROWS) return false;
    if (K % 32 != 0 || K < 32 || K > 512 || M % 16 != 0 || M < 16 || M > 256) return false;
    if (M * ((K + 127) / 128) > 512) return false;  // one accumulator [128, M] per block of 128 features: 512 columns of tensor memory
    return encoder() != nullptr;
}

int linear_tma_dw_partials(int64_t N) {
    const int64_t nchunks = (N + DW_ROWS - 1) / DW_ROWS;
    return (int)(nchunks < 148 ? (nchunks > 0 ? nchunks : 1) : 148);
}

bool make_map_f32(CUtensorMap* m, const void* ptr, int64_t rows, int cols, int box_rows);

// writes linear_tma_dw_partials(N) fp32 partials [K,M] to part
gnn_status linear_tma_dw(const void* X, const void* dY, int64_t N, int K, int M, int ldd, float* part, int* d_flag, cudaStream_t st) {
    const char* who = "gnn_linear_backward (pipelined tensor-core dW)";
    GNN_REQUIRE(aligned16(X) && aligned16(dY) && aligned16(part), GNN_ERR_INVALID_ARG, "%s: matrices must be 16-byte aligned", who);
    CUtensorMap mapX, mapD, mapP;
    if (!make_map(&mapX, X, N, K, DW_ROWS) || !make_map_ld(&mapD, dY, N, M, ldd, DW_ROWS) ||  // dY may be a block of columns: rows ldd apart
        !make_map_f32(&mapP, part, (int64_t)linear_tma_dw_partials(N) * K, M, 32))
        GNN_FAIL(GNN_ERR_CUDA, "%s: tensor map encoding failed", who);
    TmaDwParams P;
    P.part = part; P.N = N; P.K = K; P.M = M; P.status = d_flag;
    const size_t slot = (size_t)(2 * ((K + 127) / 128) + (M + 63) / 64) * DW_BOX_BYTES;
    int stages = (int)((TM_SMEM_MAX - 1024) / slot);
    P.stages = stages > TM_MAX_STAGES ? TM_MAX_STAGES : stages;
    int cols = 32;
    while (cols < M * ((K + 127) / 128)) cols <<= 1;
    P.tmem_cols = cols;
    gnn_status rc = allow_big_smem(who, (const void*)linear_tma_dw_kernel, 5, TM_SMEM_MAX);
    if (rc != GNN_OK) return rc;
    linear_tma_dw_kernel<<<linear_tma_dw_partials(N), TM_THREADS, 1024 + (size_t)P.stages * slot, st>>>(mapX, mapD, mapP, P);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

// row-major fp32 matrix [rows, cols]; box = 32 columns (128 bytes, swizzled) x box_rows rows
// the same for a block of columns of a wider matrix: rows ld elements apart
static bool make_map_f32_ld(CUtensorMap* m, const void* ptr, int64_t rows, int cols, int ld, int box_rows);
bool make_map_f32(CUtensorMap* m, const void* ptr, int64_t rows, int cols, int box_rows) {
    return make_map_f32_ld(m, ptr, rows, cols, cols, box_rows);
}
static bool make_map_f32_ld(CUtensorMap* m, const void* ptr, int64_t rows, int cols, int ld, int box_rows) {
    EncodeTiledFn enc = encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
    const cuuint32_t box[2] = {32, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ------------------------------------------------------------------ fp32: dW = X^T * dY on the bf16 tensor cores, pipelined
// Contraction over the N rows, 32 rows per pipeline slot (16 where K or M is 256, so that two operand buffers and a
// ring still fit shared memory).  Roles of the persistent CTA:
//   warp 0      loader: a slot is K/32 + M/32 boxes of 32 rows x 32 fp32 columns (128-byte rows, 128-byte swizzle)
//               of X and dY, in a ring of shared-memory slots;
//   warps 2..9  converters: split every value exactly into three bf16 terms and write the levels of both operands
//               into one of two operand buffers in the canonical no-swizzle layout, MN-major (16-byte chunk c = 8
//               features or columns of row n at c*512 + (n/8)*128 + (n%8)*16);
//   warp 1      MMA issuer: 2 k-steps of 16 rows x 6 level pairs per slot, all into one accumulator [128 features x M]
//               that stays in tensor memory for the whole kernel;
//   at the end the converter warps write the accumulator as this CTA's fp32 partial [K,M]; the caller sums the
//   partials in CTA order (fixed order: deterministic).
// K a multiple of 32 up to 128 features (the MMA has 128 rows; those past K are zeros), M a multiple of 32 up to 128.
// Every wait is bounded.
constexpr int FD_ROWS_MAX = 32;
constexpr int FD_CONV_WARPS = 8;
constexpr int FD_THREADS = 32 * (2 + FD_CONV_WARPS);
constexpr int FD_MAX_STAGES = 4;

struct TmaF32DwParams {
    float* part;  // [gridDim.x][K][M]
    int64_t N;
    int K, M;
    int rows;  // rows of X / dY per slot: 32 or 16
    int stages;
    int tmem_cols;
    int* status;
};

__global__ void __launch_bounds__(FD_THREADS, 1)
linear_tma_f32_dw_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapD, const TmaF32DwParams P) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * FD_MAX_STAGES + 5];  // f_full[S], f_empty[S], o_full[2], o_empty[2], acc_full
    __shared__ uint32_t tmem_base_slot;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = P.K, M = P.M, S = P.stages, FD_ROWS = P.rows, halves = (K + 127) / 128;
    const uint32_t FD_BOX_BYTES = (uint32_t)FD_ROWS * 128u;   // one box: FD_ROWS rows x 32 fp32 columns
    const uint32_t FD_SBO = (uint32_t)(FD_ROWS / 8) * 128u;   // next chunk of 8 features / columns in an operand level
    const int xboxes = K / 32, dboxes = M / 32;
    const uint32_t slot_bytes = (uint32_t)(xboxes + dboxes) * FD_BOX_BYTES;
    // the A operand always has whole blocks of the MMA's 128 feature rows; with K < 128 the rows past K stay zero
    const uint32_t a_level = (uint32_t)halves * 128u * FD_ROWS * 2, b_level = (uint32_t)M * FD_ROWS * 2;
    const uint32_t op_bytes = 3u * (a_level + b_level);
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t ring0 = base, op0 = ring0 + (uint32_t)S * slot_bytes;
    const uint32_t bar0 = smem_u32(bars);
    auto f_full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto f_empty = [&](int s) { return bar0 + 8u * (uint32_t)(FD_MAX_STAGES + s); };
    auto o_full = [&](int o) { return bar0 + 8u * (uint32_t)(2 * FD_MAX_STAGES + o); };
    auto o_empty = [&](int o) { return bar0 + 8u * (uint32_t)(2 * FD_MAX_STAGES + 2 + o); };
    const uint32_t acc_full = bar0 + 8u * (uint32_t)(2 * FD_MAX_STAGES + 4);

    if (tid == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(f_full(s), 1); mbar_init(f_empty(s), FD_CONV_WARPS); }
        for (int o = 0; o < 2; ++o) { mbar_init(o_full(o), FD_CONV_WARPS); mbar_init(o_empty(o), 1); }
        mbar_init(acc_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapX)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&mapD)) : "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)P.tmem_cols);
    if (K % 128 != 0) {  // the converters never write the feature rows past K: zero both buffers' A levels once
        for (int o = 0; o < 2; ++o)
            for (uint32_t off = (uint32_t)tid * 16u; off < 3u * a_level; off += FD_THREADS * 16u)
                st_shared16(op0 + (uint32_t)o * op_bytes + off, make_uint4(0u, 0u, 0u, 0u));
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    const int64_t nslots = (P.N + FD_ROWS - 1) / FD_ROWS;
    bool failed = false;

    if (warp == 0) {
        // ------------------------------------------------------------ loader
        if (lane == 0) {
            const uint64_t stream = policy_evict_first();
            uint32_t it = 0;
            for (int64_t t = blockIdx.x; t < nslots; t += gridDim.x, ++it) {
                const int s = (int)(it % (uint32_t)S);
                if (!mbar_wait_bounded(f_empty(s), ((it / (uint32_t)S) & 1u) ^ 1u)) { failed = true; break; }
                mbar_arrive_expect_tx(f_full(s), slot_bytes);  // rows past N arrive as zeros and count all the same
                const uint32_t dst = ring0 + (uint32_t)s * slot_bytes;
                for (int b = 0; b < xboxes; ++b) tma_load_2d(dst + (uint32_t)b * FD_BOX_BYTES, &mapX, b * 32, (int)(t * FD_ROWS), f_full(s), stream);
                for (int b = 0; b < dboxes; ++b) tma_load_2d(dst + (uint32_t)(xboxes + b) * FD_BOX_BYTES, &mapD, b * 32, (int)(t * FD_ROWS), f_full(s), stream);
            }
            if (failed) {  // let the copies in flight land before the CTA goes away
                const uint32_t first = it > (uint32_t)S ? it - (uint32_t)S : 0u;
                for (uint32_t i = first; i < it; ++i) mbar_wait_bounded(f_full((int)(i % (uint32_t)S)), (i / (uint32_t)S) & 1u);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc(M, 1) | (1u << 15);  // A and B both MN-major
            uint32_t it = 0;
            for (int64_t t = blockIdx.x; t < nslots; t += gridDim.x, ++it) {
                const uint32_t o = it & 1u;
                if (!mbar_wait_bounded(o_full((int)o), (it >> 1) & 1u)) { failed = true; break; }
                tc_fence_after();
                const uint32_t abuf = op0 + o * op_bytes, bbuf = abuf + 3u * a_level;
                for (int h = 0; h < halves; ++h)  // features [128h, 128h + 128): chunks 16h.., accumulator columns h*M..
                    for (int kk = 0; kk < FD_ROWS / 16; ++kk)
                        for (int q = 0; q < 6; ++q) {
                            const uint64_t adesc = make_smem_desc(abuf + (uint32_t)kPairA3[q] * a_level + (uint32_t)h * 16u * FD_SBO + (uint32_t)kk * 256u, 128, FD_SBO);
                            const uint64_t bdesc = make_smem_desc(bbuf + (uint32_t)kPairB3[q] * b_level + (uint32_t)kk * 256u, 128, FD_SBO);
                            mma_bf16_ss(tmem_base + (uint32_t)h * (uint32_t)M, adesc, bdesc, idesc, (it > 0 || kk > 0 || q > 0) ? 1u : 0u);
                        }
                mma_commit(o_empty((int)o));
            }
            if (!failed) mma_commit(acc_full);
        }
    } else {
        // ------------------------------------------------------------ converters (every warp works on every slot, in order)
        constexpr int GT = 32 * FD_CONV_WARPS;
        const int ct = tid - 64;
        const int xchunks = K / 8, dchunks = M / 8;
        const int xops = FD_ROWS * xchunks, ops = xops + FD_ROWS * dchunks;
        uint32_t it = 0;
        for (int64_t t = blockIdx.x; t < nslots && !failed; t += gridDim.x, ++it) {
            const int s = (int)(it % (uint32_t)S);
            const uint32_t o = it & 1u;
            if (!mbar_wait_bounded(f_full(s), (it / (uint32_t)S) & 1u)) { failed = true; break; }
            if (!mbar_wait_bounded(o_empty((int)o), ((it >> 1) & 1u) ^ 1u)) { failed = true; break; }
            tc_fence_after();
            const uint32_t src0 = ring0 + (uint32_t)s * slot_bytes;
            const uint32_t abuf = op0 + o * op_bytes, bbuf = abuf + 3u * a_level;
#pragma unroll 4
            for (int e = ct; e < ops; e += GT) {
                // eight consecutive threads take the eight rows of one core matrix: contiguous 16-byte stores
                const bool isx = e < xops;
                const int ee = isx ? e : e - xops, chunks = isx ? xchunks : dchunks;
                const int q = ee >> 3, rg = q / chunks, c8 = q - rg * chunks, r = rg * 8 + (ee & 7);
                const int bx = (isx ? 0 : xboxes) + (c8 >> 2), kc = c8 & 3;
                // fp32 row r of the box: 128 bytes, 16-byte chunk c at position c ^ (r % 8)
                const uint32_t rowa = src0 + (uint32_t)bx * FD_BOX_BYTES + (uint32_t)r * 128u;
                const uint4 c0 = ld_shared16(rowa + (uint32_t)(((2 * kc) ^ (r & 7)) << 4));
                const uint4 c1 = ld_shared16(rowa + (uint32_t)(((2 * kc + 1) ^ (r & 7)) << 4));
                const float x[8] = {__uint_as_float(c0.x), __uint_as_float(c0.y), __uint_as_float(c0.z), __uint_as_float(c0.w),
                                    __uint_as_float(c1.x), __uint_as_float(c1.y), __uint_as_float(c1.z), __uint_as_float(c1.w)};
                uint4 lv[3];
                split8(x, lv);
                const uint32_t level = isx ? a_level : b_level;
                const uint32_t dst = (isx ? abuf : bbuf) + (uint32_t)c8 * FD_SBO + (uint32_t)(r >> 3) * 128u + (uint32_t)(r & 7) * 16u;
#pragma unroll
                for (int l = 0; l < 3; ++l) st_shared16(dst + (uint32_t)l * level, lv[l]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
            __syncwarp();
            if (lane == 0) { mbar_arrive(f_empty(s)); mbar_arrive(o_full((int)o)); }
        }
        // accumulator -> this CTA's partial.  Lane = feature row; warps 2..5 take the lower half of the columns, 6..9 the upper
        if (!failed && !mbar_wait_bounded(acc_full, 0u)) failed = true;
        tc_fence_after();
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        for (int h = 0; h < halves && !failed; ++h) {
            const int krow = h * 128 + quarter * 32 + lane;
            if (h * 128 + quarter * 32 >= K) break;  // tcgen05.ld is warp-wide: a warp whose 32 feature rows all lie past K skips it as one
            float* prow = P.part + ((size_t)blockIdx.x * K + krow) * M;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)h * (uint32_t)M;
            for (int c0 = half * (M / 2); c0 < (half + 1) * (M / 2); c0 += 16) {
                uint32_t r[16];
                tmem_ld16(taddr + (uint32_t)c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (krow < K)
                        *reinterpret_cast<float4*>(prow + c0 + 4 * q) = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]),
                                                                                   __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
            }
        }
    }
    if (failed) atomicExch(P.status, 7);  // GNN_ERR_TIMEOUT
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols);
}

bool linear_tma_f32_dw_supported(int64_t N, int K, int M, gnn_dtype dtype) {
    if (dtype != GNN_F32 || N <= 0 || N >= ((int64_t)1 << 31) - FD_ROWS_MAX) return false;
    if (K % 32 != 0 || K < 32 || K > 512 || M % 32 != 0 || M < 32 || M > 256) return false;
    if (M * ((K + 127) / 128) > 512) return false;  // one accumulator [128, M] per block of 128 features: 512 columns of tensor memory
    return encoder() != nullptr;
}

// every CTA has at least one slot, so every partial is written
static int fd_rows(int K, int M) { return (K > 128 || M > 128) ? 16 : 32; }
int linear_tma_f32_dw_partials(int64_t N) {
    const int64_t nslots = (N + FD_ROWS_MAX - 1) / FD_ROWS_MAX;  // never more CTAs than slots, whichever the slot height
    return (int)(nslots < 148 ? (nslots > 0 ? nslots : 1) : 148);
}

// writes linear_tma_f32_dw_partials(N) fp32 partials [K,M] to part
gnn_status linear_tma_f32_dw(const void* X, const void* dY, int64_t N, int K, int M, int ldd, float* part, int* d_flag, cudaStream_t st) {
    const char* who = "gnn_linear_backward (pipelined fp32 tensor-core dW)";
    GNN_REQUIRE(aligned16(X) && aligned16(dY) && aligned16(part), GNN_ERR_INVALID_ARG, "%s: matrices must be 16-byte aligned", who);
    CUtensorMap mapX, mapD;
    const int R = fd_rows(K, M), ka = (K + 127) / 128 * 128;
    if (!make_map_f32(&mapX, X, N, K, R) || !make_map_f32_ld(&mapD, dY, N, M, ldd, R)) GNN_FAIL(GNN_ERR_CUDA, "%s: tensor map encoding failed", who);
    TmaF32DwParams P;
    P.part = part; P.N = N; P.K = K; P.M = M; P.status = d_flag; P.rows = R;
    const size_t slot = (size_t)(K / 32 + M / 32) * R * 128, ops = 2 * 3 * ((size_t)ka * R * 2 + (size_t)M * R * 2);
    int stages = (int)((TM_SMEM_MAX - 1024 - ops) / slot);
    P.stages = stages > FD_MAX_STAGES ? FD_MAX_STAGES : stages;
    int cols = 32;
    while (cols < M * (ka / 128)) cols <<= 1;
    P.tmem_cols = cols;
    gnn_status rc = allow_big_smem(who, (const void*)linear_tma_f32_dw_kernel, 12, TM_SMEM_MAX);
    if (rc != GNN_OK) return rc;
    linear_tma_f32_dw_kernel<<<linear_tma_f32_dw_partials(N), FD_THREADS, 1024 + ops + (size_t)P.stages * slot, st>>>(mapX, mapD, P);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

static size_t tf_fixed_bytes(int Kc, int Mo) {
    return 1024 + (((size_t)3 * Mo * Kc * 2 + 1023) & ~(size_t)1023) + 2 * 3 * (size_t)TF_LEVEL_BYTES + (size_t)TF_EPI_WARPS * 4096;
}

// widest block of output columns (a multiple of 16) whose three weight levels fit shared memory beside two slices
static int tf_column_block(int Kc, int Mo) {
    int mc = Mo < 256 ? Mo : 256;  // the MMA takes at most 256 columns, two accumulators of them fill tensor memory
    while (mc >= 16 && tf_fixed_bytes(Kc, mc) + 2 * TF_SLICE_BYTES > TM_SMEM_MAX) mc -= 16;
    return mc >= 16 ? mc : 0;
}

bool linear_tma_f32_supported(int64_t N, int Kc, int Mo, gnn_dtype dtype) {
    if (dtype != GNN_F32 || N <= 0 || N >= ((int64_t)1 << 31) - TC_ROWS) return false;
    if (Kc % 16 != 0 || Kc < 16 || Kc > 512 || Mo % 16 != 0 || Mo < 16 || Mo > 1024) return false;
    if (tf_column_block(Kc, Mo) == 0) return false;
    return encoder() != nullptr;
}

// Weights too large for shared memory in one piece (3 x Kc x Mo x 2 bytes: 256 x 256, 256 x 128, 192 x 192 ...) run as
// one launch per block of output columns: X is read once per block, which is still an order of magnitude faster than
// the FFMA kernel these shapes fell to before.
gnn_status linear_tma_f32_forward(const void* X, const void* W, int64_t N, int Kc, int Mo, int b_transposed, void* Y, int* d_flag,
                                  cudaStream_t st, const float* bias, int relu) {
    const char* who = "gnn_linear (pipelined fp32 tensor-core path)";
    GNN_REQUIRE(aligned16(X) && aligned16(W) && aligned16(Y), GNN_ERR_INVALID_ARG, "%s: matrices must be 16-byte aligned", who);
    const int block = tf_column_block(Kc, Mo);
    GNN_REQUIRE(block > 0, GNN_ERR_UNSUPPORTED, "%s: weights do not fit shared memory", who);
    CUtensorMap mapX;
    if (!make_map_f32(&mapX, X, N, Kc, TC_ROWS)) GNN_FAIL(GNN_ERR_CUDA, "%s: tensor map encoding failed", who);
    gnn_status rc = allow_big_smem(who, (const void*)linear_tma_f32_kernel, 6, TM_SMEM_MAX);
    if (rc != GNN_OK) return rc;
    const int64_t ntiles = (N + TC_ROWS - 1) / TC_ROWS;
    for (int c0 = 0; c0 < Mo; c0 += block) {
        const int mc = Mo - c0 < block ? Mo - c0 : block;
        CUtensorMap mapY;
        if (!make_map_f32_ld(&mapY, (const float*)Y + c0, N, mc, Mo, 32)) GNN_FAIL(GNN_ERR_CUDA, "%s: tensor map encoding failed", who);
        TmaF32Params P;
        // stored [Kc,Mo]: a block of columns starts c0 elements into every row; stored [Mo,Kc]: a block of rows
        P.W = b_transposed ? (const float*)W + (size_t)c0 * Kc : (const float*)W + c0;
        P.ldw = b_transposed ? Kc : Mo;
        P.N = N; P.Kc = Kc; P.Mo = mc; P.b_transposed = b_transposed; P.status = d_flag; P.bias = bias ? bias + c0 : nullptr; P.relu = relu;
        const size_t fixed = tf_fixed_bytes(Kc, mc);
        int stages = (int)((TM_SMEM_MAX - fixed) / TF_SLICE_BYTES);
        P.stages = stages > TF_MAX_STAGES ? TF_MAX_STAGES : stages;
        P.acc_stride = (mc + 31) & ~31;
        int cols = 32;
        while (cols < 2 * P.acc_stride) cols <<= 1;
        P.tmem_cols = cols;
        linear_tma_f32_kernel<<<(int)(ntiles < 148 ? ntiles : 148), TF_THREADS, fixed + (size_t)P.stages * TF_SLICE_BYTES, st>>>(mapX, mapY, P);
        GNN_CHECK_LAUNCH(who);
    }
    return GNN_OK;
}

}  // namespace gnn
