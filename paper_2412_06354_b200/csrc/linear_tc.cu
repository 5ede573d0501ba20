// Single-buffered tensor-core kernels of the dense node-wise transform (the pipelined ones are in
// linear_tma.cu; these serve fp32 dW, fp32 weights too large for the pipeline, and bf16 when no
// tensor-map encoder is available): Y[N,M] = X[N,K] * B, bf16 operands, fp32
// accumulation in tensor memory (tcgen05.mma, sm_100a).  fp32 inputs run on the same bf16 MMAs:
// every value is split exactly into three bf16 terms (x = x1 + x2 + x3, 8 mantissa bits each) while
// the tile is copied to shared memory, and the six products with i + j <= 4 are accumulated
// (the dropped ones are below 2^-23 of the product), which keeps the fp32 tolerance.  B is either W[K,M] as stored (columns
// contiguous: "MN-major") or the transpose of a matrix stored [M,K] (dX = dY * W^T: "K-major").
//
// One persistent CTA per SM.  The weight matrix is written once per CTA into shared memory in the
// tensor core's canonical no-swizzle layout (8x16-byte core matrices); then, per tile of 128 rows:
// the X tile is copied into the same kind of layout, one thread issues K/16 MMAs of shape
// 128 x M x 16 into a 128-lane x M-column fp32 accumulator in tensor memory, the completion is
// signalled on an mbarrier by tcgen05.commit, and four warps read the accumulator back
// (tcgen05.ld), round to bf16 and store their rows.  The contraction is short (K <= 256), so the
// kernel is bound by reading X and writing Y; the layout copies are 16-byte cp.async transfers (global to shared without registers).
//
// Every wait has an iteration limit: on expiry the CTA raises a status word, skips its stores,
// still frees its tensor memory and returns.
#include "tc_common.cuh"

namespace gnn {

constexpr int TC_THREADS = 256;   // 8 warps: warp w reads accumulator lanes 32*(w%4).. and column half w/4
constexpr int TC_THREADS2 = 256;  // dW kernel, same split

// ------------------------------------------------------------------ operand tiles
// NS = number of bf16 terms per input value (1 for bf16 input, 3 for fp32 input).  A tile holds
// NS copies ("levels") of the same layout, `level_bytes` apart.
template <typename TIn> struct Operand;
template <> struct Operand<__nv_bfloat16> {
    static constexpr int NS = 1;
    // 8 consecutive input elements (16 bytes) -> one 16-byte shared-memory chunk
    __device__ __forceinline__ static void copy8(uint32_t dst, uint32_t, const __nv_bfloat16* src, bool in) {
        cp_async16(dst, src, in ? 16u : 0u);  // src stays a valid address even when nothing is read
    }
};
template <> struct Operand<float> {
    static constexpr int NS = 3;
    __device__ __forceinline__ static uint32_t pack_bf16(float lo, float hi) {
        __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&b);
    }
    // 8 consecutive fp32 values (32 bytes) -> three 16-byte chunks, one per level: x = x1 + x2 + x3
    __device__ __forceinline__ static void copy8(uint32_t dst, uint32_t level_bytes, const float* src, bool in) {
        float x[8];
        if (in) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(src)), b = __ldg(reinterpret_cast<const float4*>(src) + 1);
            x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) x[j] = 0.f;
        }
#pragma unroll
        for (int l = 0; l < 3; ++l) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                w[j / 2] = pack_bf16(x[j], x[j + 1]);
                // remainders are exact in fp32: the rounded term shares the leading bits of x
                x[j] -= __uint_as_float(w[j / 2] << 16);
                x[j + 1] -= __uint_as_float(w[j / 2] & 0xFFFF0000u);
            }
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)l * level_bytes), "r"(w[0]), "r"(w[1]),
                         "r"(w[2]), "r"(w[3]) : "memory");
        }
    }
};

// Which 16-byte chunk (row r, chunk c) of a rows x chunks matrix thread-iteration e copies.  Register copies
// (fp32 input, NS = 3) let eight consecutive threads take the eight rows of one core matrix, so their
// 16-byte shared-memory stores are contiguous (no bank conflicts) while each still reads a full 32-byte
// sector; cp.async copies (bf16) keep consecutive threads on consecutive chunks of a row.
template <int NS>
__device__ __forceinline__ void tile_coord(int e, int chunks, int* r, int* c) {
    if (NS == 3) {
        const int q = e >> 3;
        const int rg = q / chunks;
        *c = q - rg * chunks;
        *r = rg * 8 + (e & 7);
    } else {
        *r = e / chunks;
        *c = e - *r * chunks;
    }
}

// products accumulated per k-step: levels (i of A, j of B), small terms first
template <int NS> __device__ __forceinline__ int num_pairs() { return NS == 1 ? 1 : 6; }
__device__ __constant__ unsigned char kPairA[6] = {2, 0, 1, 1, 0, 0};
__device__ __constant__ unsigned char kPairB[6] = {0, 2, 1, 0, 1, 0};

template <typename TOut> __device__ __forceinline__ void store16(TOut* dst, const float* f);
template <> __device__ __forceinline__ void store16<__nv_bfloat16>(__nv_bfloat16* dst, const float* f) {
    st_stream16(reinterpret_cast<uint4*>(dst), Chunk<__nv_bfloat16>::pack(f));
    st_stream16(reinterpret_cast<uint4*>(dst) + 1, Chunk<__nv_bfloat16>::pack(f + 8));
}
template <> __device__ __forceinline__ void store16<float>(float* dst, const float* f) {
#pragma unroll
    for (int q = 0; q < 4; ++q) st_stream16(reinterpret_cast<uint4*>(dst) + q, Chunk<float>::pack(f + 4 * q));
}

template <typename T>
struct TcParams {
    const T* X;  // [N,K]
    const T* W;  // [K,M] (b_transposed = 0) or [M,K] (b_transposed = 1)
    T* Y;        // [N,M]
    int64_t N;
    int K, M;
    int b_transposed;
    int tmem_cols;
    int* status;
};

template <typename T>
__global__ void __launch_bounds__(TC_THREADS, 1)
linear_tc_kernel(const TcParams<T> P) {
    using Op = Operand<T>;
    constexpr int NS = Op::NS;
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ __align__(8) uint64_t mbar;
    __shared__ uint32_t tmem_base_slot;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = P.K, M = P.M;
    const int kchunks = K / 8;                       // 16-byte chunks along the contraction
    const uint32_t sbo = (uint32_t)kchunks * 128;    // next group of 8 rows / 8 columns
    const uint32_t b_level = (uint32_t)M * K * 2, a_level = (uint32_t)TC_ROWS * K * 2;
    const uint32_t b0 = smem_u32(smem), a0 = b0 + NS * b_level;

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)P.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&mbar)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // weight matrix -> canonical layout.  16-byte chunk c of the stored matrix row r:
    //   stored [K,M] (MN-major B): row r = k, chunk = 8 output columns n8: offset n8*sbo + (k/8)*128 + (k%8)*16
    //   stored [M,K] (K-major  B): row r = n, chunk = 8 k's kc:            offset (n/8)*sbo + kc*128 + (n%8)*16
    {
        const int rows = P.b_transposed ? M : K, chunks = (P.b_transposed ? K : M) / 8;
#pragma unroll 4
        for (int e = tid; e < rows * chunks; e += TC_THREADS) {
            int r, c;
            tile_coord<NS>(e, chunks, &r, &c);
            const uint32_t off = P.b_transposed ? (uint32_t)(r >> 3) * sbo + (uint32_t)c * 128 + (uint32_t)(r & 7) * 16
                                                : (uint32_t)c * sbo + (uint32_t)(r >> 3) * 128 + (uint32_t)(r & 7) * 16;
            Op::copy8(b0 + off, b_level, P.W + ((size_t)r * chunks + c) * 8, true);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t idesc = make_idesc(M, P.b_transposed ? 0 : 1);
    const uint32_t bar = smem_u32(&mbar);
    const int64_t ntiles = (P.N + TC_ROWS - 1) / TC_ROWS;
    uint32_t parity = 0;
    bool failed = false;

    for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const int64_t row0 = t * TC_ROWS;
        // X tile -> canonical K-major layout: chunk kc of row r at (r/8)*sbo + kc*128 + (r%8)*16
#pragma unroll 4
        for (int e = tid; e < TC_ROWS * kchunks; e += TC_THREADS) {
            int r, kc;
            tile_coord<NS>(e, kchunks, &r, &kc);
            const bool in = row0 + r < P.N;
            Op::copy8(a0 + (uint32_t)(r >> 3) * sbo + (uint32_t)kc * 128 + (uint32_t)(r & 7) * 16, a_level,
                      P.X + (in ? ((size_t)(row0 + r) * kchunks + kc) * 8 : 0), in);
        }
        cp_async_wait_all();
        // generic-proxy writes to shared memory -> visible to the tensor core (async proxy)
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (tid == 0) {
            for (int kk = 0; kk < K / 16; ++kk)
                for (int q = 0; q < num_pairs<NS>(); ++q) {
                    const uint32_t la = NS == 1 ? 0 : kPairA[q], lb = NS == 1 ? 0 : kPairB[q];
                    const uint64_t adesc = make_smem_desc(a0 + la * a_level + (uint32_t)kk * 256, 128, sbo);
                    const uint64_t bdesc = make_smem_desc(b0 + lb * b_level + (uint32_t)kk * 256, 128, sbo);
                    mma_bf16_ss(tmem_base, adesc, bdesc, idesc, (kk > 0 || q > 0) ? 1u : 0u);
                }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
        }
        const bool ok = mbar_wait_bounded(bar, parity);
        parity ^= 1;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (!ok) {
            failed = true;
        } else {
            // accumulator row = tensor-memory lane; this thread's row and its half of the columns:
            const int lane_block = warp & 3, col_half = warp >> 2;
            const int64_t row = row0 + lane_block * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(lane_block * 32) << 16);
            for (int c0 = col_half * 16; c0 < M; c0 += 32) {
                uint32_t r[16];
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
                    : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                      "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                    : "r"(taddr + (uint32_t)c0));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (row < P.N) {
                    float f[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) f[j] = __uint_as_float(r[j]);
                    store16<T>(P.Y + (size_t)row * M + c0, f);
                }
            }
        }
        // all reads of the accumulator and of the X tile are done before the next tile overwrites them
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (failed) break;  // uniform: every thread waited on the same barrier phase
    }
    if (failed && tid == 0) atomicExch(P.status, 7);  // GNN_ERR_TIMEOUT
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)P.tmem_cols) : "memory");
}

static size_t fwd_smem(int K, int M, gnn_dtype dtype) {
    return ((size_t)M * K * 2 + (size_t)TC_ROWS * K * 2) * (dtype == GNN_F32 ? 3 : 1);
}

bool linear_tc_supported(int64_t N, int K, int M, gnn_dtype dtype) {
    if (N <= 0) return false;
    if (K % 16 != 0 || K < 16 || K > 256) return false;
    if (M % 16 != 0 || M < 16 || M > 256) return false;
    return fwd_smem(K, M, dtype) <= TC_SMEM_LIMIT - 2048;
}

template <typename T>
static gnn_status launch_fwd(const char* who, const void* X, const void* W, int64_t N, int K, int M, int w_transposed,
                             void* Y, int* d_flag, size_t smem, int which, cudaStream_t st) {
    TcParams<T> P;
    P.X = (const T*)X; P.W = (const T*)W; P.Y = (T*)Y;
    P.N = N; P.K = K; P.M = M; P.b_transposed = w_transposed; P.status = d_flag;
    int cols = 32;
    while (cols < M) cols <<= 1;
    P.tmem_cols = cols;
    gnn_status rc = allow_big_smem(who, (const void*)linear_tc_kernel<T>, which);
    if (rc != GNN_OK) return rc;
    const int64_t ntiles = (N + TC_ROWS - 1) / TC_ROWS;
    // several CTAs per SM when shared and tensor memory allow: one loads while another computes
    int per_sm = (int)(TC_SMEM_LIMIT / (smem + 1024));
    if (per_sm > 512 / cols) per_sm = 512 / cols;
    per_sm = per_sm < 1 ? 1 : (per_sm > 3 ? 3 : per_sm);
    const int64_t slots = (int64_t)148 * per_sm;
    linear_tc_kernel<T><<<(int)(ntiles < slots ? ntiles : slots), TC_THREADS, smem, st>>>(P);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

gnn_status linear_tc_forward(const void* X, const void* W, int64_t N, int K, int M, int w_transposed, gnn_dtype dtype,
                             void* Y, int* d_flag, cudaStream_t st) {
    const char* who = "gnn_linear (tensor-core path)";
    GNN_REQUIRE(aligned16(X) && aligned16(W) && aligned16(Y), GNN_ERR_INVALID_ARG, "%s: matrices must be 16-byte aligned", who);
    const size_t smem = fwd_smem(K, M, dtype);
    if (dtype == GNN_F32) return launch_fwd<float>(who, X, W, N, K, M, w_transposed, Y, d_flag, smem, 0, st);
    return launch_fwd<__nv_bfloat16>(who, X, W, N, K, M, w_transposed, Y, d_flag, smem, 1, st);
}

// ------------------------------------------------------------------ dW = X^T * dY on tcgen05
// Contraction over the N rows.  A = X^T (features x rows) and B = dY (rows x columns) are both
// "MN-major" as stored: 16-byte chunk c of row n goes to c*sbo + (n/8)*128 + (n%8)*16 with
// sbo = (128/8)*128.  MMA shape 128 x M x 16 (K = 256 uses two accumulators of 128 feature rows).
// Each CTA accumulates its row tiles (t = blockIdx.x, +gridDim.x, ...) in tensor memory and writes
// one fp32 partial [K,M]; the partials are summed in CTA order by slab_sum_kernel.
template <typename T>
struct TcDwParams {
    const T* X;   // [N,K]
    const T* dY;  // [N,M]
    float* part;  // [gridDim.x][K][M]
    int64_t N;
    int K, M;
    int tmem_cols;
    int* status;
};

template <typename T>
__global__ void __launch_bounds__(TC_THREADS2, 1)
linear_tc_dw_kernel(const TcDwParams<T> P) {
    using Op = Operand<T>;
    constexpr int NS = Op::NS;
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ __align__(8) uint64_t mbar;
    __shared__ uint32_t tmem_base_slot;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = P.K, M = P.M;
    const int kc = K / 8, mc = M / 8;              // 16-byte chunks per row of X / dY
    constexpr uint32_t sbo = (TC_ROWS / 8) * 128;  // 2048: next chunk of 8 features / columns
    const uint32_t a_level = (uint32_t)K * TC_ROWS * 2, b_level = (uint32_t)M * TC_ROWS * 2;
    const uint32_t sa0 = smem_u32(smem), sb0 = sa0 + NS * a_level;
    const int halves = K / 128;

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)P.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&mbar)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t idesc = make_idesc(M, 1) | (1u << 15);  // A and B both MN-major
    const uint32_t bar = smem_u32(&mbar);
    const int64_t ntiles = (P.N + TC_ROWS - 1) / TC_ROWS;
    uint32_t parity = 0;
    bool failed = false, first = true;

    for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const int64_t row0 = t * TC_ROWS;
#pragma unroll 4
        for (int e = tid; e < TC_ROWS * kc; e += TC_THREADS2) {
            int r, c;
            tile_coord<NS>(e, kc, &r, &c);
            const bool in = row0 + r < P.N;
            Op::copy8(sa0 + (uint32_t)c * sbo + (uint32_t)(r >> 3) * 128 + (uint32_t)(r & 7) * 16, a_level,
                      P.X + (in ? ((size_t)(row0 + r) * kc + c) * 8 : 0), in);
        }
#pragma unroll 4
        for (int e = tid; e < TC_ROWS * mc; e += TC_THREADS2) {
            int r, c;
            tile_coord<NS>(e, mc, &r, &c);
            const bool in = row0 + r < P.N;
            Op::copy8(sb0 + (uint32_t)c * sbo + (uint32_t)(r >> 3) * 128 + (uint32_t)(r & 7) * 16, b_level,
                      P.dY + (in ? ((size_t)(row0 + r) * mc + c) * 8 : 0), in);
        }
        cp_async_wait_all();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (tid == 0) {
            for (int h = 0; h < halves; ++h)
                for (int kk = 0; kk < TC_ROWS / 16; ++kk)
                    for (int q = 0; q < num_pairs<NS>(); ++q) {
                        const uint32_t la = NS == 1 ? 0 : kPairA[q], lb = NS == 1 ? 0 : kPairB[q];
                        // A: features [128h, 128h+128) = chunks 16h.., rows 16kk.. = row groups 2kk, 2kk+1
                        const uint64_t adesc = make_smem_desc(sa0 + la * a_level + (uint32_t)h * 16 * sbo + (uint32_t)kk * 256, 128, sbo);
                        const uint64_t bdesc = make_smem_desc(sb0 + lb * b_level + (uint32_t)kk * 256, 128, sbo);
                        mma_bf16_ss(tmem_base + (uint32_t)h * (uint32_t)M, adesc, bdesc, idesc, (first && kk == 0 && q == 0) ? 0u : 1u);
                    }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
        }
        first = false;
        // the shared-memory tiles may be overwritten only after the MMAs that read them have completed
        const bool ok = mbar_wait_bounded(bar, parity);
        parity ^= 1;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (!ok) failed = true;
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (failed) break;
    }
    // accumulator -> this CTA's partial.  Lane = feature row within the half; warps 4..7 take the
    // upper half of the columns.
    float* part = P.part + (size_t)blockIdx.x * K * M;
    if (!failed) {
        const int lane_block = warp & 3, col_half = warp >> 2;
        const int cbeg = col_half * (M / 2), cend = cbeg + M / 2;
        for (int h = 0; h < halves; ++h) {
            const int krow = h * 128 + lane_block * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(lane_block * 32) << 16) + (uint32_t)h * (uint32_t)M;
            for (int c0 = cbeg; c0 < cend; c0 += 8) {
                uint32_t r[8];
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n"
                             : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                             : "r"(taddr + (uint32_t)c0));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                float4* dst = reinterpret_cast<float4*>(part + (size_t)krow * M + c0);
                dst[0] = make_float4(__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2]), __uint_as_float(r[3]));
                dst[1] = make_float4(__uint_as_float(r[4]), __uint_as_float(r[5]), __uint_as_float(r[6]), __uint_as_float(r[7]));
            }
        }
    }
    if (failed && tid == 0) atomicExch(P.status, 7);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)P.tmem_cols) : "memory");
}

static size_t dw_smem(int K, int M, gnn_dtype dtype) {
    return ((size_t)TC_ROWS * K * 2 + (size_t)TC_ROWS * M * 2) * (dtype == GNN_F32 ? 3 : 1);
}

bool linear_tc_dw_supported(int64_t N, int K, int M, gnn_dtype dtype) {
    if (N <= 0) return false;
    if (K != 128 && K != 256) return false;
    if (M % 16 != 0 || M < 16 || M > 256) return false;
    return dw_smem(K, M, dtype) <= TC_SMEM_LIMIT - 2048;
}

// every CTA has at least one tile, so every partial is written
int linear_tc_dw_partials(int64_t N) {
    const int64_t ntiles = (N + TC_ROWS - 1) / TC_ROWS;
    return (int)(ntiles < 148 ? (ntiles > 0 ? ntiles : 1) : 148);
}

template <typename T>
static gnn_status launch_dw(const char* who, const void* X, const void* dY, int64_t N, int K, int M, float* part, int* d_flag,
                            size_t smem, int which, cudaStream_t st) {
    TcDwParams<T> P;
    P.X = (const T*)X; P.dY = (const T*)dY; P.part = part; P.N = N; P.K = K; P.M = M; P.status = d_flag;
    int cols = 32;
    while (cols < M * (K / 128)) cols <<= 1;
    P.tmem_cols = cols;
    gnn_status rc = allow_big_smem(who, (const void*)linear_tc_dw_kernel<T>, which);
    if (rc != GNN_OK) return rc;
    linear_tc_dw_kernel<T><<<linear_tc_dw_partials(N), TC_THREADS2, smem, st>>>(P);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

// writes linear_tc_dw_partials(N) fp32 partials [K,M] to part
gnn_status linear_tc_dw(const void* X, const void* dY, int64_t N, int K, int M, gnn_dtype dtype, float* part, int* d_flag,
                        cudaStream_t st) {
    const char* who = "gnn_linear_backward (tensor-core dW)";
    GNN_REQUIRE(aligned16(X) && aligned16(dY) && aligned16(part), GNN_ERR_INVALID_ARG, "%s: matrices must be 16-byte aligned", who);
    const size_t smem = dw_smem(K, M, dtype);
    if (dtype == GNN_F32) return launch_dw<float>(who, X, dY, N, K, M, part, d_flag, smem, 2, st);
    return launch_dw<__nv_bfloat16>(who, X, dY, N, K, M, part, d_flag, smem, 3, st);
}

}  // namespace gnn
