// Tensor-core path of the dense node-wise transform: Y[N,M] = X[N,K] * B, bf16 operands, fp32
// accumulation in tensor memory (tcgen05.mma, sm_100a).  B is either W[K,M] as stored (columns
// contiguous: "MN-major") or the transpose of a matrix stored [M,K] (dX = dY * W^T: "K-major").
//
// One persistent CTA per SM.  The weight matrix is written once per CTA into shared memory in the
// tensor core's canonical no-swizzle layout (8x16-byte core matrices); then, per tile of 128 rows:
// the X tile is copied into the same kind of layout, one thread issues K/16 MMAs of shape
// 128 x M x 16 into a 128-lane x M-column fp32 accumulator in tensor memory, the completion is
// signalled on an mbarrier by tcgen05.commit, and four warps read the accumulator back
// (tcgen05.ld), round to bf16 and store their rows.  The contraction is short (K <= 256), so the
// kernel is bound by reading X and writing Y; the layout copies are plain 16-byte loads/stores.
//
// Every wait has an iteration limit: on expiry the CTA raises a status word, skips its stores,
// still frees its tensor memory and returns.
#include "common.cuh"

namespace gnn {

constexpr int TC_ROWS = 128;     // rows of X per tile = MMA M
constexpr int TC_THREADS = 128;  // 4 warps: warp w owns accumulator lanes 32w..32w+31
constexpr uint32_t TC_WAIT_LIMIT = 1u << 20;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// shared-memory matrix descriptor, no swizzle: start address, leading/stride byte offsets (all >> 4)
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version for sm_100
    return d;                // base offset 0, layout type 0 (no swizzle)
}

// instruction descriptor for kind::f16: D = f32, A = B = bf16, A K-major, M = 128
__host__ __device__ constexpr uint32_t make_idesc(int n, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(b_mn_major ? 1 : 0) << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(TC_ROWS >> 4) << 24);
}

__device__ __forceinline__ void mma_bf16_ss(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t"
        "}\n"
        :
        : "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < TC_WAIT_LIMIT; ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}\n"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}

struct TcParams {
    const __nv_bfloat16* X;  // [N,K]
    const __nv_bfloat16* W;  // [K,M] (b_transposed = 0) or [M,K] (b_transposed = 1)
    __nv_bfloat16* Y;        // [N,M]
    int64_t N;
    int K, M;
    int b_transposed;
    int tmem_cols;
    int* status;
};

__global__ void __launch_bounds__(TC_THREADS, 1)
linear_tc_kernel(const TcParams P) {
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ __align__(8) uint64_t mbar;
    __shared__ uint32_t tmem_base_slot;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = P.K, M = P.M;
    const int kchunks = K / 8;                       // 16-byte chunks along the contraction
    const uint32_t sbo = (uint32_t)kchunks * 128;    // next group of 8 rows / 8 columns
    unsigned char* sB = smem;                        // M x K bf16
    unsigned char* sA = smem + (size_t)M * K * 2;    // 128 x K bf16

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
        const uint4* src = reinterpret_cast<const uint4*>(P.W);
        for (int e = tid; e < rows * chunks; e += TC_THREADS) {
            const int r = e / chunks, c = e - r * chunks;
            const uint32_t off = P.b_transposed ? (uint32_t)(r >> 3) * sbo + (uint32_t)c * 128 + (uint32_t)(r & 7) * 16
                                                : (uint32_t)c * sbo + (uint32_t)(r >> 3) * 128 + (uint32_t)(r & 7) * 16;
            *reinterpret_cast<uint4*>(sB + off) = src[e];
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
    const uint64_t pol_stream = policy_evict_first();

    for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const int64_t row0 = t * TC_ROWS;
        // X tile -> canonical K-major layout: chunk kc of row r at (r/8)*sbo + kc*128 + (r%8)*16
        {
            const uint4* src = reinterpret_cast<const uint4*>(P.X);
            for (int e = tid; e < TC_ROWS * kchunks; e += TC_THREADS) {
                const int r = e / kchunks, kc = e - r * kchunks;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (row0 + r < P.N) v = ld_hint16(src + (size_t)(row0 + r) * kchunks + kc, pol_stream);
                *reinterpret_cast<uint4*>(sA + (uint32_t)(r >> 3) * sbo + (uint32_t)kc * 128 + (uint32_t)(r & 7) * 16) = v;
            }
        }
        // generic-proxy writes to shared memory -> visible to the tensor core (async proxy)
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (tid == 0) {
            const uint32_t a0 = smem_u32(sA), b0 = smem_u32(sB);
            for (int kk = 0; kk < K / 16; ++kk) {
                const uint64_t adesc = make_smem_desc(a0 + (uint32_t)kk * 256, 128, sbo);
                const uint64_t bdesc = make_smem_desc(b0 + (uint32_t)kk * 256, 128, sbo);
                mma_bf16_ss(tmem_base, adesc, bdesc, idesc, kk > 0 ? 1u : 0u);
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
        }
        const bool ok = mbar_wait_bounded(bar, parity);
        parity ^= 1;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (!ok) {
            failed = true;
        } else {
            // accumulator row = tensor-memory lane; this thread's row:
            const int64_t row = row0 + warp * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
            for (int c0 = 0; c0 < M; c0 += 16) {
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
                    uint4* dst = reinterpret_cast<uint4*>(P.Y + (size_t)row * M + c0);
                    st_stream16(dst, Chunk<__nv_bfloat16>::pack(f));
                    st_stream16(dst + 1, Chunk<__nv_bfloat16>::pack(f + 8));
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

bool linear_tc_supported(int64_t N, int K, int M, gnn_dtype dtype) {
    if (dtype != GNN_BF16 || N <= 0) return false;
    if (K % 16 != 0 || K < 16 || K > 256) return false;
    if (M % 16 != 0 || M < 16 || M > 256) return false;
    return true;
}

gnn_status linear_tc_forward(const void* X, const void* W, int64_t N, int K, int M, int w_transposed, void* Y,
                             int* d_flag, cudaStream_t st) {
    const char* who = "gnn_linear (tensor-core path)";
    GNN_REQUIRE(aligned16(X) && aligned16(W) && aligned16(Y), GNN_ERR_INVALID_ARG, "%s: matrices must be 16-byte aligned", who);
    TcParams P;
    P.X = (const __nv_bfloat16*)X; P.W = (const __nv_bfloat16*)W; P.Y = (__nv_bfloat16*)Y;
    P.N = N; P.K = K; P.M = M; P.b_transposed = w_transposed; P.status = d_flag;
    int cols = 32;
    while (cols < M) cols <<= 1;
    P.tmem_cols = cols;
    const size_t smem = (size_t)M * K * 2 + (size_t)TC_ROWS * K * 2;
    cudaError_t e = cudaFuncSetAttribute(linear_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "%s: cudaFuncSetAttribute: %s", who, cudaGetErrorString(e));
    const int64_t ntiles = (N + TC_ROWS - 1) / TC_ROWS;
    const int grid = (int)(ntiles < 148 ? ntiles : 148);
    linear_tc_kernel<<<grid, TC_THREADS, smem, st>>>(P);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

}  // namespace gnn
