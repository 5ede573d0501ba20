// Measurement aid (no counterpart in the paper): a loop that does nothing but the gathers of the fused propagate
// (Sec. 3 "Message Passing": one source row per edge) and adds them up, with no row structure, no multipliers and
// no output rows.  Its rate on a given index stream and row width is the ceiling that the L2 -> SM return path sets
// for the reduction kernels on that stream; bench.py and microbench.py report the kernels against it.
#include "common.cuh"

namespace gnn {

constexpr int PG_WARPS = 8;       // warps per block
constexpr int PG_U = 8;           // gathers a lane keeps in flight
constexpr int PG_CHUNK = 1024;    // positions per warp

// lanes of a warp form 32 / lpr groups of lpr lanes; a group gathers one row per step, lane li its 16-byte chunk li
template <int LPR>
__global__ void __launch_bounds__(PG_WARPS * 32, 4)
gather_probe_kernel(const int32_t* __restrict__ col, int64_t E, const char* __restrict__ X, uint32_t row_bytes, float* __restrict__ sink) {
    constexpr int NG = 32 / LPR;
    const int lane = threadIdx.x & 31, g = lane / LPR, li = lane % LPR;
    const int64_t w = (int64_t)blockIdx.x * PG_WARPS + (threadIdx.x >> 5);
    const int64_t p0 = w * PG_CHUNK;
    if (p0 >= E) return;
    const int64_t p1 = p0 + PG_CHUNK < E ? p0 + PG_CHUNK : E;
    const uint64_t pol_keep = policy_evict_last();
    const char* const Xl = X + (size_t)li * 16;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t p = p0 + g; p < p1; p += NG * PG_U) {
        int c[PG_U];
        uint4 b[PG_U];
#pragma unroll
        for (int u = 0; u < PG_U; ++u) c[u] = __ldg(col + (p + u * NG < p1 ? p + u * NG : p));  // past the end: the same row again
#pragma unroll
        for (int u = 0; u < PG_U; ++u) b[u] = ld_hint16(Xl + (size_t)(uint32_t)c[u] * row_bytes, pol_keep);
#pragma unroll
        for (int u = 0; u < PG_U; ++u) {
            acc.x += __uint_as_float(b[u].x); acc.y += __uint_as_float(b[u].y);
            acc.z += __uint_as_float(b[u].z); acc.w += __uint_as_float(b[u].w);
        }
    }
    // one value per lane keeps every gather alive
    sink[w * 32 + lane] = (acc.x + acc.y) + (acc.z + acc.w);
}

}  // namespace gnn

using namespace gnn;

extern "C" {

size_t gnn_probe_gather_sink_floats(int64_t E) { return E > 0 ? (size_t)ceil_div(E, PG_CHUNK) * 32 : 32; }

gnn_status gnn_probe_gather(const int32_t* col, int64_t E, const void* X, int32_t N, int row_bytes, float* sink, gnn_stream stream) {
    const char* who = "gnn_probe_gather";
    GNN_REQUIRE(col && X && sink && N > 0 && E > 0, GNN_ERR_INVALID_ARG, "%s: null or empty argument", who);
    GNN_REQUIRE(row_bytes == 64 || row_bytes == 128 || row_bytes == 256 || row_bytes == 512, GNN_ERR_UNSUPPORTED,
                "%s: rows of 64, 128, 256 or 512 bytes", who);
    GNN_REQUIRE(aligned16(X), GNN_ERR_INVALID_ARG, "%s: X must be 16-byte aligned", who);
    cudaStream_t st = as_stream(stream);
    const int grid = (int)ceil_div(ceil_div(E, PG_CHUNK), PG_WARPS);
    const char* Xc = (const char*)X;
    switch (row_bytes / 16) {
        case 4: gather_probe_kernel<4><<<grid, PG_WARPS * 32, 0, st>>>(col, E, Xc, 64, sink); break;
        case 8: gather_probe_kernel<8><<<grid, PG_WARPS * 32, 0, st>>>(col, E, Xc, 128, sink); break;
        case 16: gather_probe_kernel<16><<<grid, PG_WARPS * 32, 0, st>>>(col, E, Xc, 256, sink); break;
        default: gather_probe_kernel<32><<<grid, PG_WARPS * 32, 0, st>>>(col, E, Xc, 512, sink); break;
    }
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

}  // extern "C"
