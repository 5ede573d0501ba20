// Fused propagate (Sec. 3 "Message Passing": apply_edges + aggregate_neighbors combined into a
// generalised sparse x dense product) and its backward passes.
//
// Two kernels share one decomposition and one fix-up pass: the row-walking kernel below (graphs of
// 8 Mi edges and more, and rows wider than 512 bytes) and the position-first kernel further down
// (propagate_flat_kernel: smaller graphs, whose rows are mostly a handful of edges).
//
// Work decomposition: the E positions of the sparse form are cut into fixed chunks of
// consecutive edges (64 to 1024, by graph size), one warp per chunk (merge-path style: perfect balance on power-law rows
// without any per-graph schedule).  A warp finds its first row by binary search in rowptr and
// walks the rows that start inside its chunk (runs of rows without edges are jumped over with one
// search; their zero result comes from a separate row scan).  Rows lying wholly inside the chunk are reduced
// and written directly.  A row cut by a chunk boundary leaves fp32 partials (one "head" slot and
// one "tail" slot per chunk) that a second kernel combines in ascending chunk order.  Every
// accumulation order is a fixed function of (E, F, dtype), so results are bit-reproducible and
// no floating-point atomics are needed.
//
// Inside a warp, a feature row of F*s bytes is covered by LPR lanes holding one 16-byte chunk
// each (times VPL when a row is wider than 512 bytes); the 32/LPR lane groups take alternating
// edges, and are combined by an xor-shuffle tree at the end of each row.
#include <mutex>

#include "propagate.cuh"

#ifndef PF_U_NARROW
#define PF_U_NARROW 4
#endif
#ifndef PF_U_WIDE
#define PF_U_WIDE 8
#endif
#ifndef PF_MIN_BLOCKS
#define PF_MIN_BLOCKS 4
#endif
// rows of at most 128 bytes (a lane group of 4 or 8) keep four gathers in flight per group and fit five blocks per
// SM (48 registers, 4-28 bytes spilled): 1-3 % faster on the large graph; six blocks spill into the loop
#ifndef PF_MIN_BLOCKS_NARROW
#define PF_MIN_BLOCKS_NARROW 5
#endif
#ifndef PF_NARROW_LPR
#define PF_NARROW_LPR 8
#endif

namespace gnn {

struct PropParams {
    const int64_t* rowptr;  // rows of the output
    const int32_t* col;     // gathered row of X per position (nullptr: position p gathers row p)
    const float* w;         // per-position multiplier or nullptr
    const void* X;          // gathered matrix [N,F]
    void* out;              // [N,F]
    int32_t* argmax;        // MODE_MAX/MIN: winner positions [N,F] or nullptr
    const int64_t* gscale_rowptr;  // if set: each gathered row c is divided by max(1, length of
                                   // row c in this other sparse form) -- backward of MEAN
    const int32_t* route_arg;  // MODE_ROUTE: forward argmax [N,F]
    const int32_t* route_pos;  // MODE_ROUTE: forward position of each transposed position
    int32_t N;
    int64_t E;
    int nvec;  // 16-byte chunks per feature row (of the column slab this launch covers)
    uint32_t x_ld, out_ld;  // bytes between consecutive rows of X and of out (>= nvec*16)
    int F;
    int mean;  // divide the finished row by max(1, row length)
    int chunk;  // edges per warp: 64, 128, 256 or 1024
    int64_t nchunks;
    int fix_long;           // rows cut into more than FIX_LONG chunks are left to propagate_fixup_long_kernel
    int32_t* tail_row;  // [nchunks] row whose tail partial lives in slot 1, or -1
    float* part_val;    // [nchunks][2][F]
    int32_t* part_arg;  // [nchunks][2][F] (MODE_MAX/MIN)
    // MODE_HEADSUM: multiplier per (position, head), features of head h = [h*fph, (h+1)*fph)
    const float* wh;  // [E,H]
    const int32_t* wh_index;  // flat kernel only: row of wh per position, or nullptr (= the position)
    int H, fph;
    // optional rank-1 epilogue: out[r,f] += epi_l[r,h(f)]*epi_a[f] + epi_r[r,h(f)]*epi_b[f]
    const float *epi_l, *epi_r, *epi_a, *epi_b;
    // MODE_EFSUM: multiplier per (position, feature), fp32 [E, ef_ld]
    const float* ef;
    int ef_ld;
    // optional row epilogue (has_epi), applied in fp32 to a finished row before its single rounding:
    //   v = agg_c * v + self_c * c(r) * self_X[r,f] + bias[f], then max(v, 0) if relu
    // c(r) = 1 (GNN_SELF_ALWAYS), the length of row r in self_rowptr (GNN_SELF_TIMES_DEGREE), or 1 if that
    // length is positive else 0 (GNN_SELF_IF_NONEMPTY)
    int has_epi;
    float agg_c, self_c;
    int self_mode, relu;
    const void* self_X;
    uint32_t self_ld;  // bytes between rows of self_X
    const int64_t* self_rowptr;
    const float* bias;  // [F] or nullptr
};

// the row epilogue of PropParams on the 16-byte column ci of finished row `row`
template <typename T>
__device__ __forceinline__ void row_epilogue(const PropParams& P, int64_t row, int ci, float* v) {
    constexpr int EPC = Chunk<T>::N;
    if (!P.has_epi) return;
    if (P.agg_c != 1.0f) {
#pragma unroll
        for (int j = 0; j < EPC; ++j) v[j] *= P.agg_c;
    }
    if (P.self_X) {
        float c = P.self_c;
        if (P.self_mode != GNN_SELF_ALWAYS) {
            const int64_t d = P.self_rowptr[row + 1] - P.self_rowptr[row];
            c = (P.self_mode == GNN_SELF_TIMES_DEGREE) ? c * (float)d : (d > 0 ? c : 0.f);
        }
        float x[EPC];
        Chunk<T>::unpack(__ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(P.self_X) + (size_t)row * P.self_ld + (size_t)ci * 16)), x);
#pragma unroll
        for (int j = 0; j < EPC; ++j) v[j] = fmaf(c, x[j], v[j]);
    }
    if (P.bias) {
#pragma unroll
        for (int j = 0; j < EPC; ++j) v[j] += P.bias[ci * EPC + j];
    }
    if (P.relu) {
#pragma unroll
        for (int j = 0; j < EPC; ++j) v[j] = fmaxf(v[j], 0.f);
    }
}

// d.xy += w.xy * x.xy as one packed fp32x2 FMA (each half is an IEEE fused multiply-add)
__device__ __forceinline__ void fma2(float& a0, float& a1, float x0, float x1, float w0, float w1) {
    asm("{\n\t.reg .b64 ra, rb, rc;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "mov.b64 rc, {%0, %1};\n\tfma.rn.f32x2 rc, ra, rb, rc;\n\tmov.b64 {%0, %1}, rc;\n\t}"
        : "+f"(a0), "+f"(a1)
        : "f"(x0), "f"(x1), "f"(w0), "f"(w1));
}

template <typename T, int VPL, int MODE>
struct Acc {
    static constexpr int EPC = Chunk<T>::N;
    static constexpr bool ARG = (MODE == MODE_MAX || MODE == MODE_MIN);
    float v[VPL][EPC];
    int32_t a[ARG ? VPL : 1][EPC];
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int i = 0; i < VPL; ++i)
#pragma unroll
            for (int j = 0; j < EPC; ++j) {
                v[i][j] = 0.f;
                if (ARG) a[i][j] = -1;
            }
    }
};

// does candidate (cv, ca) beat the incumbent (v, a)?  ties go to the smaller position
template <int MODE>
__device__ __forceinline__ bool beats(float cv, int32_t ca, float v, int32_t a) {
    if (ca < 0) return false;
    if (a < 0) return true;
    bool better = (MODE == MODE_MAX) ? (cv > v) : (cv < v);
    return better || (cv == v && ca < a);
}

// Smallest row r in [lo, N) with rowptr[r + 1] > v, or N: the first row at or after lo that has a
// position beyond v.  Warp-cooperative (every lane must call it with the same arguments): a look at the
// next 32 rows, then a 32-way search.
__device__ __forceinline__ int first_row_ending_after(const int64_t* __restrict__ rowptr, int lo, int N, int64_t v, int lane) {
    {  // the common case, one coalesced load: the row is among the next 32
        const int r = lo + lane;
        const unsigned m = __ballot_sync(0xffffffffu, r >= N || rowptr[r + 1] > v);
        if (m) return min(lo + __ffs(m) - 1, N);
        lo += 32;
    }
    int hi = N;
    while (hi > lo) {
        const int step = (hi - lo + 31) / 32;
        const int idx = lo + lane * step;
        const bool le = idx < hi && rowptr[idx + 1] <= v;  // true for a prefix of the lanes
        const int k = __popc(__ballot_sync(0xffffffffu, le));
        if (k == 0) { hi = lo; break; }
        const int nlo = lo + (k - 1) * step + 1;
        hi = min(lo + k * step, hi);
        lo = nlo;
    }
    return lo;
}

// Rows without edges get their (empty) result from a scan that is independent of the edge chunks:
// warp c of nchunks takes rows [c*per, (c+1)*per) and calls write_row(r) for each empty one, so a
// long run of such rows (a bipartite graph's source side, say) is spread over all warps.
template <class WriteRow>
__device__ __forceinline__ void scan_empty_rows(const int64_t* __restrict__ rowptr, int N, int64_t c, int64_t nchunks, int lane, WriteRow write_row) {
    const int64_t per = (N + nchunks - 1) / nchunks;
    const int64_t b0 = c * per;
    const int r0 = (int)(b0 < N ? b0 : N), r1 = (int)(b0 + per < N ? b0 + per : N);
    for (int rb = r0; rb < r1; rb += 32) {
        const int r = rb + lane;
        unsigned em = __ballot_sync(0xffffffffu, r < r1 && rowptr[r + 1] == rowptr[r]);
        while (em) {
            const int bit = __ffs(em) - 1;
            em &= em - 1;
            write_row(rb + bit);
        }
    }
}

// per-warp staging area for one slab of PF_SLAB consecutive positions:
// (gathered row, forward position [MODE_ROUTE], multiplier, multiplier) -- the multiplier is
// stored twice so that one 16-byte shared load yields the register pair the packed FMA wants
struct SlabSmem {
    int4 e[PF_SLAB];
};

template <typename T, int LPR, int VPL, int MODE>
struct Walker {
    // issue the last (fewer than U) gathers of a row segment together instead of one by one: measured
    // faster for max/min (-7..-29 % on short-row graphs), slower for the sum and routing modes
    static constexpr bool BATCH_TAIL = (MODE == MODE_MAX || MODE == MODE_MIN);
    // fp32 sums: the ragged end of a row segment goes through the same loop as the full batches, its missing
    // positions predicated off, so that the gathers of a short row are in flight together (measured on the large
    // graph: F = 64 -6 %, F = 128..512 -1..-2 % sustained, -7 % in a burst).  Not for bf16: with eight accumulators
    // per lane the loop spills registers on full-warp rows (a third slower) and gains nothing on narrow ones.
    static constexpr bool ONE_LOOP = MODE == MODE_SUM && VPL == 1 && Chunk<T>::N == 4;
    static constexpr int EPC = Chunk<T>::N;
    static constexpr int NG = 32 / LPR;
    static constexpr bool EF = (MODE == MODE_EFSUM);  // one multiplier per (position, feature)
    // the per-feature mode also streams EPC multipliers per gathered chunk: half as many gathers in flight
    // 256-byte rows of a sum (half a warp per row): four (bf16) or six (fp32) gathers in flight measured 3 % faster than
    // eight on the large graph (bf16 F=128 3.52 -> 3.41 ms, fp32 F=64 3.10 -> 3.01 ms)
    static constexpr int U_MID = Chunk<T>::N == 8 ? 4 : 6;
    static constexpr int U = (LPR >= 16) ? (EF ? (PF_U_WIDE / VPL > 1 ? PF_U_WIDE / VPL / 2 : 1)
                                               : (LPR == 16 && VPL == 1 && MODE == MODE_SUM ? U_MID : PF_U_WIDE / VPL))
                                         : PF_U_NARROW;
    static constexpr int MW = EF ? EPC : 1;  // multipliers a lane holds per gathered 16-byte chunk
    static constexpr bool ARG = (MODE == MODE_MAX || MODE == MODE_MIN);
    using A = Acc<T, VPL, MODE>;

    // multipliers of one position for this lane's chunk v: per head (MODE_HEADSUM) or per feature (MODE_EFSUM)
    __device__ __forceinline__ static void load_mul(const PropParams& P, const float* base, size_t rel, float* dst) {
        if (MODE == MODE_HEADSUM) {
            dst[0] = __ldg(base + rel * P.H);
        } else if (EF) {
            const float4* q = reinterpret_cast<const float4*>(base + rel * P.ef_ld);
#pragma unroll
            for (int t = 0; t < MW / 4; ++t) {
                const float4 a = __ldcs(q + t);
                dst[4 * t] = a.x; dst[4 * t + 1] = a.y; dst[4 * t + 2] = a.z; dst[4 * t + 3] = a.w;
            }
        } else {
            dst[0] = 0.f;
        }
    }

    // copy indices and multipliers of positions [sb, se) into shared memory (one round trip)
    __device__ __forceinline__ static void stage(const PropParams& P, int sb, int se, int lane,
                                                 SlabSmem& S, uint64_t pol_stream) {
        __syncwarp();
        for (int i = lane; i < se - sb; i += 32) {
            int c = P.col ? ld_hint_i32(P.col + sb + i, pol_stream) : (int)(sb + i);  // no col: row p of X
            float w = P.w ? ld_hint_f32(P.w + sb + i, pol_stream) : 1.0f;
            if (P.gscale_rowptr) {
                int64_t d = P.gscale_rowptr[c + 1] - P.gscale_rowptr[c];
                w = w / (float)(d > 1 ? d : 1);
            }
            int t = (MODE == MODE_ROUTE) ? ld_hint_i32(P.route_pos + sb + i, pol_stream) : 0;
            S.e[i] = make_int4(c, t, __float_as_int(w), __float_as_int(w));
        }
        __syncwarp();
    }

    // one gathered row chunk -> accumulator
    __device__ __forceinline__ static void consume(const PropParams& P, const int4& e, const uint4* buf,
                                                   const float* hw, int32_t pos, int lane_chunk0, A& acc) {
        const float w0 = __int_as_float(e.z), w1 = __int_as_float(e.w);
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            float x[EPC];
            Chunk<T>::unpack(buf[v], x);
            if (MODE == MODE_HEADSUM) {
                const float m = hw[v] * w0;  // w0 = 1 unless the gathered rows are rescaled (backward of the mean)
#pragma unroll
                for (int j = 0; j < EPC; j += 2) fma2(acc.v[v][j], acc.v[v][j + 1], x[j], x[j + 1], m, m);
            } else if (EF) {
#pragma unroll
                for (int j = 0; j < EPC; j += 2)
                    fma2(acc.v[v][j], acc.v[v][j + 1], x[j], x[j + 1], hw[v * MW + j] * w0, hw[v * MW + j + 1] * w0);
            } else if (MODE == MODE_SUM) {
#pragma unroll
                for (int j = 0; j < EPC; j += 2) fma2(acc.v[v][j], acc.v[v][j + 1], x[j], x[j + 1], w0, w1);
            } else if (ARG) {
#pragma unroll
                for (int j = 0; j < EPC; ++j) {
                    float m = P.w ? w0 * x[j] : x[j];
                    // positions arrive in ascending order within a group: strict comparison
                    // keeps the first of equal values
                    bool take = acc.a[ARG ? v : 0][j] < 0 ||
                                (MODE == MODE_MAX ? m > acc.v[v][j] : m < acc.v[v][j]);
                    if (take) { acc.v[v][j] = m; acc.a[ARG ? v : 0][j] = pos; }
                }
            } else {  // MODE_ROUTE: keep dOut only where this edge was the winner
                const int32_t* ap = P.route_arg + (size_t)e.x * P.F + (size_t)(v * LPR + lane_chunk0) * EPC;
                int32_t win[EPC];
#pragma unroll
                for (int j = 0; j < EPC; j += 4) {
                    int4 t = *reinterpret_cast<const int4*>(ap + j);
                    win[j] = t.x; win[j + 1] = t.y; win[j + 2] = t.z; win[j + 3] = t.w;
                }
#pragma unroll
                for (int j = 0; j < EPC; ++j)
                    if (win[j] == e.y) acc.v[v][j] = fmaf(w0, x[j], acc.v[v][j]);
            }
        }
    }

    // accumulate staged positions [p0, e1) (all inside the slab starting at sb) into acc.
    // Lanes beyond the row width (rows that do not fill LPR*VPL chunks) read chunk 0 instead:
    // always in bounds, never written back, so the loop needs no lane masking.
    __device__ __forceinline__ static void slab_segment(const PropParams& P, int sb, int p0, int e1,
                                                        int lane, const SlabSmem& S, uint64_t pol_keep, A& acc) {
        const int g = lane / LPR, li = lane % LPR;
        const uint32_t row_bytes = P.x_ld;
        const char* Xl[VPL];
        int c0[VPL];
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            c0[v] = (v * LPR + li < P.nvec) ? v * LPR + li : 0;
            Xl[v] = reinterpret_cast<const char*>(P.X) + (size_t)c0[v] * 16;
        }
        const int lane_chunk0 = (li < P.nvec) ? li : 0;  // VPL > 1 only with full rows of 32 lanes
        const float* whl[VPL];  // this lane's head column (MODE_HEADSUM) or feature columns (MODE_EFSUM) of the multipliers
#pragma unroll
        for (int v = 0; v < VPL; ++v)
            whl[v] = (MODE == MODE_HEADSUM) ? P.wh + (size_t)sb * P.H + (c0[v] * EPC) / P.fph
                     : EF ? P.ef + (size_t)sb * P.ef_ld + (size_t)c0[v] * EPC : nullptr;
        const int i1 = e1 - sb;
        int i = p0 - sb + g;
        if (ONE_LOOP) {
            for (; i < i1; i += NG * U) {
                int cols[U];
                uint4 buf[U][VPL];
#pragma unroll
                for (int u = 0; u < U; ++u) cols[u] = S.e[i + u * NG < i1 ? i + u * NG : i].x;
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (i + u * NG < i1) {
#pragma unroll
                        for (int v = 0; v < VPL; ++v) buf[u][v] = ld_hint16(Xl[v] + (size_t)(uint32_t)cols[u] * row_bytes, pol_keep);
                    }
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (i + u * NG < i1) {
                        const float w = __int_as_float(S.e[i + u * NG].z);  // read again here: not held across the gathers
#pragma unroll
                        for (int v = 0; v < VPL; ++v) {
                            float x[EPC];
                            Chunk<T>::unpack(buf[u][v], x);
#pragma unroll
                            for (int j = 0; j < EPC; j += 2) fma2(acc.v[v][j], acc.v[v][j + 1], x[j], x[j + 1], w, w);
                        }
                    }
            }
            return;
        }
        // full groups of U positions per lane group: no predicates
        for (; i + (U - 1) * NG < i1; i += NG * U) {
            int4 e[U];
            uint4 buf[U][VPL];
            float hw[U][VPL * MW];
#pragma unroll
            for (int u = 0; u < U; ++u) e[u] = S.e[i + u * NG];
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int v = 0; v < VPL; ++v) {
                    buf[u][v] = ld_hint16(Xl[v] + (size_t)(uint32_t)e[u].x * row_bytes, pol_keep);
                    load_mul(P, whl[v], (size_t)(i + u * NG), &hw[u][v * MW]);
                }
#pragma unroll
            for (int u = 0; u < U; ++u) consume(P, e[u], buf[u], hw[u], (int32_t)(sb + i + u * NG), lane_chunk0, acc);
        }
        if (BATCH_TAIL) {
            // remainder: cnt < U positions for this lane group, all their loads in flight at once
            if (i < i1) {
                const int cnt = (i1 - i + NG - 1) / NG;
                int4 e[U];
                uint4 buf[U][VPL];
                float hw[U][VPL * MW];
#pragma unroll
                for (int u = 0; u < U - 1; ++u)
                    if (u < cnt) {
                        e[u] = S.e[i + u * NG];
#pragma unroll
                        for (int v = 0; v < VPL; ++v) {
                            buf[u][v] = ld_hint16(Xl[v] + (size_t)(uint32_t)e[u].x * row_bytes, pol_keep);
                            load_mul(P, whl[v], (size_t)(i + u * NG), &hw[u][v * MW]);
                        }
                    }
#pragma unroll
                for (int u = 0; u < U - 1; ++u)
                    if (u < cnt) consume(P, e[u], buf[u], hw[u], (int32_t)(sb + i + u * NG), lane_chunk0, acc);
            }
        } else {
            // remainder: fewer than U positions for this lane group
            for (; i < i1; i += NG) {
                const int4 e = S.e[i];
                uint4 buf[VPL];
                float hw[VPL * MW];
#pragma unroll
                for (int v = 0; v < VPL; ++v) {
                    buf[v] = ld_hint16(Xl[v] + (size_t)(uint32_t)e.x * row_bytes, pol_keep);
                    load_mul(P, whl[v], (size_t)i, &hw[v * MW]);
                }
                consume(P, e, buf, hw, (int32_t)(sb + i), lane_chunk0, acc);
            }
        }
    }

    // optional rank-1 update of a finished row chunk (see PropParams::epi_*)
    __device__ __forceinline__ static void epilogue(const PropParams& P, int64_t row, int ci, float* v) {
        if (!P.epi_l) return;
        const int h = (ci * EPC) / P.fph;  // a 16-byte chunk lies inside one head
        const float el = P.epi_l[(size_t)row * P.H + h], er = P.epi_r[(size_t)row * P.H + h];
#pragma unroll
        for (int j = 0; j < EPC; ++j) v[j] += el * P.epi_a[ci * EPC + j] + er * P.epi_b[ci * EPC + j];
    }

    // combine the lane groups; afterwards every lane holds the result for its chunk index
    __device__ __forceinline__ static void combine_groups(A& acc, int lane) {
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
            const bool low = (lane & o) == 0;
#pragma unroll
            for (int v = 0; v < VPL; ++v)
#pragma unroll
                for (int j = 0; j < EPC; ++j) {
                    float mine = acc.v[v][j];
                    float ov = __shfl_xor_sync(0xffffffffu, mine, o);
                    if (ARG) {
                        int32_t ma = acc.a[ARG ? v : 0][j];
                        int32_t oa = __shfl_xor_sync(0xffffffffu, ma, o);
                        if (beats<MODE>(ov, oa, mine, ma)) { acc.v[v][j] = ov; acc.a[ARG ? v : 0][j] = oa; }
                    } else {
                        // both partners add in the same operand order -> identical bits
                        acc.v[v][j] = low ? (mine + ov) : (ov + mine);
                    }
                }
        }
    }

    __device__ __forceinline__ static void write_final(const PropParams& P, int row,
                                                       int deg, int lane, A& acc) {
        if (lane >= LPR) return;
        char* ob = reinterpret_cast<char*>(P.out) + (size_t)row * P.out_ld;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const int ci = v * LPR + lane;
            if (ci >= P.nvec) continue;
            if (P.mean) {
                float d = (float)(deg > 1 ? deg : 1);
#pragma unroll
                for (int j = 0; j < EPC; ++j) acc.v[v][j] = acc.v[v][j] / d;
            }
            if (MODE == MODE_HEADSUM) epilogue(P, row, ci, acc.v[v]);
            row_epilogue<T>(P, row, ci, acc.v[v]);
            st_stream16(ob + (size_t)ci * 16, Chunk<T>::pack(acc.v[v]));
            if (ARG && P.argmax) {
                int32_t* ap = P.argmax + (size_t)row * P.F + (size_t)ci * EPC;
#pragma unroll
                for (int j = 0; j < EPC; j += 4)
                    *reinterpret_cast<int4*>(ap + j) =
                        make_int4(acc.a[ARG ? v : 0][j], acc.a[ARG ? v : 0][j + 1],
                                  acc.a[ARG ? v : 0][j + 2], acc.a[ARG ? v : 0][j + 3]);
            }
        }
    }

    __device__ __forceinline__ static void write_partial(const PropParams& P, int chunk,
                                                         int which, int lane, const A& acc) {
        if (lane >= LPR) return;
        size_t off = ((size_t)chunk * 2 + which) * P.F;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const int ci = v * LPR + lane;
            if (ci >= P.nvec) continue;
            float* pv = P.part_val + off + (size_t)ci * EPC;
#pragma unroll
            for (int j = 0; j < EPC; j += 4)
                *reinterpret_cast<float4*>(pv + j) =
                    make_float4(acc.v[v][j], acc.v[v][j + 1], acc.v[v][j + 2], acc.v[v][j + 3]);
            if (ARG) {
                int32_t* pa = P.part_arg + off + (size_t)ci * EPC;
#pragma unroll
                for (int j = 0; j < EPC; j += 4)
                    *reinterpret_cast<int4*>(pa + j) =
                        make_int4(acc.a[ARG ? v : 0][j], acc.a[ARG ? v : 0][j + 1],
                                  acc.a[ARG ? v : 0][j + 2], acc.a[ARG ? v : 0][j + 3]);
            }
        }
    }
};

// max / min (value and winner per element): blocks per SM measured on a 12 M-edge R-MAT graph, forward time in us at
// 2 / 3 / 4 blocks: fp32 64-byte rows 479 / 458 / 440, 256-byte 754 / 684 / 692, 512-byte 954 / 873 / 891; bf16 32-byte
// rows 823 / 655 / 623, 128-byte 861 / 710 / 677, 256-byte 1024 / 1060 / 1138, 512-byte 1346 / 1341 / 1383
__host__ __device__ constexpr int pf_arg_blocks(int lpr, int elem_bytes) { return lpr <= 8 ? 4 : (elem_bytes == 4 ? 3 : 2); }

template <typename T, int LPR, int VPL, int MODE>
__global__ void __launch_bounds__(PF_WARPS * 32, (VPL == 1 && (MODE == MODE_SUM || MODE == MODE_HEADSUM)) ? (LPR <= PF_NARROW_LPR ? PF_MIN_BLOCKS_NARROW : PF_MIN_BLOCKS)
                  : ((VPL == 1 && (MODE == MODE_MAX || MODE == MODE_MIN)) ? pf_arg_blocks(LPR, (int)sizeof(T)) : 2))
propagate_chunk_kernel(const PropParams P) {
    using W = Walker<T, LPR, VPL, MODE>;
    __shared__ SlabSmem s_slab[PF_WARPS];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int c = (int)blockIdx.x * PF_WARPS + wib;  // chunk numbers and positions fit 32 bits (the host checks E < 2^31)
    if (c >= P.nchunks) return;
    SlabSmem& S = s_slab[wib];
    const uint64_t pol_keep = policy_evict_last(), pol_stream = policy_evict_first();
    const int cs = c * P.chunk;
    const int ce = ((int64_t)cs + P.chunk < P.E) ? cs + P.chunk : (int)P.E;

    typename W::A acc;

    // cur = the row containing position cs, or the first (possibly empty) row starting at cs
    int cur = lower_bound_i64(P.rowptr, P.N + 1, cs);
    if (P.rowptr[cur] > cs) --cur;
    int pos = cs;
    int sb = cs - PF_SLAB;  // nothing staged yet
    int32_t tail = -1;
    while (cur < P.N) {
        const int rs = (int)P.rowptr[cur], re = (int)P.rowptr[cur + 1];
        if (re == rs) {  // no edges (written by the scan above): jump to the next row that has some
            cur = first_row_ending_after(P.rowptr, cur + 1, P.N, rs, lane);
            if (cur >= P.N || P.rowptr[cur] >= ce) break;  // it belongs to a later chunk
            continue;
        }
        const int b = re < ce ? re : ce;
        acc.clear();
        const int pos0 = pos;
        while (pos < b) {
            if (pos >= sb + PF_SLAB) {
                sb = cs + ((pos - cs) / PF_SLAB) * PF_SLAB;
                W::stage(P, sb, (sb + PF_SLAB < ce) ? sb + PF_SLAB : ce, lane, S, pol_stream);
            }
            const int e = (b < sb + PF_SLAB) ? b : sb + PF_SLAB;
            W::slab_segment(P, sb, pos, e, lane, S, pol_keep, acc);
            pos = e;
        }
        // with at most one position only lane group 0 holds data: nothing to combine
        if (b - (pos0) > 1) W::combine_groups(acc, lane);
        const bool started_here = rs >= cs;
        if (re <= ce) {  // the row ends inside this chunk
            if (started_here) W::write_final(P, cur, re - rs, lane, acc);
            else W::write_partial(P, c, 0, lane, acc);
            ++cur;
            if (re >= ce) break;  // the next row with edges starts in the next chunk
        } else {  // the row continues in the next chunk
            W::write_partial(P, c, started_here ? 1 : 0, lane, acc);
            if (started_here) tail = cur;
            break;
        }
    }
    if (lane == 0) P.tail_row[c] = tail;
    // rows without edges, after the walk so that the hot loop's register allocation is undisturbed
    scan_empty_rows(P.rowptr, P.N, c, P.nchunks, lane, [&](int r) {
        acc.clear();
        W::write_final(P, r, 0, lane, acc);
    });
}

// Rows cut into more than FIX_LONG chunks (hub rows of large graphs) are finished by a block each instead of a
// thread per 16-byte column: one thread walking a hub's hundreds of partial rows pays a load latency per eight of
// them (45-150 us per call on a graph whose largest row spans 300 chunks, far more on a star-like graph).
constexpr int FIX_LONG = 64;
constexpr int FIXL_THREADS = 256;
constexpr int FIXL_BLOCKS = 592;
#ifndef FIXL_MIN_CHUNKS_N
#define FIXL_MIN_CHUNKS_N 16384
#endif
constexpr int64_t FIXL_MIN_CHUNKS = FIXL_MIN_CHUNKS_N;  // below this many chunks the extra launch costs more than the walk
constexpr int64_t FIXL_MIN_CHUNKS_ARG = 4096;           // the same for max / min

// second pass: finish the rows that were cut by chunk boundaries, in ascending chunk order
template <typename T, int MODE>
__global__ void propagate_fixup_kernel(const PropParams P) {
    constexpr int EPC = Chunk<T>::N;
    constexpr bool ARG = (MODE == MODE_MAX || MODE == MODE_MIN);
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t c = t / P.nvec;
    const int ci = (int)(t - c * P.nvec);
    if (c >= P.nchunks) return;
    const int32_t r = P.tail_row[c];
    if (r < 0) return;
    const int64_t rs = P.rowptr[r], re = P.rowptr[r + 1];
    const int64_t c_end = (re - 1) / P.chunk;
    if (P.fix_long && c_end - c > FIX_LONG) return;  // a hub row: propagate_fixup_long_kernel finishes it
    float v[EPC];
    int32_t a[EPC];
    const size_t F = P.F;
    {
        const float* pv = P.part_val + ((size_t)c * 2 + 1) * F + (size_t)ci * EPC;
#pragma unroll
        for (int j = 0; j < EPC; ++j) v[j] = pv[j];
        if (ARG) {
            const int32_t* pa = P.part_arg + ((size_t)c * 2 + 1) * F + (size_t)ci * EPC;
#pragma unroll
            for (int j = 0; j < EPC; ++j) a[j] = pa[j];
        }
    }
    // a hub row is cut into hundreds of chunks: eight chunks' partials are loaded together (independent
    // loads), then combined in ascending chunk order
    int64_t cc = c + 1;
    if (!ARG) {
        for (; cc + 8 <= c_end + 1; cc += 8) {
            float4 t[8][EPC / 4];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float4* pv = reinterpret_cast<const float4*>(P.part_val + ((size_t)(cc + u) * 2) * F + (size_t)ci * EPC);
#pragma unroll
                for (int q = 0; q < EPC / 4; ++q) t[u][q] = pv[q];
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
#pragma unroll
                for (int q = 0; q < EPC / 4; ++q) {
                    v[4 * q] += t[u][q].x; v[4 * q + 1] += t[u][q].y; v[4 * q + 2] += t[u][q].z; v[4 * q + 3] += t[u][q].w;
                }
        }
    }
    for (; cc <= c_end; ++cc) {
        const float* pv = P.part_val + ((size_t)cc * 2) * F + (size_t)ci * EPC;
        if (ARG) {
            const int32_t* pa = P.part_arg + ((size_t)cc * 2) * F + (size_t)ci * EPC;
#pragma unroll
            for (int j = 0; j < EPC; ++j)
                if (beats<MODE>(pv[j], pa[j], v[j], a[j])) { v[j] = pv[j]; a[j] = pa[j]; }
        } else {
#pragma unroll
            for (int j = 0; j < EPC; ++j) v[j] += pv[j];
        }
    }
    if (P.mean) {
        float d = (float)(re - rs);
#pragma unroll
        for (int j = 0; j < EPC; ++j) v[j] = v[j] / d;
    }
    if (MODE == MODE_HEADSUM && P.epi_l) {
        const int h = (ci * EPC) / P.fph;  // a 16-byte chunk lies inside one head
        const float el = P.epi_l[(size_t)r * P.H + h], er = P.epi_r[(size_t)r * P.H + h];
#pragma unroll
        for (int j = 0; j < EPC; ++j) v[j] += el * P.epi_a[ci * EPC + j] + er * P.epi_b[ci * EPC + j];
    }
    row_epilogue<T>(P, r, ci, v);
    char* ob = reinterpret_cast<char*>(P.out) + (size_t)r * P.out_ld + (size_t)ci * 16;
    *reinterpret_cast<uint4*>(ob) = Chunk<T>::pack(v);
    if (ARG && P.argmax) {
        int32_t* ap = P.argmax + (size_t)r * F + (size_t)ci * EPC;
#pragma unroll
        for (int j = 0; j < EPC; ++j) ap[j] = a[j];
    }
}

// Block b looks at its share of the chunks; for every row that starts in one of them and is cut
// into more than FIX_LONG chunks, thread (k, q) adds column float4 q of the partial rows k, k + K, k + 2K, ... of
// that row (K = 256 / (F/4) walkers per column, four loads in flight each), the K sums are added in walker order,
// and the row is scaled, given its epilogue and stored as in the kernel above.  The order of the additions is a
// fixed function of the row's length and F.  Max / min: the walkers keep (value, position) pairs and combine them
// with the same rule as everywhere else (ties go to the smaller position), which does not depend on the order.
template <typename T, int MODE>
__global__ void __launch_bounds__(FIXL_THREADS)
propagate_fixup_long_kernel(const PropParams P) {
    constexpr int EPC = Chunk<T>::N;
    constexpr bool ARG = (MODE == MODE_MAX || MODE == MODE_MIN);
    __shared__ float4 sums[FIXL_THREADS];
    __shared__ int4 args[ARG ? FIXL_THREADS : 1];
    __shared__ int todo[64];
    __shared__ int ntodo;
    const int tid = threadIdx.x;
    const int F = P.F, F4 = F / 4;
    const int K = FIXL_THREADS / F4 > 0 ? FIXL_THREADS / F4 : 1;
    const int k = tid / F4, q = tid - k * F4;
    const int64_t per = (P.nchunks + gridDim.x - 1) / gridDim.x;
    const int64_t c0 = (int64_t)blockIdx.x * per, c1 = c0 + per < P.nchunks ? c0 + per : P.nchunks;
    for (int64_t cb = c0; cb < c1; cb += 64) {  // 64 chunks at a time: find the long rows, then do them one by one
        if (tid == 0) ntodo = 0;
        __syncthreads();
        if (tid < 64 && cb + tid < c1) {
            const int32_t r = P.tail_row[cb + tid];
            if (r >= 0 && (P.rowptr[r + 1] - 1) / P.chunk - (cb + tid) > FIX_LONG) todo[atomicAdd(&ntodo, 1)] = tid;
        }
        __syncthreads();
        const int n = ntodo;
        for (int i = 0; i < n; ++i) {
            // rows of one block are independent: the order in which the list was filled does not matter
            const int64_t c = cb + todo[i];
            const int32_t r = P.tail_row[c];
            const int64_t rs = P.rowptr[r], re = P.rowptr[r + 1];
            const int64_t span = (re - 1) / P.chunk - c;  // partial rows: (c, tail), then the heads of c + 1 .. c + span
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            int4 arg = make_int4(-1, -1, -1, -1);
            if (k < K && q < F4) {
                for (int64_t j = k; j <= span; j += 4 * (int64_t)K) {
                    float4 t[4];
                    int4 ta[ARG ? 4 : 1];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int64_t jj = j + (int64_t)u * K;
                        if (jj <= span) {
                            const size_t slot = jj == 0 ? (size_t)c * 2 + 1 : (size_t)(c + jj) * 2;
                            t[u] = *(reinterpret_cast<const float4*>(P.part_val + slot * (size_t)F) + q);
                            if (ARG) ta[u] = *(reinterpret_cast<const int4*>(P.part_arg + slot * (size_t)F) + q);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (j + (int64_t)u * K <= span) {
                            if (ARG) {
                                if (beats<MODE>(t[u].x, ta[u].x, acc.x, arg.x)) { acc.x = t[u].x; arg.x = ta[u].x; }
                                if (beats<MODE>(t[u].y, ta[u].y, acc.y, arg.y)) { acc.y = t[u].y; arg.y = ta[u].y; }
                                if (beats<MODE>(t[u].z, ta[u].z, acc.z, arg.z)) { acc.z = t[u].z; arg.z = ta[u].z; }
                                if (beats<MODE>(t[u].w, ta[u].w, acc.w, arg.w)) { acc.w = t[u].w; arg.w = ta[u].w; }
                            } else {
                                acc.x += t[u].x; acc.y += t[u].y; acc.z += t[u].z; acc.w += t[u].w;
                            }
                        }
                }
                sums[k * F4 + q] = acc;
                if (ARG) args[k * F4 + q] = arg;
            }
            __syncthreads();
            if (tid < P.nvec) {
                const int ci = tid;
                float v[EPC];
                int32_t av[ARG ? EPC : 1];
#pragma unroll
                for (int j4 = 0; j4 < EPC / 4; ++j4) {
                    float4 a = sums[ci * (EPC / 4) + j4];
                    int4 aa = ARG ? args[ci * (EPC / 4) + j4] : make_int4(-1, -1, -1, -1);
                    for (int kk = 1; kk < K; ++kk) {
                        const float4 b = sums[kk * F4 + ci * (EPC / 4) + j4];
                        if (ARG) {
                            const int4 ba = args[kk * F4 + ci * (EPC / 4) + j4];
                            if (beats<MODE>(b.x, ba.x, a.x, aa.x)) { a.x = b.x; aa.x = ba.x; }
                            if (beats<MODE>(b.y, ba.y, a.y, aa.y)) { a.y = b.y; aa.y = ba.y; }
                            if (beats<MODE>(b.z, ba.z, a.z, aa.z)) { a.z = b.z; aa.z = ba.z; }
                            if (beats<MODE>(b.w, ba.w, a.w, aa.w)) { a.w = b.w; aa.w = ba.w; }
                        } else {
                            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
                        }
                    }
                    v[4 * j4] = a.x; v[4 * j4 + 1] = a.y; v[4 * j4 + 2] = a.z; v[4 * j4 + 3] = a.w;
                    if (ARG) { av[4 * j4] = aa.x; av[4 * j4 + 1] = aa.y; av[4 * j4 + 2] = aa.z; av[4 * j4 + 3] = aa.w; }
                }
                if (P.mean) {
                    const float d = (float)(re - rs);
#pragma unroll
                    for (int j = 0; j < EPC; ++j) v[j] = v[j] / d;
                }
                if (MODE == MODE_HEADSUM && P.epi_l) {
                    const int h = (ci * EPC) / P.fph;  // a 16-byte chunk lies inside one head
                    const float el = P.epi_l[(size_t)r * P.H + h], er = P.epi_r[(size_t)r * P.H + h];
#pragma unroll
                    for (int j = 0; j < EPC; ++j) v[j] += el * P.epi_a[ci * EPC + j] + er * P.epi_b[ci * EPC + j];
                }
                row_epilogue<T>(P, r, ci, v);
                char* ob = reinterpret_cast<char*>(P.out) + (size_t)r * P.out_ld + (size_t)ci * 16;
                *reinterpret_cast<uint4*>(ob) = Chunk<T>::pack(v);
                if (ARG && P.argmax) {
                    int32_t* ap = P.argmax + (size_t)r * F + (size_t)ci * EPC;
#pragma unroll
                    for (int j = 0; j < EPC; ++j) ap[j] = av[j];
                }
            }
            __syncthreads();
        }
    }
}

// ------------------------------------------------------------------ flat variant for short rows
// Sum / mean over graphs whose rows are mostly much shorter than a chunk (citation-style graphs:
// a handful of edges per row).  Walking such rows one at a time leaves one or two gathers in flight
// per lane group.  Here the gathers do not depend on the row structure:
//   1. the warp stages its 256 positions (gathered row, multiplier) and marks where rows start; a
//      prefix maximum gives every position the index of its row's start entry (row id and length
//      are kept per start entry);
//   2. each lane group takes a contiguous run of 256/NG positions and issues U = 8 independent
//      16-byte gathers at a time; the accumulator is flushed whenever the start entry changes;
//   3. rows cut by a run boundary are stitched inside the warp in run order (through shared
//      memory), rows cut by the chunk boundary leave the same head / tail partials as the
//      row-walking kernel, so the same fix-up pass finishes them.
// Rows without edges are written by a row scan that is spread over all warps (scan_empty_rows).
// All orders are fixed functions of (E, F, dtype).
constexpr int FL_WARPS = 4;
constexpr int FL_U = 8;

template <int EPC, bool ARG>
struct FlatSmem {
    int4 e[PF_SLAB];         // x: gathered row, y: start entry of the position's row, z: multiplier
    int32_t srow[PF_SLAB];   // [k] row starting at position k of the chunk ([0]: the row holding position 0)
    int32_t send[PF_SLAB];   // [k] its end, as a position of the chunk, capped at PF_SLAB + 1
    float sinv[PF_SLAB];     // [k] factor of the finished row: 1, or 1 / length for the mean
    float head[32 * EPC];    // per lane: partial of the run's first row when that row began before the run
    float tail[32 * EPC];    // per lane: partial of the run's last row when it continues past the run
    int32_t head_a[ARG ? 32 * EPC : 1];  // max/min: winner positions of those partials
    int32_t tail_a[ARG ? 32 * EPC : 1];
    int32_t hk[8], hclosed[8], tk[8];  // per run: start entries of those rows (-1: none), head row ends in the run
};

// MODE_SUM (sum / mean), MODE_MAX / MODE_MIN (winner = smallest position among equal values),
// MODE_ROUTE (backward of max/min: a sum that keeps dOut[c,f] only where position route_pos won (c,f)) or
// MODE_HEADSUM (one multiplier per position and head, optional rank-1 row epilogue)
template <typename T, int LPR, int MODE>
__global__ void __launch_bounds__(FL_WARPS * 32, (MODE == MODE_SUM || MODE == MODE_HEADSUM) ? 6 : 4)
propagate_flat_kernel(const PropParams P) {
    constexpr bool EF = MODE == MODE_EFSUM;  // one multiplier per (position, feature)
    constexpr int EPC = Chunk<T>::N, NG = 32 / LPR, U = (MODE == MODE_ROUTE || EF) ? FL_U / 2 : FL_U;
    constexpr int MW = EF ? EPC : 1;
    constexpr bool ARG = MODE == MODE_MAX || MODE == MODE_MIN;
    const int L = P.chunk / NG;  // positions per lane group; P.chunk is 64, 128 or 256 here
    __shared__ FlatSmem<EPC, ARG> s_all[FL_WARPS];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int64_t c = (int64_t)blockIdx.x * FL_WARPS + wib;
    if (c >= P.nchunks) return;
    FlatSmem<EPC, ARG>& S = s_all[wib];
    const uint64_t pol_keep = policy_evict_last(), pol_stream = policy_evict_first();
    const int64_t cs = c * P.chunk;
    const int n = (int)((cs + P.chunk < P.E ? cs + P.chunk : P.E) - cs);  // 1..256 positions
    const int g = lane / LPR, li = lane % LPR;
    const bool col_lane = li < P.nvec;  // lanes past a narrow row gather chunk 0 and never store
    char* const outb = reinterpret_cast<char*>(P.out);

    // a finished row: values (already scaled) and, for max/min, winner positions of 16-byte column ci
    auto store_row = [&](int row, int ci, float* v, const int32_t* wa) {
        if (MODE == MODE_HEADSUM && P.epi_l) {  // rank-1 row epilogue of the per-head mode
            const int h = (ci * EPC) / P.fph;  // a 16-byte chunk lies inside one head
            const float el = P.epi_l[(size_t)row * P.H + h], er = P.epi_r[(size_t)row * P.H + h];
#pragma unroll
            for (int j = 0; j < EPC; ++j) v[j] += el * P.epi_a[ci * EPC + j] + er * P.epi_b[ci * EPC + j];
        }
        row_epilogue<T>(P, row, ci, v);
        st_stream16(outb + (size_t)row * P.out_ld + (size_t)ci * 16, Chunk<T>::pack(v));
        if (ARG && P.argmax) {
            int32_t* ap = P.argmax + (size_t)row * P.F + (size_t)ci * EPC;
#pragma unroll
            for (int j = 0; j < EPC; j += 4) *reinterpret_cast<int4*>(ap + j) = make_int4(wa[j], wa[j + 1], wa[j + 2], wa[j + 3]);
        }
    };
    // a row without edges: zeros (and no winner)
    auto store_empty_row = [&](int row) {
        for (int ci = lane; ci < P.nvec; ci += 32) {
            float z[EPC];
            int32_t none[EPC];
#pragma unroll
            for (int j = 0; j < EPC; ++j) { z[j] = 0.f; none[j] = -1; }
            store_row(row, ci, z, none);
        }
    };

    // ---- 1a. the row holding position cs: largest r with rowptr[r] <= cs (32-way search)
    int lo = 0, hi = P.N;  // rowptr[lo] <= cs < rowptr[hi]
    while (hi - lo > 1) {
        const int step = (hi - lo + 31) / 32;
        const int idx = min(lo + (lane + 1) * step, hi);
        const bool le = idx < hi && P.rowptr[idx] <= cs;
        const int k = __popc(__ballot_sync(0xffffffffu, le));
        const int nlo = lo + k * step;
        hi = min(nlo + step, hi);
        lo = nlo;
    }
    const int cur0 = lo;
    const int64_t rs0 = P.rowptr[cur0], re0 = P.rowptr[cur0 + 1];
    const bool row0_before = rs0 < cs;
    auto rel_end = [&](int64_t re) { return (int)((re - cs) < (int64_t)PF_SLAB + 1 ? (re - cs) : (int64_t)PF_SLAB + 1); };
    auto row_factor = [&](int64_t len) { return P.mean ? 1.0f / (float)(len > 1 ? len : 1) : 1.0f; };

    // ---- 1b. stage gathered rows and multipliers; start entries default to 0
    for (int i = lane; i < n; i += 32) {
        const int cc = P.col ? ld_hint_i32(P.col + cs + i, pol_stream) : (int)(cs + i);
        float w = P.w ? ld_hint_f32(P.w + cs + i, pol_stream) : 1.0f;
        if (P.gscale_rowptr) {
            const int64_t d = P.gscale_rowptr[cc + 1] - P.gscale_rowptr[cc];
            w = w / (float)(d > 1 ? d : 1);
        }
        int t = 0;
        if (MODE == MODE_ROUTE) t = ld_hint_i32(P.route_pos + cs + i, pol_stream);
        if (MODE == MODE_HEADSUM) t = P.wh_index ? ld_hint_i32(P.wh_index + cs + i, pol_stream) : (int)(cs + i);  // E < 2^31 here
        S.e[i] = make_int4(cc, 0, __float_as_int(w), t);
    }
    if (lane == 0) { S.srow[0] = cur0; S.send[0] = rel_end(re0); S.sinv[0] = row_factor(re0 - rs0); }
    if (lane < 8) { S.hk[lane] = -1; S.hclosed[lane] = 0; S.tk[lane] = -1; }
    __syncwarp();

    // ---- 1c. rows after cur0 that start inside the chunk: mark the ones that have edges.  (Rows without
    // edges are written by the row scan below; a run of them is jumped over with one search.)
    for (int rb = cur0 + 1; rb < P.N;) {
        const int r = rb + lane;
        int64_t rs = 0, re = 0;
        bool live = false;
        if (r < P.N) {
            rs = P.rowptr[r];
            live = rs < cs + n;
            if (live) re = P.rowptr[r + 1];
        }
        if (live && re > rs) {
            const int k = (int)(rs - cs);
            S.srow[k] = r;
            S.send[k] = rel_end(re);
            S.sinv[k] = row_factor(re - rs);
            S.e[k].y = k;
        }
        // rowptr is non-decreasing: once a lane is past the chunk (or past the last row) so are all later rows
        if (!__all_sync(0xffffffffu, live)) break;
        if (__all_sync(0xffffffffu, re == rs)) rb = first_row_ending_after(P.rowptr, rb + 32, P.N, __shfl_sync(0xffffffffu, rs, 0), lane);
        else rb += 32;
    }
    scan_empty_rows(P.rowptr, P.N, c, P.nchunks, lane, store_empty_row);
    __syncwarp();

    // ---- 1d. prefix maximum of the start marks: lane owns positions 8*lane .. 8*lane+7
    {
        int m[8];
        int run = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = lane * 8 + q;
            const int v = i < n ? S.e[i].y : 0;
            run = max(run, v);
            m[q] = run;
        }
        int incl = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl = max(incl, t);
        }
        int before = __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == 0) before = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = lane * 8 + q;
            if (i < n) S.e[i].y = max(before, m[q]);
        }
    }
    __syncwarp();

    // ---- 2. gather: run [a, b) of this lane group
    const int a = g * L, b = min(a + L, n);
    const char* Xl = reinterpret_cast<const char*>(P.X) + (size_t)(col_lane ? li : 0) * 16;
    float acc[EPC];
    int32_t arg[ARG ? EPC : 1];
    auto clear = [&]() {
#pragma unroll
        for (int j = 0; j < EPC; ++j) {
            acc[j] = 0.f;
            if (ARG) arg[j] = -1;
        }
    };
    clear();
    int curk = -1;
    // only the run's first row can have begun before the run (in an earlier run or chunk)
    bool first_began_before = a < b && (S.e[a].y < a || (a == 0 && row0_before));
    auto park = [&](float* dv, int32_t* da) {  // accumulator -> this lane's slot of a head / tail array
#pragma unroll
        for (int j = 0; j < EPC; ++j) {
            dv[lane * EPC + j] = acc[j];
            if (ARG) da[lane * EPC + j] = arg[j];
        }
    };
    // the row of start entry k ends inside this run
    auto flush = [&](int k) {
        if (first_began_before) {
            park(S.head, S.head_a);
            if (li == 0) { S.hk[g] = k; S.hclosed[g] = 1; }
            first_began_before = false;
        } else if (col_lane) {
            float v[EPC];
            const float f = S.sinv[k];
#pragma unroll
            for (int j = 0; j < EPC; ++j) v[j] = ARG ? acc[j] : acc[j] * f;
            store_row(S.srow[k], li, v, arg);
        }
    };
    const int32_t* const route_l = (MODE == MODE_ROUTE) ? P.route_arg + (size_t)(col_lane ? li : 0) * EPC : nullptr;
    // per-head mode: this lane's head column of the [E,H] multiplier matrix, at the chunk's first position
    const float* const wh_l = (MODE == MODE_HEADSUM) ? P.wh + ((col_lane ? li : 0) * EPC) / P.fph : nullptr;
    // per-feature mode: this lane's feature columns of the [E,F] multiplier matrix, at the chunk's first position
    const float* const ef_l = EF ? P.ef + (size_t)cs * P.ef_ld + (size_t)(col_lane ? li : 0) * EPC : nullptr;
    auto load_ef = [&](int pos_in_chunk, float* dst) {
        const float4* q = reinterpret_cast<const float4*>(ef_l + (size_t)pos_in_chunk * P.ef_ld);
#pragma unroll
        for (int t = 0; t < MW / 4; ++t) {
            const float4 a4 = __ldcs(q + t);
            dst[4 * t] = a4.x; dst[4 * t + 1] = a4.y; dst[4 * t + 2] = a4.z; dst[4 * t + 3] = a4.w;
        }
    };
    for (int i = a; i < b; i += U) {
        uint4 buf[U];
        float hw[(MODE == MODE_HEADSUM || EF) ? U : 1][MW];
        int4 win[MODE == MODE_ROUTE ? U : 1][MODE == MODE_ROUTE ? EPC / 4 : 1];
        const int nu = min(U, b - i);  // U except at the ragged end of the last chunk
        if (nu == U) {
            int cols[U];
#pragma unroll
            for (int u = 0; u < U; ++u) cols[u] = S.e[i + u].x;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                buf[u] = ld_hint16(Xl + (size_t)(uint32_t)cols[u] * P.x_ld, pol_keep);
                if (MODE == MODE_HEADSUM) hw[MODE == MODE_HEADSUM ? u : 0][0] = __ldg(wh_l + (size_t)(uint32_t)S.e[i + u].w * P.H);
                if (EF) load_ef(i + u, hw[EF ? u : 0]);
                if (MODE == MODE_ROUTE) {
#pragma unroll
                    for (int q = 0; q < EPC / 4; ++q)
                        win[MODE == MODE_ROUTE ? u : 0][MODE == MODE_ROUTE ? q : 0] =
                            __ldg(reinterpret_cast<const int4*>(route_l + (size_t)cols[u] * P.F) + q);
                }
            }
        } else {
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (u < nu) {
                    const int cc = S.e[i + u].x;
                    buf[u] = ld_hint16(Xl + (size_t)(uint32_t)cc * P.x_ld, pol_keep);
                    if (MODE == MODE_HEADSUM) hw[MODE == MODE_HEADSUM ? u : 0][0] = __ldg(wh_l + (size_t)(uint32_t)S.e[i + u].w * P.H);
                    if (EF) load_ef(i + u, hw[EF ? u : 0]);
                    if (MODE == MODE_ROUTE) {
#pragma unroll
                        for (int q = 0; q < EPC / 4; ++q)
                            win[MODE == MODE_ROUTE ? u : 0][MODE == MODE_ROUTE ? q : 0] =
                                __ldg(reinterpret_cast<const int4*>(route_l + (size_t)cc * P.F) + q);
                    }
                }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (u >= nu) break;
            const int4 e = S.e[i + u];
            if (e.y != curk) {
                if (curk >= 0) flush(curk);
                curk = e.y;
                clear();
            }
            float x[EPC];
            Chunk<T>::unpack(buf[u], x);
            const float w = __int_as_float(e.z);
            if (ARG) {
                const int32_t pos = (int32_t)(cs + i + u);
#pragma unroll
                for (int j = 0; j < EPC; ++j) {
                    const float m = P.w ? w * x[j] : x[j];
                    // positions ascend along a run: a strict comparison keeps the first of equal values
                    const bool take = arg[ARG ? j : 0] < 0 || (MODE == MODE_MAX ? m > acc[j] : m < acc[j]);
                    if (take) { acc[j] = m; arg[ARG ? j : 0] = pos; }
                }
            } else if (MODE == MODE_ROUTE) {
#pragma unroll
                for (int q = 0; q < EPC / 4; ++q) {
                    const int4 t = win[MODE == MODE_ROUTE ? u : 0][MODE == MODE_ROUTE ? q : 0];
                    if (t.x == e.w) acc[4 * q] = fmaf(w, x[4 * q], acc[4 * q]);
                    if (t.y == e.w) acc[4 * q + 1] = fmaf(w, x[4 * q + 1], acc[4 * q + 1]);
                    if (t.z == e.w) acc[4 * q + 2] = fmaf(w, x[4 * q + 2], acc[4 * q + 2]);
                    if (t.w == e.w) acc[4 * q + 3] = fmaf(w, x[4 * q + 3], acc[4 * q + 3]);
                }
            } else if (EF) {
#pragma unroll
                for (int j = 0; j < EPC; j += 2)
                    fma2(acc[j], acc[j + 1], x[j], x[j + 1], hw[EF ? u : 0][EF ? j : 0] * w, hw[EF ? u : 0][EF ? j + 1 : 0] * w);
            } else {
                // w = 1 in the per-head mode unless the gathered rows are rescaled (backward of the mean)
                const float m = (MODE == MODE_HEADSUM) ? hw[MODE == MODE_HEADSUM ? u : 0][0] * w : w;
#pragma unroll
                for (int j = 0; j < EPC; j += 2) fma2(acc[j], acc[j + 1], x[j], x[j + 1], m, m);
            }
        }
    }
    if (curk >= 0) {  // the run's last row
        if (S.send[curk] <= b) {
            flush(curk);
        } else {  // continues past the run
            if (first_began_before) park(S.head, S.head_a);
            else park(S.tail, S.tail_a);
            if (li == 0) {
                if (first_began_before) { S.hk[g] = curk; S.hclosed[g] = 0; }
                else S.tk[g] = curk;
            }
        }
    }
    __syncwarp();

    // ---- 3. stitch the runs in order; lanes 0..LPR-1 each own one 16-byte column
    int32_t tail_row = -1;
    if (lane < LPR) {
        float carry[EPC];
        int32_t carg[ARG ? EPC : 1];
        bool have = false, before_chunk = false;
        int ck = -1;
        auto write_partial = [&](int which) {
            if (!col_lane) return;
            const size_t off = ((size_t)c * 2 + which) * P.F + (size_t)lane * EPC;
#pragma unroll
            for (int j = 0; j < EPC; j += 4) {
                *reinterpret_cast<float4*>(P.part_val + off + j) = make_float4(carry[j], carry[j + 1], carry[j + 2], carry[j + 3]);
                if (ARG)
                    *reinterpret_cast<int4*>(P.part_arg + off + j) =
                        make_int4(carg[ARG ? j : 0], carg[ARG ? j + 1 : 0], carg[ARG ? j + 2 : 0], carg[ARG ? j + 3 : 0]);
            }
        };
        for (int gg = 0; gg < NG; ++gg) {
            const int hk = S.hk[gg];
            if (hk >= 0) {
                const int slot = (gg * LPR + lane) * EPC;
                if (have) {  // later positions: the carry wins ties
#pragma unroll
                    for (int j = 0; j < EPC; ++j) {
                        if (ARG) {
                            if (beats<MODE>(S.head[slot + j], S.head_a[ARG ? slot + j : 0], carry[j], carg[ARG ? j : 0])) {
                                carry[j] = S.head[slot + j];
                                carg[ARG ? j : 0] = S.head_a[ARG ? slot + j : 0];
                            }
                        } else {
                            carry[j] += S.head[slot + j];
                        }
                    }
                } else {  // only the chunk's first run can begin without a carry
#pragma unroll
                    for (int j = 0; j < EPC; ++j) {
                        carry[j] = S.head[slot + j];
                        if (ARG) carg[ARG ? j : 0] = S.head_a[ARG ? slot + j : 0];
                    }
                    before_chunk = true;
                    have = true;
                }
                ck = hk;
                if (S.hclosed[gg]) {
                    if (before_chunk) {
                        write_partial(0);
                    } else if (col_lane) {
                        float v[EPC];
                        const float f = S.sinv[ck];
#pragma unroll
                        for (int j = 0; j < EPC; ++j) v[j] = ARG ? carry[j] : carry[j] * f;
                        store_row(S.srow[ck], lane, v, carg);
                    }
                    have = false;
                }
            }
            const int tk = S.tk[gg];
            if (tk >= 0) {
                const int slot = (gg * LPR + lane) * EPC;
#pragma unroll
                for (int j = 0; j < EPC; ++j) {
                    carry[j] = S.tail[slot + j];
                    if (ARG) carg[ARG ? j : 0] = S.tail_a[ARG ? slot + j : 0];
                }
                have = true;
                before_chunk = false;
                ck = tk;
            }
        }
        if (have) {  // the row continues in the next chunk
            write_partial(before_chunk ? 0 : 1);
            if (!before_chunk) tail_row = S.srow[ck];
        }
    }
    if (lane == 0) P.tail_row[c] = tail_row;
}

// ------------------------------------------------------------------ edge-weight gradient (SDDMM)
// dW[p] = scale(i) * <X[col[p],:], dOut[i,:]> for p in row i.  Same chunking; every edge is
// independent, so no partials.  The dOut row stays in registers along the row.
struct SddmmParams {
    const int64_t* rowptr;
    const int32_t* col;
    const void* X;
    const void* dOut;
    float* dW;
    int32_t N;
    int64_t E;
    int nvec;
    int mean;
    int64_t nchunks;
    int H, lph;  // lph > 0: one result per (edge, head), a head = lph adjacent 16-byte chunks
};

template <typename T, int LPR, int VPL>
__global__ void __launch_bounds__(PF_WARPS * 32)
sddmm_chunk_kernel(const SddmmParams P) {
    constexpr int EPC = Chunk<T>::N;
    constexpr int NG = 32 / LPR;
    constexpr int U = (LPR >= 16) ? (8 / VPL) : 4;
    const int lane = threadIdx.x & 31, g = lane / LPR, li = lane % LPR;
    const int64_t c = (int64_t)blockIdx.x * PF_WARPS + (threadIdx.x >> 5);
    if (c >= P.nchunks) return;
    const int64_t cs = c * PF_SLAB;
    const int64_t ce = (cs + PF_SLAB < P.E) ? cs + PF_SLAB : P.E;
    if (cs >= ce) return;
    const uint64_t pol_keep = policy_evict_last(), pol_stream = policy_evict_first();
    const size_t row_bytes = (size_t)P.nvec * 16;
    const char* Xb = reinterpret_cast<const char*>(P.X);
    const char* Db = reinterpret_cast<const char*>(P.dOut);
    // row containing position cs: last row with rowptr[r] <= cs
    int r = lower_bound_i64(P.rowptr, P.N + 1, cs + 1) - 1;
    int64_t pos = cs;
    while (pos < ce) {
        r = first_row_ending_after(P.rowptr, r, P.N, pos, lane);  // skip rows that end at or before pos
        const int64_t rs = P.rowptr[r], re = P.rowptr[r + 1];
        const int64_t b = re < ce ? re : ce;
        float d[VPL][EPC];
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            const int ci = v * LPR + li;
            if (ci < P.nvec) {
                Chunk<T>::unpack(ld_hint16(Db + (size_t)r * row_bytes + (size_t)ci * 16, pol_stream), d[v]);
            } else {
#pragma unroll
                for (int j = 0; j < EPC; ++j) d[v][j] = 0.f;
            }
        }
        const float scale = P.mean ? 1.0f / (float)(re - rs) : 1.0f;
        for (int64_t base = pos; base < b; base += 32) {
            const int n = (int)((b - base) < 32 ? (b - base) : 32);
            int myc = lane < n ? ld_hint_i32(P.col + base + lane, pol_stream) : 0;
            const int rounds = (n + NG - 1) / NG;
            for (int r0 = 0; r0 < rounds; r0 += U) {
                uint4 buf[U][VPL];
                bool ok[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int e = (r0 + u) * NG + g;
                    ok[u] = e < n;
                    int cv = __shfl_sync(0xffffffffu, myc, e & 31);
                    if (ok[u]) {
#pragma unroll
                        for (int v = 0; v < VPL; ++v) {
                            const int ci = v * LPR + li;
                            if (ci < P.nvec) buf[u][v] = ld_hint16(Xb + (size_t)cv * row_bytes + (size_t)ci * 16, pol_keep);
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    float dotv[VPL];
#pragma unroll
                    for (int v = 0; v < VPL; ++v) {
                        dotv[v] = 0.f;
                        const int ci = v * LPR + li;
                        if (ok[u] && ci < P.nvec) {
                            float x[EPC];
                            Chunk<T>::unpack(buf[u][v], x);
#pragma unroll
                            for (int j = 0; j < EPC; ++j) dotv[v] = fmaf(x[j], d[v][j], dotv[v]);
                        }
                    }
                    const int64_t p = base + (r0 + u) * NG + g;
                    if (P.lph == 0) {  // one dot product per edge over the whole row
                        float dot = dotv[0];
#pragma unroll
                        for (int v = 1; v < VPL; ++v) dot += dotv[v];
#pragma unroll
                        for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                        if (ok[u] && li == 0) P.dW[p] = scale * dot;
                    } else {  // one per (edge, head): a head covers lph adjacent lanes
#pragma unroll
                        for (int v = 0; v < VPL; ++v) {
                            float dot = dotv[v];
                            for (int o = P.lph >> 1; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                            const int ci = v * LPR + li;
                            if (ok[u] && ci < P.nvec && (li % P.lph) == 0) P.dW[p * P.H + ci / P.lph] = scale * dot;
                        }
                    }
                }
            }
        }
        pos = b;
    }
}

// ------------------------------------------------------------------ flat SDDMM for short rows
// Same idea as propagate_flat_kernel: positions first, rows second.  The warp stages the gathered
// rows of its 256 positions and finds, by marking row starts and a prefix maximum, the row of every
// position; each lane group then takes a contiguous run and issues, per batch of 4 positions, the
// independent loads of X[col[p]] and, where the row changes, dOut[row(p)].  Every position is independent, so there are no partials and no second pass.
constexpr int SF_U = 4;

struct SddmmFlatSmem {
    int2 e[PF_SLAB];        // x: gathered row of X, y: start entry of the position's row
    int32_t srow[PF_SLAB];  // [k] row starting at position k of the chunk ([0]: the row holding position 0)
    float sinv[PF_SLAB];    // [k] 1, or 1 / row length for the mean
};

template <typename T, int LPR>
__global__ void __launch_bounds__(FL_WARPS * 32, 8)
sddmm_flat_kernel(const SddmmParams P) {
    constexpr int EPC = Chunk<T>::N, NG = 32 / LPR, U = SF_U, L = PF_SLAB / NG;
    __shared__ SddmmFlatSmem s_all[FL_WARPS];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int64_t c = (int64_t)blockIdx.x * FL_WARPS + wib;
    if (c >= P.nchunks) return;
    SddmmFlatSmem& S = s_all[wib];
    const uint64_t pol_keep = policy_evict_last(), pol_stream = policy_evict_first();
    const int64_t cs = c * PF_SLAB;
    const int n = (int)((cs + PF_SLAB < P.E ? cs + PF_SLAB : P.E) - cs);
    const int g = lane / LPR, li = lane % LPR;
    const bool col_lane = li < P.nvec;

    // the row holding position cs: largest r with rowptr[r] <= cs (32-way search)
    int lo = 0, hi = P.N;
    while (hi - lo > 1) {
        const int step = (hi - lo + 31) / 32;
        const int idx = min(lo + (lane + 1) * step, hi);
        const bool le = idx < hi && P.rowptr[idx] <= cs;
        const int k = __popc(__ballot_sync(0xffffffffu, le));
        const int nlo = lo + k * step;
        hi = min(nlo + step, hi);
        lo = nlo;
    }
    const int cur0 = lo;
    auto row_factor = [&](int64_t len) { return P.mean ? 1.0f / (float)(len > 1 ? len : 1) : 1.0f; };
    for (int i = lane; i < n; i += 32) S.e[i] = make_int2(ld_hint_i32(P.col + cs + i, pol_stream), 0);
    if (lane == 0) { S.srow[0] = cur0; S.sinv[0] = row_factor(P.rowptr[cur0 + 1] - P.rowptr[cur0]); }
    __syncwarp();
    for (int rb = cur0 + 1; rb < P.N;) {  // non-empty rows starting inside the chunk
        const int r = rb + lane;
        int64_t rs = 0, re = 0;
        bool live = false;
        if (r < P.N) {
            rs = P.rowptr[r];
            live = rs < cs + n;
            if (live) re = P.rowptr[r + 1];
        }
        if (live && re > rs) {
            const int k = (int)(rs - cs);
            S.srow[k] = r;
            S.sinv[k] = row_factor(re - rs);
            S.e[k].y = k;
        }
        if (!__all_sync(0xffffffffu, live)) break;
        // 32 rows without edges: jump over the rest of the run
        if (__all_sync(0xffffffffu, re == rs)) rb = first_row_ending_after(P.rowptr, rb + 32, P.N, __shfl_sync(0xffffffffu, rs, 0), lane);
        else rb += 32;
    }
    __syncwarp();
    {  // prefix maximum of the start marks: lane owns positions 8*lane .. 8*lane+7
        int m[8];
        int run = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = lane * 8 + q;
            run = max(run, i < n ? S.e[i].y : 0);
            m[q] = run;
        }
        int incl = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl = max(incl, t);
        }
        int before = __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == 0) before = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int i = lane * 8 + q;
            if (i < n) S.e[i].y = max(before, m[q]);
        }
    }
    __syncwarp();

    const int a = g * L, b = min(a + L, n);
    const size_t row_bytes = (size_t)P.nvec * 16;
    const char* Xl = reinterpret_cast<const char*>(P.X) + (size_t)(col_lane ? li : 0) * 16;
    const char* Dl = reinterpret_cast<const char*>(P.dOut) + (size_t)(col_lane ? li : 0) * 16;
    const int span = P.lph == 0 ? LPR : P.lph;  // lanes per result: the whole row, or one head
    const bool writer = col_lane && (li % span) == 0;
    const int head = P.lph == 0 ? 0 : li / P.lph, wstride = P.lph == 0 ? 1 : P.H;
    const uint32_t row_bytes32 = (uint32_t)row_bytes;
    int kprev = -1;   // start entry of the position before this batch
    uint4 dcur = make_uint4(0, 0, 0, 0);  // this lane's chunk of the current row of dOut: reloaded only when the row changes
    for (int i = a; i < a + L; i += U) {  // same trip count in every lane: the shuffles below are warp-wide
        uint4 xb[U], db[U];
        int k[U];
        bool fresh[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const bool ok = i + u < b;
            const int2 e = S.e[ok ? i + u : 0];
            k[u] = ok ? e.y : -1;
            fresh[u] = ok && k[u] != (u == 0 ? kprev : k[u - 1]);
            if (ok) xb[u] = ld_hint16(Xl + (size_t)((uint32_t)e.x) * row_bytes32, pol_keep);
            if (fresh[u]) db[u] = __ldg(reinterpret_cast<const uint4*>(Dl + (size_t)((uint32_t)S.srow[e.y]) * row_bytes32));
        }
        kprev = k[U - 1];
        static_assert(SF_U == 4, "the reductions below fold four positions at a time");
        float dot[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (fresh[u]) dcur = db[u];
            dot[u] = 0.f;
            if (k[u] >= 0 && col_lane) {
                float x[EPC], d[EPC];
                Chunk<T>::unpack(xb[u], x);
                Chunk<T>::unpack(dcur, d);
#pragma unroll
                for (int j = 0; j < EPC; ++j) dot[u] = fmaf(x[j], d[j], dot[u]);
            }
        }
        if (span >= 4) {
            // fold the four positions while reducing over the span lanes: the first two levels halve the values
            // a lane carries (2 + 1 shuffles), the rest reduce the one left; the quarter of the span a lane
            // sits in decides which position it ends up with: 6 shuffles for 32 lanes instead of 20
            const int h1 = span >> 1, h2 = span >> 2;
            const bool up1 = (li & h1) != 0, up2 = (li & h2) != 0;
            const float s0 = up1 ? dot[0] : dot[2], s1 = up1 ? dot[1] : dot[3];
            const float r0 = (up1 ? dot[2] : dot[0]) + __shfl_xor_sync(0xffffffffu, s0, h1);
            const float r1 = (up1 ? dot[3] : dot[1]) + __shfl_xor_sync(0xffffffffu, s1, h1);
            float v = (up2 ? r1 : r0) + __shfl_xor_sync(0xffffffffu, up2 ? r0 : r1, h2);
            for (int o = span >> 3; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            const int mine = (up1 ? 2 : 0) + (up2 ? 1 : 0);  // the position of the batch this lane holds
            const int km = mine == 0 ? k[0] : mine == 1 ? k[1] : mine == 2 ? k[2] : k[3];
            // any lane of the span may end up holding a result (with whole-row results also a lane past a narrow row)
            if ((P.lph == 0 || col_lane) && (li & (h2 - 1)) == 0 && km >= 0) P.dW[(cs + i + mine) * wstride + head] = S.sinv[km] * v;
        } else {  // heads of one or two 16-byte chunks
#pragma unroll
            for (int u = 0; u < U; ++u) {
                float v = dot[u];
                for (int o = span >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (k[u] >= 0 && writer) P.dW[(cs + i + u) * wstride + head] = S.sinv[k[u]] * v;
            }
        }
    }
}

// ------------------------------------------------------------------ host dispatch
bool pick_shape(int nvec, int* lpr, int* vpl) {
    if (nvec < 1 || nvec > 128) return false;
    if (nvec <= 4) { *lpr = 4; *vpl = 1; }
    else if (nvec <= 8) { *lpr = 8; *vpl = 1; }
    else if (nvec <= 16) { *lpr = 16; *vpl = 1; }
    else if (nvec <= 32) { *lpr = 32; *vpl = 1; }
    else if (nvec <= 64) { *lpr = 32; *vpl = 2; }
    else { *lpr = 32; *vpl = 4; }
    return true;
}

template <typename T, int MODE>
static void launch_chunks(const PropParams& P, int lpr, int vpl, cudaStream_t st) {
    const int grid = (int)ceil_div(P.nchunks, PF_WARPS);
    const int thr = PF_WARPS * 32;
#define GNN_PF_CASE(L, V) \
    if (lpr == L && vpl == V) { propagate_chunk_kernel<T, L, V, MODE><<<grid, thr, 0, st>>>(P); }
    GNN_PF_CASE(4, 1) GNN_PF_CASE(8, 1) GNN_PF_CASE(16, 1) GNN_PF_CASE(32, 1) GNN_PF_CASE(32, 2) GNN_PF_CASE(32, 4)
#undef GNN_PF_CASE
    const int64_t threads = P.nchunks * P.nvec;
    propagate_fixup_kernel<T, MODE><<<(int)ceil_div(threads, 256), 256, 0, st>>>(P);
    if (P.fix_long) propagate_fixup_long_kernel<T, MODE><<<FIXL_BLOCKS, FIXL_THREADS, 0, st>>>(P);
}

// sum / mean / max / min over rows of at most 512 bytes on graphs small enough for one-slab chunks
template <typename T, int MODE>
static void launch_flat(const PropParams& P, int lpr, cudaStream_t st) {
    const int grid = (int)ceil_div(P.nchunks, FL_WARPS);
    const int thr = FL_WARPS * 32;
    switch (lpr) {
        case 4: propagate_flat_kernel<T, 4, MODE><<<grid, thr, 0, st>>>(P); break;
        case 8: propagate_flat_kernel<T, 8, MODE><<<grid, thr, 0, st>>>(P); break;
        case 16: propagate_flat_kernel<T, 16, MODE><<<grid, thr, 0, st>>>(P); break;
        default: propagate_flat_kernel<T, 32, MODE><<<grid, thr, 0, st>>>(P); break;
    }
    const int64_t threads = P.nchunks * P.nvec;
    propagate_fixup_kernel<T, MODE><<<(int)ceil_div(threads, 256), 256, 0, st>>>(P);
    if (P.fix_long) propagate_fixup_long_kernel<T, MODE><<<FIXL_BLOCKS, FIXL_THREADS, 0, st>>>(P);
}

template <typename T>
static void launch_mode(const PropParams& P, int mode, int lpr, int vpl, cudaStream_t st) {
    if (vpl == 1 && P.chunk <= PF_SLAB && P.E > 0) {
        if (mode == MODE_SUM) launch_flat<T, MODE_SUM>(P, lpr, st);
        else if (mode == MODE_HEADSUM) launch_flat<T, MODE_HEADSUM>(P, lpr, st);
        else if (mode == MODE_EFSUM) launch_flat<T, MODE_EFSUM>(P, lpr, st);
        else if (mode == MODE_MAX) launch_flat<T, MODE_MAX>(P, lpr, st);
        else if (mode == MODE_MIN) launch_flat<T, MODE_MIN>(P, lpr, st);
        else launch_flat<T, MODE_ROUTE>(P, lpr, st);
        return;
    }
    switch (mode) {
        case MODE_SUM: launch_chunks<T, MODE_SUM>(P, lpr, vpl, st); break;
        case MODE_MAX: launch_chunks<T, MODE_MAX>(P, lpr, vpl, st); break;
        case MODE_MIN: launch_chunks<T, MODE_MIN>(P, lpr, vpl, st); break;
        case MODE_HEADSUM: launch_chunks<T, MODE_HEADSUM>(P, lpr, vpl, st); break;
        case MODE_EFSUM: launch_chunks<T, MODE_EFSUM>(P, lpr, vpl, st); break;
        default: launch_chunks<T, MODE_ROUTE>(P, lpr, vpl, st); break;
    }
}

template <typename T>
static void launch_sddmm(const SddmmParams& P, int lpr, int vpl, cudaStream_t st) {
    if (vpl == 1) {  // positions first
        const int grid = (int)ceil_div(P.nchunks, FL_WARPS);
        switch (lpr) {
            case 4: sddmm_flat_kernel<T, 4><<<grid, FL_WARPS * 32, 0, st>>>(P); break;
            case 8: sddmm_flat_kernel<T, 8><<<grid, FL_WARPS * 32, 0, st>>>(P); break;
            case 16: sddmm_flat_kernel<T, 16><<<grid, FL_WARPS * 32, 0, st>>>(P); break;
            default: sddmm_flat_kernel<T, 32><<<grid, FL_WARPS * 32, 0, st>>>(P); break;
        }
        return;
    }
    const int grid = (int)ceil_div(P.nchunks, PF_WARPS);
    const int thr = PF_WARPS * 32;
#define GNN_SD_CASE(L, V) \
    if (lpr == L && vpl == V) { sddmm_chunk_kernel<T, L, V><<<grid, thr, 0, st>>>(P); }
    GNN_SD_CASE(4, 1) GNN_SD_CASE(8, 1) GNN_SD_CASE(16, 1) GNN_SD_CASE(32, 1) GNN_SD_CASE(32, 2) GNN_SD_CASE(32, 4)
#undef GNN_SD_CASE
}

// edges per warp: four slabs once there are enough edges to fill the machine many times over (fewer
// partial rows to write and re-read), one slab below that, and a half or a quarter slab on graphs so
// small that whole slabs would leave most SMs without a warp
#ifndef PF_BIG_E
#define PF_BIG_E ((int64_t)8 * 1024 * 1024)
#endif
static int chunk_edges(int64_t E) {
    if (E >= PF_BIG_E) return 4 * PF_SLAB;
    if (E >= 512 * 1024) return PF_SLAB;
    return E >= 128 * 1024 ? PF_SLAB / 2 : PF_SLAB / 4;
}
static int64_t num_chunks(int64_t E) { return E > 0 ? ceil_div(E, chunk_edges(E)) : 1; }
static int64_t num_slabs(int64_t E) { return E > 0 ? ceil_div(E, PF_SLAB) : 1; }

// Large graphs of low mean degree: almost every row is a handful of positions, and the position-first kernel
// (one-slab chunks) beats the row walk at any size.  Measured on uniform random graphs of 1-8 M rows (times in
// ms, row walk / positions first, 4 M rows): mean degree 4: 64-byte rows 1.34 / 0.70, 256-byte bf16 rows
// 2.03 / 1.08, 512-byte rows 2.21 / 1.91; mean degree 8: 1.55 / 1.26, 2.92 / 1.93, 3.10 / 3.44; mean degree 16:
// 2.37 / 2.39, 4.06 / 3.61, 5.46 / 6.48.  fp32 rows walk faster (one predicated loop per row), so their
// crossover is lower: 256-byte rows 1.70 / 1.08 at mean degree 4, 1.84 / 1.92 at 8.  Graphs with hub rows
// and a higher mean degree keep the row walk (hubs are where it is strongest).
// Sums over rows of 256 bytes and more on graphs of 0.5-4 M edges: a one-slab chunk of such rows is 64-128 KB of
// gathers behind one warp, and the graph fills the machine only one to five times, so half slabs balance better
// (1.36 M edges, 128 features: fp32 sums 129 -> 113 us, backward of the mean 145 -> 125 us, bf16 75 -> 74 us).
// Not for narrower rows (the 32-byte rows of the attention backward lose 2 %), nor for max / min and the
// per-head mode (+5..8 %), nor where the mean degree says that hub rows carry the edges: every extra cut of a hub
// row is one more partial row (R-MAT graph of 1.6 M edges, mean degree 16, 512-byte rows: 148 -> 167 us).
constexpr int64_t SUM_HALF_SLAB_BELOW = (int64_t)4 * 1024 * 1024;
static bool sum_half_slab(int mode, int32_t N, int64_t E, int nvec) {
    return mode == MODE_SUM && nvec >= 16 && nvec <= 32 && E >= 512 * 1024 && E < SUM_HALF_SLAB_BELOW && E <= (int64_t)12 * N;
}

static bool flat_by_degree(int mode, int32_t N, int64_t E, int nvec, int elem_bytes) {
    if (mode != MODE_SUM || nvec > 32 || N <= 0 || E <= 0) return false;
    const double d = (double)E / (double)N;
    if (nvec > 16) return d <= 4.0;
    return elem_bytes == 2 ? d <= 12.0 : d <= 6.0;
}

struct PfWs {
    int32_t* tail_row;
    float* part_val;
    int32_t* part_arg;
    size_t bytes;
};
static PfWs pf_carve(void* ws, int64_t E, int F, bool with_arg) {
    PfWs w;
    // sums over rows that the position-first kernel can take (at most 512 bytes: F <= 256 whatever the type) may
    // run on one-slab chunks at any size (flat_by_degree): room for the larger of the two chunk counts
    int64_t nc = num_chunks(E);
    if (F <= 256 && num_slabs(E) > nc) nc = num_slabs(E);
    if (E < SUM_HALF_SLAB_BELOW && ceil_div(E, PF_SLAB / 2) > nc) nc = ceil_div(E, PF_SLAB / 2);
    char* p = (char*)ws;
    size_t off = 0;
    w.tail_row = (int32_t*)(p + off); off += up256((size_t)nc * 4);
    w.part_val = (float*)(p + off); off += up256((size_t)nc * 2 * F * 4);
    w.part_arg = (int32_t*)(p + off); if (with_arg) off += up256((size_t)nc * 2 * F * 4);
    w.bytes = off;
    return w;
}

size_t chunked_workspace(int64_t E, int F, bool with_arg) { return pf_carve(nullptr, E, F, with_arg).bytes; }

bool chunked_is_flat(int64_t E, int F, gnn_dtype dtype) {
    const int nvec = F * elem_size(dtype) / 16;
    return E > 0 && chunk_edges(E) <= PF_SLAB && nvec >= 1 && nvec <= 32;
}

gnn_status run_chunked(const char* who, int mode, int32_t N, int64_t E, const int64_t* rowptr,
                       const int32_t* col, const float* w, const void* X, void* out,
                       int32_t* argmax, const int64_t* gscale_rowptr, const int32_t* route_arg,
                       const int32_t* route_pos, int mean, int F, gnn_dtype dtype, void* ws,
                       size_t ws_bytes, cudaStream_t st, const HeadExtra* hx, const RowExtra* rx) {
    const int s = elem_size(dtype);
    GNN_REQUIRE(F > 0 && ((size_t)F * s) % 16 == 0, GNN_ERR_UNSUPPORTED,
                "%s: F*sizeof(element) = %d must be a multiple of 16 bytes", who, F * s);
    const int nvec = F * s / 16;
    int lpr, vpl;
    GNN_REQUIRE(pick_shape(nvec, &lpr, &vpl), GNN_ERR_UNSUPPORTED,
                "%s: feature rows wider than 2048 bytes are not supported (F=%d)", who, F);
    GNN_REQUIRE(aligned16(X) && aligned16(out), GNN_ERR_INVALID_ARG, "%s: feature matrices must be 16-byte aligned", who);
    GNN_REQUIRE(E >= 0 && E < ((int64_t)1 << 31) - 4 * PF_SLAB, GNN_ERR_UNSUPPORTED, "%s: positions must fit 32 bits (E < 2^31)", who);
    const bool with_arg = (mode == MODE_MAX || mode == MODE_MIN);
    PfWs wsv = pf_carve(ws, E, F, with_arg);
    GNN_REQUIRE(ws && ws_bytes >= wsv.bytes && aligned16(ws), GNN_ERR_WORKSPACE_TOO_SMALL,
                "%s: workspace of %zu bytes (16-byte aligned) needed, %zu given", who, wsv.bytes, ws_bytes);
    if (N == 0) return GNN_OK;
    PropParams P;
    P.rowptr = rowptr; P.col = col; P.w = w; P.X = X; P.out = out; P.argmax = argmax;
    P.gscale_rowptr = gscale_rowptr; P.route_arg = route_arg; P.route_pos = route_pos;
    P.N = N; P.E = E; P.nvec = nvec; P.F = F; P.mean = mean; P.chunk = chunk_edges(E); P.nchunks = num_chunks(E);
    if (flat_by_degree(mode, N, E, nvec, s)) { P.chunk = P.chunk < PF_SLAB ? P.chunk : PF_SLAB; P.nchunks = ceil_div(E, (int64_t)P.chunk); }
    if (sum_half_slab(mode, N, E, nvec)) { P.chunk = PF_SLAB / 2; P.nchunks = ceil_div(E, (int64_t)P.chunk); }
    P.tail_row = wsv.tail_row; P.part_val = wsv.part_val; P.part_arg = wsv.part_arg;
    // also where the mean row is long (pooling over a few large graphs), and from fewer chunks on for max / min, whose
    // walk compares (value, position) pairs one partial row after the other
    const bool long_mean = E / N > (int64_t)FIX_LONG * P.chunk && P.nchunks > FIX_LONG;
    P.fix_long = (P.nchunks >= (with_arg ? FIXL_MIN_CHUNKS_ARG : FIXL_MIN_CHUNKS) || long_mean) ? 1 : 0;
    P.wh = nullptr; P.wh_index = nullptr; P.H = 1; P.fph = F; P.epi_l = P.epi_r = P.epi_a = P.epi_b = nullptr;
    if (hx) {
        const int epc = 16 / s;
        GNN_REQUIRE(mode == MODE_HEADSUM && (hx->wh || E == 0) && hx->H >= 1 && F % hx->H == 0 && (F / hx->H) % epc == 0, GNN_ERR_UNSUPPORTED,
                    "%s: per-head weights need F divisible by H and F/H a multiple of %d elements", who, epc);
        GNN_REQUIRE(!hx->wh_index || chunked_is_flat(E, F, dtype), GNN_ERR_INVALID_ARG, "%s: indexed per-head weights need the flat kernel", who);
        P.wh = hx->wh; P.wh_index = hx->wh_index; P.H = hx->H; P.fph = F / hx->H;
        P.epi_l = hx->epi_l; P.epi_r = hx->epi_r; P.epi_a = hx->epi_a; P.epi_b = hx->epi_b;
    } else {
        GNN_REQUIRE(mode != MODE_HEADSUM, GNN_ERR_INVALID_ARG, "%s: per-head mode without weights", who);
    }
    P.x_ld = P.out_ld = (uint32_t)nvec * 16;
    P.ef = nullptr; P.ef_ld = 0; P.has_epi = 0; P.agg_c = 1.0f; P.self_c = 0.f; P.self_mode = GNN_SELF_ALWAYS; P.relu = 0;
    P.self_X = nullptr; P.self_ld = (uint32_t)nvec * 16; P.self_rowptr = rowptr; P.bias = nullptr;
    if (rx) {
        GNN_REQUIRE(mode == MODE_EFSUM ? (rx->ef != nullptr || E == 0) : rx->ef == nullptr, GNN_ERR_INVALID_ARG,
                    "%s: per-feature multipliers and mode disagree", who);
        GNN_REQUIRE(!rx->ef || (rx->ef_ld >= F && rx->ef_ld % 4 == 0 && aligned16(rx->ef)), GNN_ERR_INVALID_ARG,
                    "%s: per-feature multipliers must be 16-byte aligned rows of at least F floats", who);
        GNN_REQUIRE(!rx->self_X || aligned16(rx->self_X), GNN_ERR_INVALID_ARG, "%s: the self-term matrix must be 16-byte aligned", who);
        GNN_REQUIRE(rx->self_mode >= GNN_SELF_ALWAYS && rx->self_mode <= GNN_SELF_IF_NONEMPTY, GNN_ERR_INVALID_ARG, "%s: bad self mode", who);
        P.ef = rx->ef; P.ef_ld = rx->ef_ld;
        P.agg_c = rx->agg_c; P.self_X = rx->self_X; P.self_c = rx->self_c; P.self_mode = rx->self_mode;
        if (rx->self_rowptr) P.self_rowptr = rx->self_rowptr;
        P.bias = rx->bias; P.relu = rx->relu;
        P.has_epi = (rx->agg_c != 1.0f || rx->self_X || rx->bias || rx->relu) ? 1 : 0;
    } else {
        GNN_REQUIRE(mode != MODE_EFSUM, GNN_ERR_INVALID_ARG, "%s: per-feature mode without multipliers", who);
    }
    // Column slabs: when rows are wider than 512 bytes and the gathered matrix is far larger than L2,
    // sum reductions run one 512-byte column slab at a time.  Each pass re-reads the index stream but
    // gathers from a 4x (2x) narrower matrix, of which 4x (2x) more rows stay in L2: fewer DRAM
    // re-reads and a shorter run in total.  The result is the same arithmetic in the same order.
    // ... and on graphs small enough for one-slab chunks every pass takes the position-first kernel, which rows over
    // 512 bytes otherwise cannot (1.36 M edges: 1024-byte fp32 rows 267 us as one row walk, 2 x 115 us as two passes)
    const bool slabs = mode == MODE_SUM && nvec > 32 && nvec % 32 == 0 &&
                       ((size_t)N * nvec * 16 > ((size_t)256 << 20) || (E > 0 && chunk_edges(E) <= PF_SLAB));
    if (slabs) {
        if (sum_half_slab(mode, N, E, 32)) { P.chunk = PF_SLAB / 2; P.nchunks = ceil_div(E, (int64_t)P.chunk); }  // the rule of 512-byte rows, per pass
        const int nslab = nvec / 32, fslab = F / nslab;
        P.nvec = 32; P.F = fslab;
        for (int sl = 0; sl < nslab; ++sl) {
            P.X = (const char*)X + (size_t)sl * 512;
            P.out = (char*)out + (size_t)sl * 512;
            if (rx && rx->self_X) P.self_X = (const char*)rx->self_X + (size_t)sl * 512;
            if (rx && rx->bias) P.bias = rx->bias + (size_t)sl * fslab;
            if (dtype == GNN_F32) launch_mode<float>(P, mode, 32, 1, st);
            else launch_mode<__nv_bfloat16>(P, mode, 32, 1, st);
        }
    } else if (dtype == GNN_F32) launch_mode<float>(P, mode, lpr, vpl, st);
    else launch_mode<__nv_bfloat16>(P, mode, lpr, vpl, st);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

// dW[p,h] = <X[col[p],h,:], dOut[i,h,:]> for p in row i: the per-head edge dot products of the
// attention backward pass
gnn_status sddmm_heads(const char* who, const gnn_csr* g, const void* X, const void* dOut, int H, int C,
                       gnn_dtype dtype, float* dW_EH, cudaStream_t st, int mean) {
    const int s = elem_size(dtype), F = H * C;
    GNN_REQUIRE(((size_t)C * s) % 16 == 0, GNN_ERR_UNSUPPORTED, "%s: a head must be a multiple of 16 bytes wide", who);
    const int lph = C * s / 16;
    GNN_REQUIRE(lph <= 32 && (lph & (lph - 1)) == 0, GNN_ERR_UNSUPPORTED,
                "%s: a head must span a power-of-two number (<= 32) of 16-byte chunks (C=%d)", who, C);
    int lpr, vpl;
    GNN_REQUIRE(pick_shape(F * s / 16, &lpr, &vpl), GNN_ERR_UNSUPPORTED, "%s: feature rows wider than 2048 bytes", who);
    GNN_REQUIRE(lph <= lpr, GNN_ERR_UNSUPPORTED, "%s: head wider than the row layout", who);
    GNN_REQUIRE(aligned16(X) && aligned16(dOut), GNN_ERR_INVALID_ARG, "%s: feature matrices must be 16-byte aligned", who);
    if (g->E == 0) return GNN_OK;
    SddmmParams S;
    S.rowptr = g->rowptr; S.col = g->col; S.X = X; S.dOut = dOut; S.dW = dW_EH;
    S.N = g->N; S.E = g->E; S.nvec = F * s / 16; S.mean = mean; S.nchunks = num_slabs(g->E); S.H = H; S.lph = lph;
    if (dtype == GNN_F32) launch_sddmm<float>(S, lpr, vpl, st);
    else launch_sddmm<__nv_bfloat16>(S, lpr, vpl, st);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

// one dot product per edge (H == 1; scaled by 1 / row length if mean) or per edge and head
gnn_status run_sddmm(const char* who, const gnn_csr* g, const void* X, const void* D, int H, int C, int mean,
                     gnn_dtype dtype, float* dW, cudaStream_t st) {
    if (H > 1) {
        return sddmm_heads(who, g, X, D, H, C, dtype, dW, st, mean);
    }
    const int s = elem_size(dtype), F = C;
    GNN_REQUIRE(F > 0 && ((size_t)F * s) % 16 == 0, GNN_ERR_UNSUPPORTED, "%s: F*sizeof(element) must be a multiple of 16 bytes", who);
    int lpr, vpl;
    GNN_REQUIRE(pick_shape(F * s / 16, &lpr, &vpl), GNN_ERR_UNSUPPORTED, "%s: feature rows wider than 2048 bytes", who);
    GNN_REQUIRE(aligned16(X) && aligned16(D), GNN_ERR_INVALID_ARG, "%s: feature matrices must be 16-byte aligned", who);
    if (g->E == 0) return GNN_OK;
    SddmmParams S;
    S.rowptr = g->rowptr; S.col = g->col; S.X = X; S.dOut = D; S.dW = dW;
    S.N = g->N; S.E = g->E; S.nvec = F * s / 16; S.mean = mean; S.nchunks = num_slabs(g->E); S.H = 1; S.lph = 0;
    if (dtype == GNN_F32) launch_sddmm<float>(S, lpr, vpl, st);
    else launch_sddmm<__nv_bfloat16>(S, lpr, vpl, st);
    GNN_CHECK_LAUNCH(who);
    return GNN_OK;
}

// ------------------------------------------------------------------ built-in scratch
// Scratch for gnn_propagate_fused_static: lives in the library image, so every GPU that loads the
// library carries these bytes until the process exits.  Host code must not hand this name to a
// kernel: on the host it is only a handle for cudaGetSymbolAddress.
constexpr size_t STATIC_WS_BYTES = (size_t)8 << 20;  // 8 MiB
static __device__ __align__(256) unsigned char g_static_ws[STATIC_WS_BYTES];

constexpr int STATIC_MAX_DEVICES = 64;
static void* g_static_ws_addr[STATIC_MAX_DEVICES];  // device address of g_static_ws, per device ordinal
static std::mutex g_static_ws_mutex;

// device address of the built-in scratch on the current device (looked up once per device)
static gnn_status static_ws_address(const char* who, void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "%s: cudaGetDevice: %s", who, cudaGetErrorString(e));
    GNN_REQUIRE(dev >= 0 && dev < STATIC_MAX_DEVICES, GNN_ERR_UNSUPPORTED, "%s: device ordinal %d not supported", who, dev);
    std::lock_guard<std::mutex> lock(g_static_ws_mutex);
    if (!g_static_ws_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_ws);
        if (e != cudaSuccess || !p)
            GNN_FAIL(GNN_ERR_CUDA, "%s: cudaGetSymbolAddress failed: %s", who, cudaGetErrorString(e));
        g_static_ws_addr[dev] = p;
    }
    *out = g_static_ws_addr[dev];
    return GNN_OK;
}

}  // namespace gnn

using namespace gnn;

extern "C" {

size_t gnn_propagate_fused_workspace(int64_t E, int F, gnn_op op) {
    if (E < 0 || F <= 0) return 0;
    // MAX/MIN keep winner positions beside the partial values; their backward needs values
    // only, so the forward size always suffices for the backward call
    return chunked_workspace(E, F, op == GNN_MAX || op == GNN_MIN);
}

gnn_status gnn_propagate_fused(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* X,
                               const float* w_csr, int F, gnn_dtype dtype, void* out,
                               int32_t* argmax, void* ws, size_t ws_bytes, gnn_stream stream) {
    GNN_REQUIRE(g && g->rowptr && X && out, GNN_ERR_INVALID_ARG, "gnn_propagate_fused: null argument");
    GNN_REQUIRE(g->E == 0 || g->col, GNN_ERR_INVALID_ARG, "gnn_propagate_fused: null col");
    GNN_REQUIRE(msg == GNN_MSG_COPY_XJ || msg == GNN_MSG_E_MUL_XJ, GNN_ERR_UNSUPPORTED,
                "gnn_propagate_fused: message must be COPY_XJ or E_MUL_XJ");
    GNN_REQUIRE(msg == GNN_MSG_COPY_XJ || w_csr, GNN_ERR_INVALID_ARG, "gnn_propagate_fused: E_MUL_XJ needs w_csr");
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "gnn_propagate_fused: bad dtype");
    GNN_REQUIRE(op >= GNN_SUM && op <= GNN_MIN, GNN_ERR_INVALID_ARG, "gnn_propagate_fused: bad op");
    GNN_REQUIRE(!argmax || aligned16(argmax), GNN_ERR_INVALID_ARG, "gnn_propagate_fused: argmax must be 16-byte aligned");
    const float* w = (msg == GNN_MSG_E_MUL_XJ) ? w_csr : nullptr;
    const int mode = op == GNN_MAX ? MODE_MAX : op == GNN_MIN ? MODE_MIN : MODE_SUM;
    return run_chunked("gnn_propagate_fused", mode, g->N, g->E, g->rowptr, g->col, w, X, out,
                       argmax, nullptr, nullptr, nullptr, op == GNN_MEAN, F, dtype, ws, ws_bytes,
                       as_stream(stream));
}

gnn_status gnn_propagate_fused_backward(const gnn_csr* g, gnn_msg msg, gnn_op op,
                                        const void* dOut, const void* X, const float* w_csrT,
                                        const int32_t* argmax, int F, gnn_dtype dtype, void* dX,
                                        float* dW, void* ws, size_t ws_bytes, gnn_stream stream) {
    const char* who = "gnn_propagate_fused_backward";
    GNN_REQUIRE(g && g->rowptr && g->rowptrT && dOut, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(g->E == 0 || (g->col && g->colT), GNN_ERR_INVALID_ARG, "%s: null col", who);
    GNN_REQUIRE(msg == GNN_MSG_COPY_XJ || msg == GNN_MSG_E_MUL_XJ, GNN_ERR_UNSUPPORTED,
                "%s: message must be COPY_XJ or E_MUL_XJ", who);
    GNN_REQUIRE(dtype == GNN_F32 || dtype == GNN_BF16, GNN_ERR_INVALID_ARG, "%s: bad dtype", who);
    GNN_REQUIRE(op >= GNN_SUM && op <= GNN_MIN, GNN_ERR_INVALID_ARG, "%s: bad op", who);
    const bool mm = (op == GNN_MAX || op == GNN_MIN);
    cudaStream_t st = as_stream(stream);
    if (dX) {
        GNN_REQUIRE(msg == GNN_MSG_COPY_XJ || w_csrT, GNN_ERR_INVALID_ARG, "%s: E_MUL_XJ needs w_csrT for dX", who);
        const float* w = (msg == GNN_MSG_E_MUL_XJ) ? w_csrT : nullptr;
        gnn_status rc;
        if (mm) {
            GNN_REQUIRE(argmax && (g->E == 0 || g->t2f) && aligned16(argmax), GNN_ERR_INVALID_ARG,
                        "%s: MAX/MIN need the forward argmax (16-byte aligned) and t2f", who);
            rc = run_chunked(who, MODE_ROUTE, g->N, g->E, g->rowptrT, g->colT, w, dOut, dX, nullptr,
                             nullptr, argmax, g->t2f, 0, F, dtype, ws, ws_bytes, st);
        } else {
            rc = run_chunked(who, MODE_SUM, g->N, g->E, g->rowptrT, g->colT, w, dOut, dX, nullptr,
                             op == GNN_MEAN ? g->rowptr : nullptr, nullptr, nullptr, 0, F, dtype, ws,
                             ws_bytes, st);
        }
        if (rc != GNN_OK) return rc;
    }
    if (dW) {
        GNN_REQUIRE(!mm, GNN_ERR_UNSUPPORTED, "%s: dW is defined for SUM/MEAN only", who);
        GNN_REQUIRE(X, GNN_ERR_INVALID_ARG, "%s: dW needs X", who);
        gnn_status rc = run_sddmm(who, g, X, dOut, 1, F, op == GNN_MEAN, dtype, dW, st);
        if (rc != GNN_OK) return rc;
    }
    return GNN_OK;
}

static gnn_status copy_async(const char* who, void* dst, const void* src, size_t bytes,
                             cudaMemcpyKind kind, cudaStream_t st) {
    if (bytes == 0) return GNN_OK;
    cudaError_t e = cudaMemcpyAsync(dst, src, bytes, kind, st);
    if (e != cudaSuccess) GNN_FAIL(GNN_ERR_CUDA, "%s: copy failed: %s", who, cudaGetErrorString(e));
    return GNN_OK;
}

gnn_status gnn_propagate_fused_host(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* h_X,
                                    const float* w_csr, int F, gnn_dtype dtype, void* h_out,
                                    int32_t* argmax, void* d_in, void* d_out, void* ws,
                                    size_t ws_bytes, gnn_stream stream) {
    const char* who = "gnn_propagate_fused_host";
    GNN_REQUIRE(g && h_X && h_out && d_in && d_out, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(F > 0 && (dtype == GNN_F32 || dtype == GNN_BF16), GNN_ERR_INVALID_ARG, "%s: bad F or dtype", who);
    const size_t bytes = (size_t)g->N * F * elem_size(dtype);
    cudaStream_t st = as_stream(stream);
    gnn_status rc = copy_async(who, d_in, h_X, bytes, cudaMemcpyHostToDevice, st);
    if (rc != GNN_OK) return rc;
    rc = gnn_propagate_fused(g, msg, op, d_in, w_csr, F, dtype, d_out, argmax, ws, ws_bytes, stream);
    if (rc != GNN_OK) return rc;
    return copy_async(who, h_out, d_out, bytes, cudaMemcpyDeviceToHost, st);
}

gnn_status gnn_propagate_fused_backward_host(const gnn_csr* g, gnn_msg msg, gnn_op op,
                                             const void* h_dOut, const float* w_csrT,
                                             const int32_t* argmax, int F, gnn_dtype dtype,
                                             void* h_dX, void* d_in, void* d_out, void* ws,
                                             size_t ws_bytes, gnn_stream stream) {
    const char* who = "gnn_propagate_fused_backward_host";
    GNN_REQUIRE(g && h_dOut && h_dX && d_in && d_out, GNN_ERR_INVALID_ARG, "%s: null argument", who);
    GNN_REQUIRE(F > 0 && (dtype == GNN_F32 || dtype == GNN_BF16), GNN_ERR_INVALID_ARG, "%s: bad F or dtype", who);
    const size_t bytes = (size_t)g->N * F * elem_size(dtype);
    cudaStream_t st = as_stream(stream);
    gnn_status rc = copy_async(who, d_in, h_dOut, bytes, cudaMemcpyHostToDevice, st);
    if (rc != GNN_OK) return rc;
    rc = gnn_propagate_fused_backward(g, msg, op, d_in, nullptr, w_csrT, argmax, F, dtype, d_out, nullptr, ws, ws_bytes, stream);
    if (rc != GNN_OK) return rc;
    return copy_async(who, h_dX, d_out, bytes, cudaMemcpyDeviceToHost, st);
}

size_t gnn_propagate_fused_static_max_bytes(void) { return STATIC_WS_BYTES; }

gnn_status gnn_propagate_fused_static(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* X,
                                      const float* w_csr, int F, gnn_dtype dtype, void* out,
                                      int32_t* argmax, gnn_stream stream) {
    const char* who = "gnn_propagate_fused_static";
    GNN_REQUIRE(g && F > 0, GNN_ERR_INVALID_ARG, "%s: null graph or bad F", who);
    const size_t need = gnn_propagate_fused_workspace(g->E, F, op);
    GNN_REQUIRE(need <= STATIC_WS_BYTES, GNN_ERR_WORKSPACE_TOO_SMALL,
                "%s: E=%lld, F=%d needs %zu bytes of scratch; the built-in scratch holds %zu. "
                "Use gnn_propagate_fused with a caller-provided workspace", who, (long long)g->E, F, need, STATIC_WS_BYTES);
    void* ws = nullptr;
    gnn_status rc = static_ws_address(who, &ws);
    if (rc != GNN_OK) return rc;
    return gnn_propagate_fused(g, msg, op, X, w_csr, F, dtype, out, argmax, ws, STATIC_WS_BYTES, stream);
}

}  // extern "C"
