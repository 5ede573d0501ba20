/* CPU checker ("oracle") for graph message passing.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64 loops over the COO edge list (source vector + target vector, Sec. 3
 * "Graph Data Structures") in the original edge order.  It shares no code with the GPU
 * library and is never on the product path: only the tests, the smoke check and the
 * benchmark's CPU-baseline leg call it.
 *
 * What it follows (Sec. 3 "Message Passing"):
 *   m    = apply_edges(message, g, xi, xj, eji)   one message per edge j -> i from the target
 *                                                 features xi, the source features xj and the
 *                                                 edge features eji
 *   mbar = aggregate_neighbors(g, op, m)          reduce the messages of each neighbourhood
 *   propagate = the two combined; for copy_xj / e_mul_xj with '+' it is a generalised
 *               (sparse x dense) matrix product.
 * The method is exact (fusion only avoids materialising the E x F message tensor), so every
 * function here is the plain definition written out.  Conventions the paper leaves open are
 * stated at each function.
 *
 * Edge k runs from source src[k] = j to target dst[k] = i; the neighbourhood of i is the set
 * of its incoming edges; multi-edges and self-loops each count separately.
 *
 * Inputs may be fp64, fp32 or bf16 (raw uint16); they are widened exactly.  Results are fp64.
 * Where an output element is a sum, the function can also return S = sum of |terms|, the
 * scale a floating-point comparison is made against.
 *
 * Threading: ORACLE_THREADS-way split over *target rows*; every thread scans the whole edge
 * list and keeps only its own rows, so the per-row accumulation order is the edge order
 * whatever the thread count.
 *
 * Parity pins: every function below is pinned by tests/test_oracle_pins.py (closed forms on
 * star/path graphs, dense A^T X brute force, invariants, fp64 finite differences).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { DT_F64 = 0, DT_F32 = 1, DT_BF16 = 2 };
enum { OP_SUM = 0, OP_MEAN = 1, OP_MAX = 2, OP_MIN = 3 };
enum { MSG_COPY_XJ = 0, MSG_E_MUL_XJ = 1, MSG_GAT_LOGIT = 2, MSG_XI_SUB_XJ = 3, MSG_XI_DOT_XJ = 4 };

static inline double ld(const void* p, int dt, int64_t i) {
    if (dt == DT_F64) return ((const double*)p)[i];
    if (dt == DT_F32) return (double)((const float*)p)[i];
    uint32_t u = (uint32_t)((const uint16_t*)p)[i] << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

static int g_threads = 1;
void oracle_set_threads(int t) { g_threads = t < 1 ? 1 : t; }
int oracle_get_threads(void) { return g_threads; }

static inline void row_range(int32_t N, int t, int T, int32_t* lo, int32_t* hi) {
    *lo = (int32_t)((int64_t)N * t / T);
    *hi = (int32_t)((int64_t)N * (t + 1) / T);
}

/* ---------------------------------------------------------------- topology */

/* Sparse form of the COO graph: rows = key[k], stable (ties keep ascending edge index).
 * rowptr[N+1], eid[E] = original edge index at each position, col[E] = other[eid].
 * Call with (key=dst, other=src) for the by-target form, (key=src, other=dst) for the
 * transposed one.  Returns 0, or 1 if an index is outside [0,N). */
int oracle_coo_to_csr(int32_t N, int64_t E, const int32_t* key, const int32_t* other,
                      int64_t* rowptr, int32_t* col, int32_t* eid) {
    for (int64_t k = 0; k < E; ++k)
        if (key[k] < 0 || key[k] >= N || other[k] < 0 || other[k] >= N) return 1;
    for (int32_t i = 0; i <= N; ++i) rowptr[i] = 0;
    for (int64_t k = 0; k < E; ++k) rowptr[key[k] + 1]++;
    for (int32_t i = 0; i < N; ++i) rowptr[i + 1] += rowptr[i];
    int64_t* cur = (int64_t*)malloc(((size_t)N + 1) * sizeof(int64_t));
    memcpy(cur, rowptr, ((size_t)N + 1) * sizeof(int64_t));
    for (int64_t k = 0; k < E; ++k) {
        int64_t p = cur[key[k]]++;
        eid[p] = (int32_t)k;
        col[p] = other[k];
    }
    free(cur);
    return 0;
}

/* position in the by-target form of the edge sitting at each position of the transposed form */
void oracle_t2f(int64_t E, const int32_t* eid, const int32_t* eidT, int32_t* t2f) {
    int32_t* pos = (int32_t*)malloc((size_t)(E > 0 ? E : 1) * sizeof(int32_t));
    for (int64_t p = 0; p < E; ++p) pos[eid[p]] = (int32_t)p;
    for (int64_t q = 0; q < E; ++q) t2f[q] = pos[eidT[q]];
    free(pos);
}

/* number of edges whose idx[k] == i (duplicates and loops counted); weighted: sum of w */
void oracle_degree(int32_t N, int64_t E, const int32_t* idx, const float* w, int64_t* deg_i,
                   double* deg_w) {
    for (int32_t i = 0; i < N; ++i) { if (deg_i) deg_i[i] = 0; if (deg_w) deg_w[i] = 0.0; }
    for (int64_t k = 0; k < E; ++k) {
        if (deg_i) deg_i[idx[k]]++;
        if (deg_w) deg_w[idx[k]] += w ? (double)w[k] : 1.0;
    }
}

/* GCN normalisation (the GCNConv layer named in Sec. 3 "Graph Convolutional Layers" and used
 * in the training example): the edge list passed in already holds the self-loops of
 * A^ = A + I.  d_i = sum of w over edges INTO i (w == 1 when NULL);
 * c_k = 1 / sqrt(d_dst[k] * d_src[k]), and c_k = 0 if either degree is 0.
 * Reading: the in-degree of A^ is used for both endpoints (equal to the out-degree on the
 * symmetric graphs this is used on). */
void oracle_gcn_norm(int32_t N, int64_t E, const int32_t* src, const int32_t* dst, const float* w,
                     double* coef) {
    double* d = (double*)calloc((size_t)N, sizeof(double));
    for (int64_t k = 0; k < E; ++k) d[dst[k]] += w ? (double)w[k] : 1.0;
    for (int64_t k = 0; k < E; ++k) {
        double a = d[dst[k]], b = d[src[k]];
        coef[k] = (a > 0.0 && b > 0.0) ? (w ? (double)w[k] : 1.0) / sqrt(a * b) : 0.0;
    }
    free(d);
}

/* ---------------------------------------------------------------- gather / apply_edges */

/* gather: out[k,:] = X[idx[k],:] */
void oracle_gather(int64_t E, const int32_t* idx, const void* X, int dt, int F, double* out) {
    for (int64_t k = 0; k < E; ++k)
        for (int f = 0; f < F; ++f) out[k * F + f] = ld(X, dt, (int64_t)idx[k] * F + f);
}

/* apply_edges, the per-edge message m_k of edge j -> i (Sec. 3 "Message Passing": a message function of
 * the target features xi, the source features xj and the edge features eji):
 *   COPY_XJ    m_k[f] = x_j[f]
 *   E_MUL_XJ   m_k[f] = e_k[g(f)] * x_j[f], e of width 1 (one scalar per edge), H (one per head,
 *              head of feature f is f / (F/H)) or F (element-wise)
 *   GAT_LOGIT  m_k[h] = LeakyReLU_slope(al[j,h] + ar[i,h]), F = H here; LeakyReLU(x) = x for
 *              x > 0, slope*x otherwise
 *   XI_SUB_XJ  m_k[f] = x_i[f] - x_j[f]
 *   XI_DOT_XJ  m_k[h] = sum_c x_i[h*C+c] * x_j[h*C+c], one value per head; ew = H here (number of heads,
 *              C = F/H) and m is [E,H]
 * X holds the source features x_j (for GAT_LOGIT: al); Y the second node array: ar for GAT_LOGIT, the
 * target features x_i for XI_SUB_XJ / XI_DOT_XJ, NULL otherwise. */
void oracle_apply_edges(int msg, int64_t E, const int32_t* src, const int32_t* dst, const void* X,
                        int dtx, const void* Y, int dty, const void* e, int dte, int ew, int F,
                        double slope, double* m) {
    if (msg == MSG_XI_DOT_XJ) {
        int H = ew, C = F / H;
        for (int64_t k = 0; k < E; ++k) {
            int64_t j = src[k], i = dst[k];
            for (int h = 0; h < H; ++h) {
                double a = 0.0;
                for (int c = 0; c < C; ++c) a += ld(Y, dty, i * F + h * C + c) * ld(X, dtx, j * F + h * C + c);
                m[k * H + h] = a;
            }
        }
        return;
    }
    for (int64_t k = 0; k < E; ++k) {
        int64_t j = src[k], i = dst[k];
        for (int f = 0; f < F; ++f) {
            double v;
            if (msg == MSG_COPY_XJ) {
                v = ld(X, dtx, j * F + f);
            } else if (msg == MSG_E_MUL_XJ) {
                int g = (ew == 1) ? 0 : (ew == F ? f : f / (F / ew));
                v = ld(e, dte, k * ew + g) * ld(X, dtx, j * F + f);
            } else if (msg == MSG_XI_SUB_XJ) {
                v = ld(Y, dty, i * F + f) - ld(X, dtx, j * F + f);
            } else {
                double s = ld(X, dtx, j * F + f) + ld(Y, dty, i * F + f);
                v = s > 0.0 ? s : slope * s;
            }
            m[k * F + f] = v;
        }
    }
}

/* backward of apply_edges for dL/dm = dm (fp64; [E,F], or [E,H] for XI_DOT_XJ), original edge order:
 *   COPY_XJ    dXj[j,:] += dm[k,:]
 *   E_MUL_XJ   dXj[j,f] += e_k[g(f)] * dm[k,f];  de[k,g] = sum over the features f of group g of x_j[f]*dm[k,f]
 *   XI_SUB_XJ  dXi[i,:] += dm[k,:];  dXj[j,:] -= dm[k,:]
 *   XI_DOT_XJ  dXi[i,h,:] += dm[k,h] * x_j[h,:];  dXj[j,h,:] += dm[k,h] * x_i[h,:]
 * dXj, dXi [N,F] and de [E,ew] are optional (NULL: not wanted); SXj, SXi, Se hold the sums of |terms|. */
void oracle_apply_edges_backward(int msg, int32_t N, int64_t E, const int32_t* src, const int32_t* dst,
                                 const void* X, int dtx, const void* Y, int dty, const void* e, int dte,
                                 int ew, int F, const double* dm, double* dXj, double* SXj, double* dXi,
                                 double* SXi, double* de, double* Se) {
    for (int64_t x = 0; x < (int64_t)N * F; ++x) {
        if (dXj) dXj[x] = 0.0;
        if (SXj) SXj[x] = 0.0;
        if (dXi) dXi[x] = 0.0;
        if (SXi) SXi[x] = 0.0;
    }
    if (de) for (int64_t x = 0; x < E * ew; ++x) { de[x] = 0.0; if (Se) Se[x] = 0.0; }
    for (int64_t k = 0; k < E; ++k) {
        int64_t j = src[k], i = dst[k];
        for (int f = 0; f < F; ++f) {
            if (msg == MSG_COPY_XJ) {
                double g = dm[k * F + f];
                if (dXj) { dXj[j * F + f] += g; if (SXj) SXj[j * F + f] += fabs(g); }
            } else if (msg == MSG_E_MUL_XJ) {
                int g = (ew == 1) ? 0 : (ew == F ? f : f / (F / ew));
                double d = dm[k * F + f];
                if (dXj) {
                    double t = ld(e, dte, k * ew + g) * d;
                    dXj[j * F + f] += t;
                    if (SXj) SXj[j * F + f] += fabs(t);
                }
                if (de) {
                    double t = ld(X, dtx, j * F + f) * d;
                    de[k * ew + g] += t;
                    if (Se) Se[k * ew + g] += fabs(t);
                }
            } else if (msg == MSG_XI_SUB_XJ) {
                double g = dm[k * F + f];
                if (dXi) { dXi[i * F + f] += g; if (SXi) SXi[i * F + f] += fabs(g); }
                if (dXj) { dXj[j * F + f] -= g; if (SXj) SXj[j * F + f] += fabs(g); }
            } else if (msg == MSG_XI_DOT_XJ) {
                int H = ew, C = F / H;
                double g = dm[k * H + f / C];
                if (dXi) {
                    double t = g * ld(X, dtx, j * F + f);
                    dXi[i * F + f] += t;
                    if (SXi) SXi[i * F + f] += fabs(t);
                }
                if (dXj) {
                    double t = g * ld(Y, dty, i * F + f);
                    dXj[j * F + f] += t;
                    if (SXj) SXj[j * F + f] += fabs(t);
                }
            }
        }
    }
}

/* ---------------------------------------------------------------- aggregate */

/* aggregate_neighbors(g, op, m): out[i,:] = op over the edges k with dst[k] == i of m[k,:].
 *   sum : empty neighbourhood -> 0
 *   mean: sum / number of incoming edges; empty -> 0
 *   max / min: element-wise; arg[i,f] = edge index k of the winner, the FIRST edge (smallest k)
 *              among equal values (strict comparison while scanning in edge order, so +0 and
 *              -0 tie); empty -> value 0, arg -1.
 * S (optional) = sum over the same edges of |m| (divided like the mean). m is fp64 [E,F] in
 * the original edge order. */
void oracle_aggregate(int op, int32_t N, int64_t E, const int32_t* dst, const double* m, int F,
                      double* out, double* S, int64_t* arg) {
    int T = g_threads;
#pragma omp parallel for num_threads(T) schedule(static, 1)
    for (int t = 0; t < T; ++t) {
        int32_t lo, hi;
        row_range(N, t, T, &lo, &hi);
        int64_t* cnt = (int64_t*)calloc((size_t)(hi - lo) + 1, sizeof(int64_t));
        for (int64_t x = (int64_t)lo * F; x < (int64_t)hi * F; ++x) {
            out[x] = 0.0;
            if (S) S[x] = 0.0;
            if (arg) arg[x] = -1;
        }
        for (int64_t k = 0; k < E; ++k) {
            int32_t i = dst[k];
            if (i < lo || i >= hi) continue;
            int first = (cnt[i - lo]++ == 0);
            for (int f = 0; f < F; ++f) {
                double v = m[k * F + f];
                int64_t o = (int64_t)i * F + f;
                if (op == OP_SUM || op == OP_MEAN) {
                    out[o] += v;
                    if (S) S[o] += fabs(v);
                } else if (first || (op == OP_MAX ? v > out[o] : v < out[o])) {
                    out[o] = v;
                    if (S) S[o] = fabs(v);
                    if (arg) arg[o] = k;
                }
            }
        }
        if (op == OP_MEAN)
            for (int32_t i = lo; i < hi; ++i)
                if (cnt[i - lo] > 0)
                    for (int f = 0; f < F; ++f) {
                        out[(int64_t)i * F + f] /= (double)cnt[i - lo];
                        if (S) S[(int64_t)i * F + f] /= (double)cnt[i - lo];
                    }
        free(cnt);
    }
}

/* propagate(message, g, op) written directly (no E x F tensor): message COPY_XJ (w == NULL)
 * or E_MUL_XJ with one scalar w[k] per edge.  By definition equal to
 * aggregate(op, apply_edges(message)).  If slot != NULL only the rows i with slot[i] >= 0 are
 * computed, into row slot[i] of out/S/arg (sampled checking of large graphs); else slot[i] = i.
 * Reading for max/min over weighted messages of stored (fp32 / bf16) features: the winner is an
 * integer decided by floating point, so the comparison is made on the message as a device holds
 * it, w[k]*x rounded once to fp32 (the fp64 product of two fp32 values is exact, so the cast
 * below is that single rounding); fp64 features are compared unrounded. */
void oracle_propagate(int op, int32_t N, int64_t E, const int32_t* src, const int32_t* dst,
                      const void* X, int dt, const float* w, int F, const int32_t* slot,
                      int32_t nslots, double* out, double* S, int64_t* arg) {
    int T = g_threads;
    int32_t R = slot ? nslots : N;
    int64_t* cnt = (int64_t*)calloc((size_t)R + 1, sizeof(int64_t));
    for (int64_t x = 0; x < (int64_t)R * F; ++x) {
        out[x] = 0.0;
        if (S) S[x] = 0.0;
        if (arg) arg[x] = -1;
    }
#pragma omp parallel for num_threads(T) schedule(static, 1)
    for (int t = 0; t < T; ++t) {
        int32_t lo, hi;
        row_range(N, t, T, &lo, &hi);
        for (int64_t k = 0; k < E; ++k) {
            int32_t i = dst[k];
            if (i < lo || i >= hi) continue;
            int64_t r = slot ? slot[i] : i;
            if (r < 0) continue;
            int64_t j = src[k];
            double wk = w ? (double)w[k] : 1.0;
            int first = (cnt[r]++ == 0);
            int as_f32 = (op == OP_MAX || op == OP_MIN) && w && dt != DT_F64;
            for (int f = 0; f < F; ++f) {
                double v = wk * ld(X, dt, j * F + f);
                if (as_f32) v = (double)(float)v;
                int64_t o = r * F + f;
                if (op == OP_SUM || op == OP_MEAN) {
                    out[o] += v;
                    if (S) S[o] += fabs(v);
                } else if (first || (op == OP_MAX ? v > out[o] : v < out[o])) {
                    out[o] = v;
                    if (S) S[o] = fabs(v);
                    if (arg) arg[o] = k;
                }
            }
        }
    }
    if (op == OP_MEAN)
        for (int64_t r = 0; r < R; ++r)
            if (cnt[r] > 0)
                for (int f = 0; f < F; ++f) {
                    out[r * F + f] /= (double)cnt[r];
                    if (S) S[r * F + f] /= (double)cnt[r];
                }
    free(cnt);
}

/* ---------------------------------------------------------------- backward of the linear ops
 * For a scalar loss L with dL/dout = R [N,F] (fp64 or stored dtype):
 *   propagate sum/mean:  dX[j,:]  = sum_{k: src[k]=j} w_k * scale_{dst[k]} * R[dst[k],:]
 *                        dw[k]    = scale_{dst[k]} * <X[src[k],:], R[dst[k],:]>
 *   with scale_i = 1 (sum) or 1/indeg(i) (mean).
 *   propagate max/min:   dX[src[arg[i,f]], f] += R[i,f]   (the single tie-break winner)
 * slot as in oracle_propagate but over SOURCE rows j of dX.  dw / Sw optional (may be NULL). */
void oracle_propagate_backward(int op, int32_t N, int64_t E, const int32_t* src,
                               const int32_t* dst, const void* X, int dtx, const float* w,
                               const void* Rm, int dtr, const int64_t* arg, int F,
                               const int32_t* slot, int32_t nslots, double* dX, double* SdX,
                               double* dw, double* Sdw) {
    int32_t Rn = slot ? nslots : N;
    if (dX) for (int64_t x = 0; x < (int64_t)Rn * F; ++x) { dX[x] = 0.0; if (SdX) SdX[x] = 0.0; }
    int64_t* indeg = (int64_t*)calloc((size_t)N + 1, sizeof(int64_t));
    for (int64_t k = 0; k < E; ++k) indeg[dst[k]]++;
    if (op == OP_MAX || op == OP_MIN) {
        if (dX)
            for (int32_t i = 0; i < N; ++i)
                for (int f = 0; f < F; ++f) {
                    int64_t k = arg[(int64_t)i * F + f];
                    if (k < 0) continue;
                    int64_t r = slot ? slot[src[k]] : src[k];
                    if (r < 0) continue;
                    double wk = w ? (double)w[k] : 1.0;
                    double g = wk * ld(Rm, dtr, (int64_t)i * F + f);
                    dX[r * F + f] += g;
                    if (SdX) SdX[r * F + f] += fabs(g);
                }
        free(indeg);
        return;
    }
    int T = g_threads;
    if (dX) {
#pragma omp parallel for num_threads(T) schedule(static, 1)
        for (int t = 0; t < T; ++t) {
            int32_t lo, hi;
            row_range(N, t, T, &lo, &hi);
            for (int64_t k = 0; k < E; ++k) {
                int32_t j = src[k];
                if (j < lo || j >= hi) continue;
                int64_t r = slot ? slot[j] : j;
                if (r < 0) continue;
                int64_t i = dst[k];
                double c = (w ? (double)w[k] : 1.0) * (op == OP_MEAN ? 1.0 / (double)indeg[i] : 1.0);
                for (int f = 0; f < F; ++f) {
                    double g = c * ld(Rm, dtr, i * F + f);
                    dX[r * F + f] += g;
                    if (SdX) SdX[r * F + f] += fabs(g);
                }
            }
        }
    }
    if (dw) {
#pragma omp parallel for num_threads(T) schedule(static)
        for (int64_t k = 0; k < E; ++k) {
            int64_t i = dst[k], j = src[k];
            double sc = (op == OP_MEAN ? 1.0 / (double)indeg[i] : 1.0), a = 0.0, s = 0.0;
            for (int f = 0; f < F; ++f) {
                double p = ld(X, dtx, j * F + f) * ld(Rm, dtr, i * F + f);
                a += p;
                s += fabs(p);
            }
            dw[k] = sc * a;
            if (Sdw) Sdw[k] = sc * s;
        }
    }
    free(indeg);
}

/* backward of gather: dX[n,:] = sum_{k: idx[k]=n} R[k,:]  (R is [E,F], original edge order) */
void oracle_gather_backward(int32_t N, int64_t E, const int32_t* idx, const void* Rm, int dtr,
                            int F, double* dX, double* SdX) {
    for (int64_t x = 0; x < (int64_t)N * F; ++x) { dX[x] = 0.0; if (SdX) SdX[x] = 0.0; }
    for (int64_t k = 0; k < E; ++k)
        for (int f = 0; f < F; ++f) {
            double g = ld(Rm, dtr, k * F + f);
            dX[(int64_t)idx[k] * F + f] += g;
            if (SdX) SdX[(int64_t)idx[k] * F + f] += fabs(g);
        }
}

/* backward of aggregate w.r.t. the message tensor:
 *   sum: dm[k,:] = R[dst[k],:]   mean: R[dst[k],:] / indeg(dst[k])
 *   max/min: dm[k,f] = R[dst[k],f] if arg[dst[k],f] == k else 0 */
void oracle_aggregate_backward(int op, int32_t N, int64_t E, const int32_t* dst, const void* Rm,
                               int dtr, const int64_t* arg, int F, double* dm) {
    int64_t* indeg = (int64_t*)calloc((size_t)N + 1, sizeof(int64_t));
    for (int64_t k = 0; k < E; ++k) indeg[dst[k]]++;
    for (int64_t k = 0; k < E; ++k) {
        int64_t i = dst[k];
        for (int f = 0; f < F; ++f) {
            double r = ld(Rm, dtr, i * F + f);
            if (op == OP_SUM) dm[k * F + f] = r;
            else if (op == OP_MEAN) dm[k * F + f] = r / (double)indeg[i];
            else dm[k * F + f] = (arg[i * F + f] == k) ? r : 0.0;
        }
    }
    free(indeg);
}

/* ---------------------------------------------------------------- edge softmax (GAT, Sec. 3
 * "Graph Convolutional Layers"): over the incoming edges of each target i, per head h:
 *   alpha[k,h] = exp(s[k,h] - max_i) / sum_{k' into i} exp(s[k',h] - max_i)
 * logits s are [E,H] in the original edge order. */
void oracle_edge_softmax(int32_t N, int64_t E, const int32_t* dst, const void* s, int dts, int H,
                         double* alpha) {
    double* mx = (double*)malloc((size_t)N * H * sizeof(double));
    double* sm = (double*)calloc((size_t)N * H, sizeof(double));
    char* seen = (char*)calloc((size_t)N + 1, 1);
    for (int64_t k = 0; k < E; ++k) {
        int64_t i = dst[k];
        for (int h = 0; h < H; ++h) {
            double v = ld(s, dts, k * H + h);
            if (!seen[i] || v > mx[i * H + h]) mx[i * H + h] = v;
        }
        seen[i] = 1;
    }
    for (int64_t k = 0; k < E; ++k)
        for (int h = 0; h < H; ++h) {
            double ex = exp(ld(s, dts, k * H + h) - mx[(int64_t)dst[k] * H + h]);
            alpha[k * H + h] = ex;
            sm[(int64_t)dst[k] * H + h] += ex;
        }
    for (int64_t k = 0; k < E; ++k)
        for (int h = 0; h < H; ++h) alpha[k * H + h] /= sm[(int64_t)dst[k] * H + h];
    free(mx); free(sm); free(seen);
}

/* backward: ds[k,h] = alpha[k,h] * (dalpha[k,h] - sum_{k' into dst[k]} alpha[k',h]*dalpha[k',h]) */
void oracle_edge_softmax_backward(int32_t N, int64_t E, const int32_t* dst, const void* alpha,
                                  int dta, const void* dalpha, int dtd, int H, double* ds,
                                  double* Sds) {
    double* dot = (double*)calloc((size_t)N * H, sizeof(double));
    double* adot = (double*)calloc((size_t)N * H, sizeof(double));
    for (int64_t k = 0; k < E; ++k)
        for (int h = 0; h < H; ++h) {
            double p = ld(alpha, dta, k * H + h) * ld(dalpha, dtd, k * H + h);
            dot[(int64_t)dst[k] * H + h] += p;
            adot[(int64_t)dst[k] * H + h] += fabs(p);
        }
    for (int64_t k = 0; k < E; ++k)
        for (int h = 0; h < H; ++h) {
            double a = ld(alpha, dta, k * H + h), d = ld(dalpha, dtd, k * H + h);
            ds[k * H + h] = a * (d - dot[(int64_t)dst[k] * H + h]);
            if (Sds) Sds[k * H + h] = fabs(a) * (fabs(d) + adot[(int64_t)dst[k] * H + h]);
        }
    free(dot); free(adot);
}

/* ---------------------------------------------------------------- GAT layer core
 * Wx [N,H,C] is the already transformed node tensor; a_src, a_dst [H,C].
 *   al[n,h] = <a_src[h,:], Wx[n,h,:]>,  ar[n,h] = <a_dst[h,:], Wx[n,h,:]>
 *   s[k,h]  = LeakyReLU_slope(al[src[k],h] + ar[dst[k],h])
 *   alpha   = edge_softmax(s)
 *   out[i,h,:] = sum_{k into i} alpha[k,h] * Wx[src[k],h,:]      (heads concatenated)
 * No self-loops are added; a node with no incoming edge gets 0.  Outputs al, ar [N,H],
 * alpha [E,H] (edge order), out and S [N,H*C]. */
void oracle_gat(int32_t N, int64_t E, const int32_t* src, const int32_t* dst, const void* Wx,
                int dt, const float* a_src, const float* a_dst, int H, int C, double slope,
                double* al, double* ar, double* alpha, double* out, double* S) {
    int F = H * C;
    for (int64_t n = 0; n < N; ++n)
        for (int h = 0; h < H; ++h) {
            double sl = 0.0, sr = 0.0;
            for (int c = 0; c < C; ++c) {
                double x = ld(Wx, dt, n * F + h * C + c);
                sl += (double)a_src[h * C + c] * x;
                sr += (double)a_dst[h * C + c] * x;
            }
            al[n * H + h] = sl;
            ar[n * H + h] = sr;
        }
    double* s = (double*)malloc((size_t)(E > 0 ? E : 1) * H * sizeof(double));
    for (int64_t k = 0; k < E; ++k)
        for (int h = 0; h < H; ++h) {
            double v = al[(int64_t)src[k] * H + h] + ar[(int64_t)dst[k] * H + h];
            s[k * H + h] = v > 0.0 ? v : slope * v;
        }
    oracle_edge_softmax(N, E, dst, s, DT_F64, H, alpha);
    free(s);
    for (int64_t x = 0; x < (int64_t)N * F; ++x) { out[x] = 0.0; if (S) S[x] = 0.0; }
    for (int64_t k = 0; k < E; ++k) {
        int64_t i = dst[k], j = src[k];
        for (int h = 0; h < H; ++h)
            for (int c = 0; c < C; ++c) {
                double v = alpha[k * H + h] * ld(Wx, dt, j * F + h * C + c);
                out[i * F + h * C + c] += v;
                if (S) S[i * F + h * C + c] += fabs(v);
            }
    }
}

/* backward of the GAT core for dL/dout = R [N,H*C]; al, ar, alpha are those of the forward.
 *   dalpha[k,h] = <R[i,h,:], Wx[j,h,:]>
 *   ds          = edge_softmax_backward(alpha, dalpha)
 *   dz[k,h]     = ds[k,h] * (z > 0 ? 1 : slope),  z = al[j,h] + ar[i,h]   (derivative at 0: slope)
 *   dal[j,h]   += dz[k,h];  dar[i,h] += dz[k,h]
 *   dWx[j,h,:] += alpha[k,h] * R[i,h,:]
 *   dWx[n,h,:] += dal[n,h]*a_src[h,:] + dar[n,h]*a_dst[h,:]
 *   da_src[h,:] = sum_n dal[n,h]*Wx[n,h,:];  da_dst likewise with dar
 * Outputs dWx, SdWx [N,H*C]; da_src, da_dst, Sda_src, Sda_dst [H,C]. */
void oracle_gat_backward(int32_t N, int64_t E, const int32_t* src, const int32_t* dst,
                         const void* Wx, int dt, const float* a_src, const float* a_dst, int H,
                         int C, double slope, const double* al, const double* ar,
                         const double* alpha, const void* Rm, int dtr, double* dWx, double* SdWx,
                         double* da_src, double* da_dst, double* Sda_src, double* Sda_dst) {
    int F = H * C;
    size_t EH = (size_t)(E > 0 ? E : 1) * H;
    double* dalpha = (double*)malloc(EH * sizeof(double));
    double* ds = (double*)malloc(EH * sizeof(double));
    double* Sds = (double*)malloc(EH * sizeof(double));
    double* dal = (double*)calloc((size_t)N * H, sizeof(double));
    double* dar = (double*)calloc((size_t)N * H, sizeof(double));
    double* Sal = (double*)calloc((size_t)N * H, sizeof(double));
    double* Sar = (double*)calloc((size_t)N * H, sizeof(double));
    for (int64_t x = 0; x < (int64_t)N * F; ++x) { dWx[x] = 0.0; if (SdWx) SdWx[x] = 0.0; }
    for (int64_t k = 0; k < E; ++k) {
        int64_t i = dst[k], j = src[k];
        for (int h = 0; h < H; ++h) {
            double d = 0.0;
            for (int c = 0; c < C; ++c)
                d += ld(Rm, dtr, i * F + h * C + c) * ld(Wx, dt, j * F + h * C + c);
            dalpha[k * H + h] = d;
        }
    }
    oracle_edge_softmax_backward(N, E, dst, alpha, DT_F64, dalpha, DT_F64, H, ds, Sds);
    for (int64_t k = 0; k < E; ++k) {
        int64_t i = dst[k], j = src[k];
        for (int h = 0; h < H; ++h) {
            double z = al[j * H + h] + ar[i * H + h];
            double g = z > 0.0 ? 1.0 : slope;
            dal[j * H + h] += ds[k * H + h] * g;
            dar[i * H + h] += ds[k * H + h] * g;
            Sal[j * H + h] += Sds[k * H + h] * fabs(g);
            Sar[i * H + h] += Sds[k * H + h] * fabs(g);
            for (int c = 0; c < C; ++c) {
                double v = alpha[k * H + h] * ld(Rm, dtr, i * F + h * C + c);
                dWx[j * F + h * C + c] += v;
                if (SdWx) SdWx[j * F + h * C + c] += fabs(v);
            }
        }
    }
    for (int x = 0; x < F; ++x) {
        da_src[x] = 0.0; da_dst[x] = 0.0;
        if (Sda_src) Sda_src[x] = 0.0;
        if (Sda_dst) Sda_dst[x] = 0.0;
    }
    for (int64_t n = 0; n < N; ++n)
        for (int h = 0; h < H; ++h)
            for (int c = 0; c < C; ++c) {
                double x = ld(Wx, dt, n * F + h * C + c);
                double t1 = dal[n * H + h] * (double)a_src[h * C + c];
                double t2 = dar[n * H + h] * (double)a_dst[h * C + c];
                dWx[n * F + h * C + c] += t1 + t2;
                if (SdWx)
                    SdWx[n * F + h * C + c] += Sal[n * H + h] * fabs((double)a_src[h * C + c]) +
                                               Sar[n * H + h] * fabs((double)a_dst[h * C + c]);
                da_src[h * C + c] += dal[n * H + h] * x;
                da_dst[h * C + c] += dar[n * H + h] * x;
                if (Sda_src) Sda_src[h * C + c] += Sal[n * H + h] * fabs(x);
                if (Sda_dst) Sda_dst[h * C + c] += Sar[n * H + h] * fabs(x);
            }
    free(dalpha); free(ds); free(Sds); free(dal); free(dar); free(Sal); free(Sar);
}

/* ---------------------------------------------------------------- pooling over a batch
 * (GlobalPool in the training example): nodes of graph g are the contiguous range
 * graph_ptr[g] .. graph_ptr[g+1]-1.  out[g,:] = op over those rows of X; empty graph -> 0,
 * arg -1; max/min tie-break: first node.  arg holds node ids. */
void oracle_reduce_nodes(int op, int32_t G, const int32_t* graph_ptr, const void* X, int dt, int F,
                         double* out, double* S, int64_t* arg) {
    for (int32_t g = 0; g < G; ++g) {
        int64_t a = graph_ptr[g], b = graph_ptr[g + 1];
        for (int f = 0; f < F; ++f) {
            double acc = 0.0, s = 0.0;
            int64_t am = -1;
            for (int64_t n = a; n < b; ++n) {
                double v = ld(X, dt, n * F + f);
                if (op == OP_SUM || op == OP_MEAN) { acc += v; s += fabs(v); }
                else if (n == a || (op == OP_MAX ? v > acc : v < acc)) { acc = v; s = fabs(v); am = n; }
            }
            if (op == OP_MEAN && b > a) { acc /= (double)(b - a); s /= (double)(b - a); }
            out[(int64_t)g * F + f] = acc;
            if (S) S[(int64_t)g * F + f] = s;
            if (arg) arg[(int64_t)g * F + f] = am;
        }
    }
}

/* backward: sum: dX[n,:] = R[g(n),:]; mean: / n_g; max/min: R[g,f] to node arg[g,f] only */
void oracle_reduce_nodes_backward(int op, int32_t G, const int32_t* graph_ptr, const void* Rm,
                                  int dtr, const int64_t* arg, int F, double* dX) {
    for (int32_t g = 0; g < G; ++g) {
        int64_t a = graph_ptr[g], b = graph_ptr[g + 1];
        for (int64_t n = a; n < b; ++n)
            for (int f = 0; f < F; ++f) {
                double r = ld(Rm, dtr, (int64_t)g * F + f);
                if (op == OP_SUM) dX[n * F + f] = r;
                else if (op == OP_MEAN) dX[n * F + f] = r / (double)(b - a);
                else dX[n * F + f] = (arg[(int64_t)g * F + f] == n) ? r : 0.0;
            }
    }
}

/* ---------------------------------------------------------------- dense node-wise transform
 * (the Dense layer / the weight of a conv layer in the training example): Y = A * B with
 * A [n,k] (optionally read transposed), B [k,m] (optionally transposed), textbook triple loop.
 * ta: A is stored [k,n] and used as its transpose; tb: B is stored [m,k]. */
void oracle_matmul(const void* A, int dta, int ta, const void* B, int dtb, int tb, int64_t n,
                   int64_t k, int64_t m, double* Y, double* S) {
    int T = g_threads;
#pragma omp parallel for num_threads(T) schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int64_t j = 0; j < m; ++j) {
            double acc = 0.0, s = 0.0;
            for (int64_t l = 0; l < k; ++l) {
                double a = ta ? ld(A, dta, l * n + i) : ld(A, dta, i * k + l);
                double b = tb ? ld(B, dtb, j * k + l) : ld(B, dtb, l * m + j);
                acc += a * b;
                s += fabs(a * b);
            }
            Y[i * m + j] = acc;
            if (S) S[i * m + j] = s;
        }
}
