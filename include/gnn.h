/* gnn.h -- C ABI of libgnn_b200: graph message passing on one NVIDIA B200 (sm_100a).
 *
 * The calls follow the message-passing primitives of Sec. 3 ("Message Passing") of
 * "GraphNeuralNetworks.jl: Deep Learning on Graphs with Julia" (arXiv 2412.06354):
 * gather / scatter, apply_edges, aggregate_neighbors, and propagate, which fuses the two
 * into a generalised sparse x dense product; plus the pieces of Sec. 3 "Graph Data
 * Structures" (COO -> sparse form, batching) and "Graph Convolutional Layers" (GCN
 * normalisation, GAT edge softmax) that the hot path needs, each with its backward pass.
 *
 * Conventions (all calls)
 *  - Edge k runs from source src[k] = j to target dst[k] = i.  Messages flow j -> i and are
 *    reduced at i over its incoming edges.  Indices are 0-based.  Node ids and edge ids are
 *    int32 (E < 2^31), row pointers int64.
 *  - Every pointer is a DEVICE pointer unless its name starts with h_ or the comment says
 *    host.  gnn_csr itself is a host struct holding device pointers.
 *  - The caller owns every buffer, including workspaces; the library never allocates or
 *    frees device memory.  Calls enqueue work on the given stream and return without
 *    synchronising, except gnn_coo_to_csr, which synchronises the stream once to read its
 *    4-byte validation word, and the *_host calls, which are documented where declared.
 *  - Feature matrices are row-major with the feature index contiguous ([N,F], [E,F], [G,F]),
 *    base address 16-byte aligned, and F*sizeof(element) a multiple of 16 bytes and at most
 *    2048 bytes for the row-gathering calls (GNN_ERR_UNSUPPORTED otherwise).
 *  - Edge-aligned arrays passed to calls that take a gnn_csr are in CSR order (position p of
 *    the by-target form) unless stated; use gnn_permute_edge_data(eid, ...) once to reorder
 *    COO-ordered data.  Backward calls take weights in transposed-CSR order.
 *  - Sums accumulate in fp32 in a fixed order: results are bit-identical from run to run.
 *    No floating-point atomics are used anywhere.
 *  - Errors: argument errors are detected on the host before any launch and returned as a
 *    gnn_status; nothing traps.  Outputs are unspecified after an error.
 */
#ifndef GNN_B200_H
#define GNN_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* opaque stream handle: a cudaStream_t (0 = default stream) */
typedef void* gnn_stream;

typedef enum {
    GNN_OK = 0,
    GNN_ERR_INVALID_ARG = 1,
    GNN_ERR_INDEX_OUT_OF_RANGE = 2,
    GNN_ERR_NOT_SORTED = 3,
    GNN_ERR_WORKSPACE_TOO_SMALL = 4,
    GNN_ERR_UNSUPPORTED = 5,
    GNN_ERR_CUDA = 6,
    GNN_ERR_TIMEOUT = 7
} gnn_status;

typedef enum { GNN_F32 = 0, GNN_BF16 = 1 } gnn_dtype;
typedef enum { GNN_SUM = 0, GNN_MEAN = 1, GNN_MAX = 2, GNN_MIN = 3 } gnn_op;
typedef enum {
    GNN_MSG_COPY_XJ = 0,   /* m = x_j */
    GNN_MSG_E_MUL_XJ = 1,  /* m = e_ji * x_j */
    GNN_MSG_GAT_LOGIT = 2, /* m = LeakyReLU(al_j + ar_i), per head */
    GNN_MSG_XI_SUB_XJ = 3, /* m = x_i - x_j */
    GNN_MSG_XI_DOT_XJ = 4  /* m = <x_i, x_j>, per head */
} gnn_msg;
/* which multiple c(i) of its self term a row i receives in a gnn_row_epilogue */
typedef enum { GNN_SELF_ALWAYS = 0, GNN_SELF_TIMES_DEGREE = 1, GNN_SELF_IF_NONEMPTY = 2 } gnn_self_mode;

/* Sparse form of a graph (Sec. 3 "Graph Data Structures": the sparse adjacency encoding the
 * fused operations run on).  Host struct, device arrays, all caller-owned.
 *   by target:  rows = targets; rowptr[N+1]; col[p] = source of the edge at position p;
 *               eid[p] = index of that edge in the original COO list.  Within a row, positions
 *               are in ascending eid (stable), which makes the form unique.
 *   transposed: rows = sources; rowptrT[N+1]; colT[q] = target; eidT[q] likewise.
 *   t2f[q]    = position p in the by-target form of the edge at transposed position q. */
typedef struct {
    int32_t N;
    int64_t E;
    int64_t* rowptr;
    int32_t* col;
    int32_t* eid;
    int64_t* rowptrT;
    int32_t* colT;
    int32_t* eidT;
    int32_t* t2f;
} gnn_csr;

const char* gnn_status_string(gnn_status s);
/* text of the most recent error on the calling thread ("" if none); host string */
const char* gnn_last_error_string(void);
int gnn_version(void);

/* ------------------------------------------------------------------ graph set-up ---------- */

/* COO (the default topology format, Sec. 3 "Graph Data Structures") -> both sparse forms.
 * src, dst: int32 [E].  out: host struct whose seven array pointers the caller has set to
 * device buffers of sizes rowptr,rowptrT [N+1] int64 and col,eid,colT,eidT,t2f [E] int32; N and
 * E are filled in.  Validates 0 <= src,dst < N first (GNN_ERR_INDEX_OUT_OF_RANGE; one stream
 * synchronisation to read the flag).  ws: scratch of at least gnn_coo_to_csr_workspace bytes.
 * The result is unique, so it can be compared bit for bit. */
size_t gnn_coo_to_csr_workspace(int32_t N, int64_t E);
gnn_status gnn_coo_to_csr(int32_t N, int64_t E, const int32_t* src, const int32_t* dst,
                          gnn_csr* out, void* ws, size_t ws_bytes, gnn_stream stream);

/* Check of a gnn_csr that did not come from gnn_coo_to_csr (a caller who converts the sparse adjacency form of
 * Sec. 3 "Graph Data Structures" elsewhere): row pointers from 0 to E and non-decreasing, node and edge indices
 * in range, eid / eidT / t2f permutations, edge ids ascending inside every row (the order gnn_coo_to_csr
 * produces, which the deterministic reductions and the argmax convention rely on), and position t2f[q] of the
 * form by target the same edge as position q of the form by source.  Reads the graph only; every read stays in
 * bounds whatever the arrays hold.  Returns GNN_OK, or GNN_ERR_INVALID_ARG with the failed checks named in
 * gnn_last_error_string().  Synchronises the stream (once or twice) to read the result.
 * ws: gnn_csr_validate_workspace(E) bytes of device scratch. */
size_t gnn_csr_validate_workspace(int64_t E);
gnn_status gnn_csr_validate(const gnn_csr* g, void* ws, size_t ws_bytes, gnn_stream stream);

/* Degrees (graph utility of Sec. 3 "Graph Data Structures").  transposed == 0: incoming edges
 * per node; != 0: outgoing.  w == NULL: deg_out is int32 [N] (edge counts, duplicates and
 * loops included).  w != NULL: float [N], the sum of w over the row, w in the order of the
 * chosen form (CSR order, or transposed-CSR order when transposed != 0). */
gnn_status gnn_degree(const gnn_csr* g, int transposed, const float* w, void* deg_out,
                      gnn_stream stream);

/* Append one self-loop per node after the original edges, in node order (A^ = A + I of the GCN
 * layer named in Sec. 3 "Graph Convolutional Layers").  src_out, dst_out: int32 [E+N]. */
gnn_status gnn_add_self_loops(int32_t N, int64_t E, const int32_t* src, const int32_t* dst,
                              int32_t* src_out, int32_t* dst_out, gnn_stream stream);

/* Symmetric GCN normalisation for a graph that already contains its self-loops:
 * d_i = sum of w over the edges into i (w == NULL: every edge counts 1);
 * coefficient of edge j->i = w / sqrt(d_i * d_j), or 0 if either degree is 0.
 * w_csr: NULL or float [E] in CSR order.  Outputs: deg_out float [N] (d), coef_csr float [E] in
 * CSR order, coef_csrT float [E] in transposed-CSR order (either coef pointer may be NULL). */
gnn_status gnn_gcn_norm(const gnn_csr* g, const float* w_csr, float* deg_out, float* coef_csr,
                        float* coef_csrT, gnn_stream stream);

/* out[p, 0..width) = in[perm[p], 0..width) for p < E: reorders edge data, e.g. perm = eid turns
 * COO order into CSR order, perm = t2f turns CSR order into transposed-CSR order.
 * elem_bytes is the size of one element (1, 2, 4 or 8).  in and out must not overlap. */
gnn_status gnn_permute_edge_data(const int32_t* perm, int64_t E, int width, int elem_bytes,
                                 const void* in, void* out, gnn_stream stream);

/* ------------------------------------------------------------------ fused propagate -------- */

/* propagate (Sec. 3 "Message Passing": apply_edges and aggregate_neighbors combined, the
 * generalised matrix product), never materialising the E x F message tensor:
 *   out[i,:] = op over positions p in [rowptr[i], rowptr[i+1]) of  w[p] * X[col[p],:]
 * msg = GNN_MSG_COPY_XJ (w_csr ignored, may be NULL) or GNN_MSG_E_MUL_XJ (w_csr float [E], one
 * scalar per edge, CSR order).  op: SUM; MEAN (sum divided by the number of incoming edges);
 * MAX / MIN (element-wise; argmax int32 [N,F] receives the CSR position of the winner, the
 * smallest position among equal values; may be NULL).  A node with no incoming edge gets 0 and
 * argmax -1.  X, out: [N,F] of dtype.  ws: at least gnn_propagate_fused_workspace bytes, asked for the E and
 * the F of this very call: the edges-per-chunk of the reduction steps with the graph size and the row width,
 * so the size is monotone neither in E nor in F (a workspace sized for a larger graph, or for wider rows, can
 * be too small; take the maximum over the calls that share it).
 * Which of the two reduction kernels runs (rows walked one by one, or positions first) is a fixed function of
 * N, E, F, dtype and op (small graphs and, for sums, large graphs of low mean degree take positions first);
 * results are bit-reproducible for a given graph and shape.
 * Bytes moved per call: at least 4E (+4E with weights) + 8N + 2*N*F*s, at most
 * 4E (+4E) + 8N + (E+N)*F*s when no source row is found in L2. */
size_t gnn_propagate_fused_workspace(int64_t E, int F, gnn_op op);
gnn_status gnn_propagate_fused(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* X,
                               const float* w_csr, int F, gnn_dtype dtype, void* out,
                               int32_t* argmax, void* ws, size_t ws_bytes, gnn_stream stream);

/* gnn_propagate_fused for callers that cannot provide a workspace.  (The paper has no counterpart;
 * this exists for the way the library gets embedded.)  Some hosts give a plugin only the input and
 * output buffers of a fixed memory plan and forbid it to allocate on the device: an inference
 * server whose allocator has already claimed the GPU, so that a raw cudaMalloc may fail or
 * fragment its pool; a latency-bound loop that cannot afford the device-wide synchronisation and
 * unbounded cost of cudaMalloc / cudaFree.  For them the partial-row scratch of the fused propagate
 * is a fixed 8 MiB array inside the library image (gnn_propagate_fused_static_max_bytes()); every
 * GPU that loads the library holds those 8 MiB until the process exits.
 *  - Same arguments and results as gnn_propagate_fused, minus ws / ws_bytes.  No cudaMalloc, cudaFree
 *    or other allocating routine is called.
 *  - Size limit: gnn_propagate_fused_workspace(E, F, op) must not exceed the 8 MiB (ask that function:
 *    the size is not monotone in E); larger problems are rejected with
 *    GNN_ERR_WORKSPACE_TOO_SMALL and a message, before anything is launched.
 *  - The first call on each device looks up the device address of the array (with that device
 *    current) and caches it; make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps whatever the previous call left.  The
 *    kernels write every word of it that they later read, so nothing has to be cleared between
 *    calls; but two calls that overlap on the GPU (different streams, no ordering) race on it. */
size_t gnn_propagate_fused_static_max_bytes(void);
gnn_status gnn_propagate_fused_static(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* X,
                                      const float* w_csr, int F, gnn_dtype dtype, void* out,
                                      int32_t* argmax, gnn_stream stream);

/* Backward of gnn_propagate_fused for dL/dout = dOut [N,F]:
 *   SUM/MEAN: dX[j,:] = sum over transposed positions q of row j of
 *                       wT[q] * scale(colT[q]) * dOut[colT[q],:],  scale = 1 or 1/indegree
 *             dW[p]   = scale(i) * <X[col[p],:], dOut[i,:]>  for p in row i (CSR order)
 *   MAX/MIN : dX[j,f] = sum over q in row j of [argmax[colT[q],f] == t2f[q]] * wT[q]*dOut[colT[q],f]
 * w_csrT: float [E] in transposed-CSR order (E_MUL_XJ) or NULL.  X is needed only for dW.
 * dX [N,F] and dW float [E] may each be NULL (skipped).  ws as for the forward call. */
gnn_status gnn_propagate_fused_backward(const gnn_csr* g, gnn_msg msg, gnn_op op,
                                        const void* dOut, const void* X, const float* w_csrT,
                                        const int32_t* argmax, int F, gnn_dtype dtype, void* dX,
                                        float* dW, void* ws, size_t ws_bytes, gnn_stream stream);

/* ------------------------------------------------------------------ more fused (message, op) pairs */

/* Element-wise tail of a layer, applied to each finished row of a fused call in fp32 before its
 * single rounding (the bias / relu of the conv layers in the training example; the self term of the
 * GIN layer named in Sec. 3 "Graph Convolutional Layers"):
 *   z[i,f]  = agg[i,f] + self_coef * c(i) * Xself[i,f] + bias[f]
 *   out[i,f] = relu ? max(z[i,f], 0) : z[i,f]
 * c(i) = 1 (GNN_SELF_ALWAYS), the number of incoming edges of i (GNN_SELF_TIMES_DEGREE), or 1 if i
 * has an incoming edge and 0 otherwise (GNN_SELF_IF_NONEMPTY).  Xself: [N,F] of the call's dtype or
 * NULL (no self term); bias: float [F] or NULL.  Host struct of device pointers. */
typedef struct {
    const void* Xself;
    float self_coef;
    int self_mode; /* gnn_self_mode */
    const float* bias;
    int relu;
} gnn_row_epilogue;

/* propagate for further "specific message functions and aggregation operations" (Sec. 3 "Message
 * Passing"), still without materialising the E x F message tensor:
 *   out[i,:] = epilogue( op over p in row i of m[p,:] )
 *   COPY_XJ    m[p,:] = Xj[col[p],:]
 *   E_MUL_XJ   m[p,f] = e[p, f / (F / e_width)] * Xj[col[p],f]; e_csr float [E,e_width] in CSR
 *              order, e_width = 1 (any op), or H dividing F with F/H a multiple of 16 bytes worth
 *              of elements, or F (one factor per edge and feature; e rows 16-byte aligned); widths
 *              above 1 take SUM or MEAN only
 *   XI_SUB_XJ  m[p,:] = Xi[i,:] - Xj[col[p],:] for p in row i; Xi [N,F] of dtype.  Computed as
 *              c(i) * Xi[i,:] - (op' over the row of Xj[col[p],:]) with op' = op for SUM / MEAN and
 *              the opposite extremum for MAX / MIN (the difference falls as x_j grows, and rounding
 *              keeps that order); argmax is the position of the winning edge, the smallest among
 *              equal x_j.  epi->Xself must be NULL for this message (the self slot is taken).
 * epi: NULL or an epilogue.  A node with no incoming edge gets epilogue(0) and argmax -1.
 * GIN: COPY_XJ, SUM, epi = {X, 1 + eps, GNN_SELF_ALWAYS}.  ws as for gnn_propagate_fused. */
gnn_status gnn_propagate_msg(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* Xj, const void* Xi,
                             const float* e_csr, int e_width, int F, gnn_dtype dtype,
                             const gnn_row_epilogue* epi, void* out, int32_t* argmax, void* ws,
                             size_t ws_bytes, gnn_stream stream);

/* Backward of gnn_propagate_msg for dL/d(op result) = dOut [N,F] (run gnn_row_epilogue_backward
 * first if the forward call had a bias or relu).  Each output may be NULL (skipped):
 *   dXj [N,F]  gradient that reaches Xj through the messages, reduced over the outgoing edges of
 *              each node in the transposed form (E_MUL_XJ: e_csrT = e in transposed-CSR order,
 *              see gnn_permute_edge_data(t2f); MAX/MIN: argmax of the forward call), plus, if
 *              self_grad is given, self_coef * c(j) * self_grad->Xself[j,:] in the same pass (c(j)
 *              counts the INCOMING edges of j, as in the forward call).  Use it for the self term of
 *              GIN (Xself = dOut, 1 + eps, GNN_SELF_ALWAYS) or when Xi and Xj of XI_SUB_XJ are one
 *              tensor (Xself = dOut, 1, GNN_SELF_TIMES_DEGREE for SUM, GNN_SELF_IF_NONEMPTY else).
 *              self_grad->bias must be NULL and relu 0.
 *   dXi [N,F]  XI_SUB_XJ only: c(i) * dOut[i,:]
 *   de_csr     E_MUL_XJ with SUM / MEAN only: float [E,e_width] in CSR order,
 *              de[p,k] = scale(i) * sum over the features f under factor k of Xj[col[p],f]*dOut[i,f]
 * ws as for the forward call. */
gnn_status gnn_propagate_msg_backward(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* dOut,
                                      const void* Xj, const float* e_csrT, int e_width,
                                      const int32_t* argmax, int F, gnn_dtype dtype,
                                      const gnn_row_epilogue* self_grad, void* dXj, void* dXi,
                                      float* de_csr, void* ws, size_t ws_bytes, gnn_stream stream);

/* Backward of a gnn_row_epilogue's bias and relu for Y = the forward output [N,F]:
 *   dZ[i,f] = dY[i,f] if (!relu or Y[i,f] > 0) else 0   (dZ may alias dY)
 *   dbias[f] = sum over i of dZ[i,f]  (float [F], may be NULL; fixed-order two-stage sum)
 * The gradient of the self term is self_coef * c(i) * dZ[i,:] (see self_grad above).
 * ws: gnn_row_epilogue_backward_workspace(N, F) bytes (needed only with dbias). */
size_t gnn_row_epilogue_backward_workspace(int32_t N, int F);
gnn_status gnn_row_epilogue_backward(const void* Y, const void* dY, int32_t N, int F, gnn_dtype dtype,
                                     int relu, void* dZ, float* dbias, void* ws, size_t ws_bytes,
                                     gnn_stream stream);

/* GIN aggregation (the GINConv layer named in Sec. 3 "Graph Convolutional Layers"):
 *   out[i,:] = (1 + eps) * X[i,:] + sum over incoming edges of X[j,:]       (one pass, one rounding)
 * Backward for dL/dout = dOut: dX[j,:] = (1 + eps) * dOut[j,:] + sum over outgoing edges of
 * dOut[target,:]; deps (device float[1], may be NULL; needs X) = <dOut, X>, a fixed-order sum.
 * ws: gnn_gin_workspace(E, F) bytes for both calls. */
size_t gnn_gin_workspace(int64_t E, int F);
gnn_status gnn_gin(const gnn_csr* g, const void* X, float eps, int F, gnn_dtype dtype, void* out,
                   void* ws, size_t ws_bytes, gnn_stream stream);
gnn_status gnn_gin_backward(const gnn_csr* g, const void* dOut, const void* X, float eps, int F,
                            gnn_dtype dtype, void* dX, float* deps, void* ws, size_t ws_bytes,
                            gnn_stream stream);

/* XI_DOT_XJ message (Sec. 3 "Message Passing": apply_edges with the target and source features):
 *   s[p,h] = <Xi[i,h,:], Xj[col[p],h,:]> for p in row i, float [E,H] in CSR order; Xi, Xj [N,H,C]
 * of dtype, H = 1 or a head spanning a power-of-two number (1..32) of 16-byte chunks.
 * Backward for ds_csr float [E,H] (CSR order):
 *   dXi[i,h,:] = sum over p in row i of ds[p,h] * Xj[col[p],h,:]
 *   dXj[j,h,:] = sum over the outgoing edges of j of ds[.,h] * Xi[target,h,:]
 * (either may be NULL).  ws: gnn_edge_dot_backward_workspace(E, H, C) bytes. */
gnn_status gnn_edge_dot(const gnn_csr* g, const void* Xj, const void* Xi, int H, int C,
                        gnn_dtype dtype, float* s_csr, gnn_stream stream);
size_t gnn_edge_dot_backward_workspace(int64_t E, int H, int C);
gnn_status gnn_edge_dot_backward(const gnn_csr* g, const void* Xj, const void* Xi,
                                 const float* ds_csr, int H, int C, gnn_dtype dtype, void* dXj,
                                 void* dXi, void* ws, size_t ws_bytes, gnn_stream stream);

/* GATv2-style attention logits (Sec. 3 "Message Passing": apply_edges with target and source features; the
 * attention layers of Sec. 3 "Graph Convolutional Layers"): the nonlinearity sits between the sum of the two
 * transformed endpoints and the attention vector, so both rows meet at every edge:
 *   s[p,h] = sum_c a[h,c] * LeakyReLU_slope(Xl[col[p],h,c] + Xr[i,h,c])     for p in row i
 * Xl, Xr: [N,H,C] of dtype (source-side and target-side transforms), a: float [H,C], s_csr: float [E,H] in CSR
 * order (feed it to gnn_edge_softmax, then aggregate Xl with the coefficients through gnn_propagate_msg with
 * e_width = H).  Rows of H*C elements up to 512 bytes; with H > 1 a head must span a power-of-two number of
 * 16-byte chunks.  The E x F tensor is never formed.
 * Backward for ds_csr float [E,H]: dXl, dXr [N,H,C] of dtype and da float [H,C] (da needs dXr and the
 * workspace; each may be NULL); the derivative of LeakyReLU at 0 is slope.  Rows are walked by a warp, rows over
 * 256 positions by a block, in a fixed order.  ws: gnn_gatv2_logits_backward_workspace(N, H, C) bytes. */
gnn_status gnn_gatv2_logits(const gnn_csr* g, const void* Xl, const void* Xr, const float* a, int H, int C,
                            gnn_dtype dtype, float slope, float* s_csr, gnn_stream stream);
size_t gnn_gatv2_logits_backward_workspace(int32_t N, int H, int C);
gnn_status gnn_gatv2_logits_backward(const gnn_csr* g, const void* Xl, const void* Xr, const float* a,
                                     const float* ds_csr, int H, int C, gnn_dtype dtype, float slope,
                                     void* dXl, void* dXr, float* da, void* ws, size_t ws_bytes,
                                     gnn_stream stream);

/* ------------------------------------------------------------------ heterogeneous and temporal graphs */

/* A heterogeneous graph (Sec. 3 "Graph Data Structures": several node and edge types) or a sequence
 * of temporal snapshots is run as ONE sparse form: the edge lists of the relations (snapshots) are
 * concatenated, each with its own offsets into a common numbering of source rows and target rows.
 *   relations    : source nodes of type t start at src_offset = first row of type t in the stacked
 *                  feature matrix; all relations into one target type share dst_offset
 *   snapshots    : dst_offset = t * N (every snapshot owns its block of output rows); src_offset =
 *                  t * N for per-snapshot features or 0 for static features, which then stay
 *                  resident in L2 across the snapshots
 * gnn_merge_edge_lists writes the merged COO list (segment by segment, edges in their given order)
 * and seg_out[k] = segment of merged edge k.  Build the sparse form with gnn_coo_to_csr over
 * max(rows, columns) nodes; inside a row the positions are then ordered by segment, so the sum over
 * relations is taken in relation order, deterministically, by the one launch of the fused
 * propagate.  segs: HOST array of host structs holding device pointers. */
typedef struct {
    int64_t E;
    const int32_t* src;
    const int32_t* dst;
    int32_t src_offset;
    int32_t dst_offset;
} gnn_edge_segment;
gnn_status gnn_merge_edge_lists(const gnn_edge_segment* segs, int S, int32_t* src_out,
                                int32_t* dst_out, int32_t* seg_out, gnn_stream stream);

/* Per-position multipliers that give every segment its own reduction inside the merged form:
 *   coef[p] = w[p] / max(1, number of positions of row i that belong to the segment of p)
 * if seg_is_mean[segment] != 0, else w[p] (w == NULL: 1).  seg_csr: int32 [E], the segment of each
 * CSR position (gnn_permute_edge_data(eid) of seg_out); seg_is_mean: device int32 [S].
 * coef_csr / coef_csrT: float [E] in CSR / transposed-CSR order (either may be NULL).  Then
 *   forward : gnn_propagate_fused(g, E_MUL_XJ, SUM, Xstacked, coef_csr, ...)
 *   backward: gnn_propagate_fused_backward(g, E_MUL_XJ, SUM, dOut, ..., coef_csrT, ...) */
gnn_status gnn_segment_coef(const gnn_csr* g, const int32_t* seg_csr, const float* w_csr,
                            const int32_t* seg_is_mean, int S, float* coef_csr, float* coef_csrT,
                            gnn_stream stream);

/* ------------------------------------------------------------------ unfused primitives ------ */

/* gather (Sec. 3 "Message Passing"): out[k,:] = X[idx[k],:] for k < E; idx = the source vector
 * gives x_j per edge, the target vector gives x_i.  Indices must lie in [0,N) (the vectors that
 * gnn_coo_to_csr accepted do).  A bit-exact copy. */
gnn_status gnn_gather(const int32_t* idx, int64_t E, const void* X, int32_t N, int F,
                      gnn_dtype dtype, void* out, gnn_stream stream);

/* Backward of gather = scatter-add, run as a segmented sum: dX[n,:] = sum of dOut[k,:] over the
 * edges k with dst[k] == n (by_src == 0) or src[k] == n (by_src != 0).  dOut_EF is [E,F] in the
 * ORIGINAL COO edge order (rows are found through eid / eidT).  ws as for gnn_propagate_fused
 * with op SUM. */
gnn_status gnn_gather_backward(const gnn_csr* g, int by_src, const void* dOut_EF, int F,
                               gnn_dtype dtype, void* dX, void* ws, size_t ws_bytes,
                               gnn_stream stream);

/* apply_edges (Sec. 3 "Message Passing"): one message per edge, written in CSR order.
 *   COPY_XJ    m[p,:] = X[col[p],:]
 *   E_MUL_XJ   m[p,f] = e[p, f / (F / e_width)] * X[col[p], f]; e is float [E, e_width] in CSR
 *              order, e_width = 1 (one scalar per edge), H (one per head) or F (element-wise)
 *   GAT_LOGIT  m[p,h] = LeakyReLU_slope(al[col[p],h] + ar[i,h]) for p in row i; here
 *              X_or_al = al and ar are float [N,F] with F = number of heads, dtype must be F32
 * The message function set is fixed; arbitrary closures cannot cross a C ABI. */
gnn_status gnn_apply_edges(const gnn_csr* g, gnn_msg msg, const void* X_or_al, const void* ar,
                           const float* e, int e_width, int F, gnn_dtype dtype, float slope,
                           void* m_out, gnn_stream stream);

/* aggregate_neighbors (Sec. 3 "Message Passing"): out[i,:] = op over p in row i of m[p,:], with
 * m [E,F] in CSR order; ops, empty rows, argmax and ws as for gnn_propagate_fused. */
gnn_status gnn_aggregate(const gnn_csr* g, gnn_op op, const void* m_EF, int F, gnn_dtype dtype,
                         void* out, int32_t* argmax, void* ws, size_t ws_bytes, gnn_stream stream);

/* Backward of aggregate w.r.t. the messages (CSR order): SUM dm[p,:] = dOut[i,:]; MEAN divided
 * by the in-degree of i; MAX/MIN dm[p,f] = dOut[i,f] if argmax[i,f] == p else 0. */
gnn_status gnn_aggregate_backward(const gnn_csr* g, gnn_op op, const void* dOut_NF,
                                  const int32_t* argmax, int F, gnn_dtype dtype, void* dm_EF,
                                  gnn_stream stream);

/* out[i] = alpha*a[i] + beta*b[i] for i < n, computed in fp32 and rounded once (out may alias a or
 * b).  The element-wise glue of layers built from the primitives: W_self*x_i + W_neigh*agg
 * (GraphConv / SAGEConv), (1+eps)*x_i + sum_j x_j (the GIN layer named in Sec. 3 "Graph
 * Convolutional Layers").  n must be a multiple of 16 bytes worth of elements. */
gnn_status gnn_axpby(float alpha, const void* a, float beta, const void* b, int64_t n, gnn_dtype dtype,
                     void* out, gnn_stream stream);

/* ------------------------------------------------------------------ edge softmax ------------ */

/* Attention normalisation of the GAT layer (Sec. 3 "Graph Convolutional Layers"): for every node
 * i and head h, over the incoming edges p of i:
 *   alpha[p,h] = exp(s[p,h] - max_i) / sum_p' exp(s[p',h] - max_i)
 * logits_EH, alpha_EH: [E,H] of dtype in CSR order; math in fp32.  rowmax, rowsum: optional
 * float [N,H] (0 for nodes without incoming edges). */
gnn_status gnn_edge_softmax(const gnn_csr* g, const void* logits_EH, int H, gnn_dtype dtype,
                            void* alpha_EH, float* rowmax, float* rowsum, gnn_stream stream);

/* dLogits[p,h] = alpha[p,h] * (dAlpha[p,h] - sum over the row of alpha*dAlpha) */
gnn_status gnn_edge_softmax_backward(const gnn_csr* g, const void* alpha_EH, const void* dAlpha_EH,
                                     int H, gnn_dtype dtype, void* dLogits_EH, gnn_stream stream);

/* ------------------------------------------------------------------ fused GAT layer core ---- */

/* GAT attention (Sec. 3 "Graph Convolutional Layers" names the layer) on an already transformed
 * node tensor Wx [N,H,C] of dtype; a_src, a_dst float [H,C]:
 *   al[n,h] = <a_src[h,:], Wx[n,h,:]>,  ar[n,h] = <a_dst[h,:], Wx[n,h,:]>
 *   s[p,h]  = LeakyReLU_slope(al[col[p],h] + ar[i,h]),  alpha = edge softmax of s per row and head
 *   out[i,h,:] = sum over p in row i of alpha[p,h] * Wx[col[p],h,:]      (heads concatenated)
 * No self-loops are added; a node without incoming edges gets 0.  Saved for the backward call:
 * alpha_csr float [E,H] (CSR order), al, ar float [N,H].  H must be a power of two <= 32 and a
 * head must span a power-of-two number (1..32) of 16-byte chunks (C = 4, 8, 16, ... for float,
 * 8, 16, 32, ... for bf16); other shapes return GNN_ERR_UNSUPPORTED from the forward and the
 * backward call alike.  The E x F message tensor is never formed.
 * The first gnn_gat_fused / _backward call on a device creates two helper streams and three events (no device
 * memory) on which row classes of the attention kernels run side by side; they are forked from and joined back
 * into `stream`, so the call keeps its place in the stream's order.  Make that first call outside a stream capture.
 * ws: gnn_gat_fused_workspace(N, E, H, C, backward) bytes. */
size_t gnn_gat_fused_workspace(int32_t N, int64_t E, int H, int C, int backward);
gnn_status gnn_gat_fused(const gnn_csr* g, const void* Wx, const float* a_src, const float* a_dst,
                         int H, int C, gnn_dtype dtype, float slope, void* out, float* alpha_csr,
                         float* al, float* ar, void* ws, size_t ws_bytes, gnn_stream stream);

/* Backward for dL/dout = dOut [N,H,C]: dWx [N,H,C] of dtype, da_src, da_dst float [H,C].
 * alpha_csr, al, ar are the forward call's outputs.  The derivative of LeakyReLU at 0 is slope. */
gnn_status gnn_gat_fused_backward(const gnn_csr* g, const void* Wx, const float* a_src,
                                  const float* a_dst, const float* alpha_csr, const float* al,
                                  const float* ar, const void* dOut, int H, int C, gnn_dtype dtype,
                                  float slope, void* dWx, float* da_src, float* da_dst, void* ws,
                                  size_t ws_bytes, gnn_stream stream);

/* ------------------------------------------------------------------ batched-graph pooling --- */

/* A batch of graphs is one block-diagonal graph whose nodes are numbered graph by graph
 * (Sec. 3 "Graph Data Structures": batching).  graph_id: int32 [N], non-decreasing, in [0,G).
 * graph_ptr: int64 [G+1], node range of graph g = graph_ptr[g] .. graph_ptr[g+1]-1.
 * Returns GNN_ERR_NOT_SORTED if the ids are not sorted or out of range (one stream
 * synchronisation to read the flag; ws: at least 4 bytes of device scratch). */
gnn_status gnn_graph_ptr_from_ids(const int32_t* graph_id, int32_t N, int32_t G, int64_t* graph_ptr,
                                  void* ws, size_t ws_bytes, gnn_stream stream);

/* Global pooling (GlobalPool in the training example): out[g,:] = op over the nodes of graph g
 * of X[n,:]; an empty graph gives 0; MAX/MIN: argmax int32 [G,F] = winning node id (first node
 * among equals), -1 if none.  ws: gnn_propagate_fused_workspace(N, F, op) bytes. */
gnn_status gnn_reduce_nodes(const int64_t* graph_ptr, int32_t G, int32_t N, gnn_op op, const void* X,
                            int F, gnn_dtype dtype, void* out_GF, int32_t* argmax, void* ws,
                            size_t ws_bytes, gnn_stream stream);

/* dX[n,:] = dOut[g(n),:] (SUM), / n_g (MEAN), or routed to the argmax node only (MAX/MIN) */
gnn_status gnn_reduce_nodes_backward(const int64_t* graph_ptr, int32_t G, int32_t N, gnn_op op,
                                     const void* dOut_GF, const int32_t* argmax, int F,
                                     gnn_dtype dtype, void* dX_NF, gnn_stream stream);

/* ------------------------------------------------------------------ dense node-wise transform */

/* Y = X * W (the Dense layer / the weight of a conv layer in the training example): X [N,K],
 * W [K,M], Y [N,M], all row-major and of dtype, 16-byte aligned.  With K and M multiples of 16
 * (K up to 512, M up to 1024) the product runs on the tensor cores with fp32 accumulation: bf16 directly, fp32 by an exact
 * three-term bf16 split of every value, which keeps fp32 accuracy (weights that do not fit shared memory
 * three times, e.g. 256x256, run as one launch per block of output columns).  The weight gradient of
 * gnn_linear_backward takes the tensor cores for K and M multiples of 32 (bf16: M of 16).  Other cases use an
 * fp32 FFMA kernel, several times slower.  The first call on a device looks up the driver's tensor-map encoder; the calls
 * themselves allocate nothing.
 * ws: gnn_linear_workspace(N, K, M) bytes; its first 4 bytes are a device status word that the
 * tensor-core path sets to GNN_ERR_TIMEOUT if one of its bounded waits expired (0 otherwise);
 * read it after synchronising if you want to check. */
size_t gnn_linear_workspace(int32_t N, int K, int M);
gnn_status gnn_linear(const void* X, const void* W, int32_t N, int K, int M, gnn_dtype dtype, void* Y,
                      void* ws, size_t ws_bytes, gnn_stream stream);

/* Y = act(X * W + bias): gnn_linear with the element-wise tail of a conv / Dense layer in the training
 * example (bias float [M] or NULL; relu != 0: max(., 0)) applied to the fp32 accumulator before the single
 * rounding, inside the epilogue of the product kernel (no extra pass over Y).  Backward:
 * gnn_row_epilogue_backward(Y, dY, ...) gives dZ and dbias, then gnn_linear_backward on dZ. */
gnn_status gnn_linear_bias_act(const void* X, const void* W, int32_t N, int K, int M, gnn_dtype dtype,
                               const float* bias, int relu, void* Y, void* ws, size_t ws_bytes,
                               gnn_stream stream);

/* dX = dY * W^T ([N,K]) and dW = X^T * dY ([K,M], of dtype); either output may be NULL.  dW sums
 * over the N rows in fixed slabs (one per thread block) whose fp32 partials are added in a
 * fixed order, so the result is reproducible.  X is needed only for dW, W only for dX. */
gnn_status gnn_linear_backward(const void* X, const void* W, const void* dY, int32_t N, int K, int M,
                               gnn_dtype dtype, void* dX, void* dW, void* ws, size_t ws_bytes,
                               gnn_stream stream);

/* ------------------------------------------------------------------ aggregate -> transform fusion */

/* Y = act( (op over p in row i of w[p] * X[col[p],:]) * W + bias ): the fused propagate followed by the
 * weight of a conv layer (Sec. 3 "Message Passing": operations fused "for efficiency"; the GCNConv of
 * the training example) in ONE kernel.  The aggregated [N,K] matrix is never written: a thread block
 * reduces 128 target rows into a shared-memory operand tile (bf16; fp32 input is split exactly into
 * three bf16 terms, which keeps fp32 accuracy) that the tensor cores multiply with the resident W.
 * msg COPY_XJ / E_MUL_XJ (w_csr float [E], CSR order); op SUM or MEAN; X [N,K], W [K,M], Y [N,M] of
 * dtype; bias float [M] or NULL.  Fused for K, M multiples of 16 up to 256 with K*sizeof(element) <= 512
 * and W small enough for shared memory (bf16: up to 256 x 256; fp32: up to 128 x 128); other shapes run
 * aggregate and transform one after the other through the workspace, with the same results.
 * For bf16 the aggregated row is rounded to bf16 once before the product, as the unfused sequence does
 * when it stores it.  ws: gnn_propagate_linear_workspace(N, E, K, M) bytes; its first 4 bytes are the
 * status word of the tensor-core kernels (see gnn_linear).
 * Backward for dL/dY = dY [N,M] (run gnn_row_epilogue_backward first if bias / relu were used):
 *   dX = (A^T dY) * W^T, dW = X^T * (A^T dY), A the weighted adjacency of the forward call.
 * With dW == NULL the same fused kernel runs on the transposed form; with dW the transposed aggregate
 * is needed in memory anyway and goes through the workspace.  w_csrT: transposed-CSR order.
 * Cost: the fusion saves one write and one read of the aggregated matrix (2 of the d + 2 row transfers of a
 * graph of mean degree d).  Measured on a B200, the one-kernel path is slower than gnn_propagate_fused
 * followed by gnn_linear while that matrix fits the 126 MB L2 (its gather warps share the SM with the
 * tensor-core operands); callers who want the fastest path at such sizes make the two calls. */
size_t gnn_propagate_linear_workspace(int32_t N, int64_t E, int K, int M);
gnn_status gnn_propagate_linear(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* X, const float* w_csr,
                                const void* W, int K, int M, gnn_dtype dtype, const float* bias, int relu,
                                void* Y, void* ws, size_t ws_bytes, gnn_stream stream);
gnn_status gnn_propagate_linear_backward(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* dY, const void* X,
                                         const float* w_csrT, const void* W, int K, int M, gnn_dtype dtype,
                                         void* dX, void* dW, void* ws, size_t ws_bytes, gnn_stream stream);

/* Measurement aid (no counterpart in the paper): the bare gathers of a fused propagate.  For every position p of
 * col int32 [E] the 16-byte chunks of row col[p] of X (rows of row_bytes = 64, 128, 256 or 512 bytes, at least
 * max(col) + 1 of them) are loaded and added up; nothing else is computed and no row is written.  The rate
 * E * row_bytes / time is the ceiling that the L2 -> SM return path sets for the reduction kernels on that index
 * stream and row width.  sink: float [gnn_probe_gather_sink_floats(E)], receives one meaningless value per lane. */
size_t gnn_probe_gather_sink_floats(int64_t E);
gnn_status gnn_probe_gather(const int32_t* col, int64_t E, const void* X, int32_t N, int row_bytes, float* sink,
                            gnn_stream stream);

/* Host-buffer variants for callers whose features live in host memory (one call = copy in,
 * compute, copy out; no counterpart in the paper beyond its "transfer the batch to the gpu"
 * step in the training example).  h_X / h_dOut and h_out / h_dX are HOST arrays [N,F] (pinned
 * memory makes the copies asynchronous); d_in and d_out are device staging buffers of N*F*s
 * bytes each; the graph, the weights, argmax and ws are device memory as above.  The calls
 * enqueue host->device copy, kernels and device->host copy on the stream and return without
 * synchronising: the host arrays must stay valid, and h_out / h_dX are complete, only once the
 * stream has been synchronised.  The backward variant computes dX only. */
gnn_status gnn_propagate_fused_host(const gnn_csr* g, gnn_msg msg, gnn_op op, const void* h_X,
                                    const float* w_csr, int F, gnn_dtype dtype, void* h_out,
                                    int32_t* argmax, void* d_in, void* d_out, void* ws,
                                    size_t ws_bytes, gnn_stream stream);
gnn_status gnn_propagate_fused_backward_host(const gnn_csr* g, gnn_msg msg, gnn_op op,
                                             const void* h_dOut, const float* w_csrT,
                                             const int32_t* argmax, int F, gnn_dtype dtype,
                                             void* h_dX, void* d_in, void* d_out, void* ws,
                                             size_t ws_bytes, gnn_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* GNN_B200_H */
