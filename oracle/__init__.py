"""CPU checker ("oracle") for graph message passing -- TEST INFRASTRUCTURE ONLY.

numpy-facing wrapper over ``oracle.c`` (plain fp64 loops over the COO edge list).  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the GPU
library never does, and the two share no code.

Arrays: ``src``/``dst`` int32 [E]; features float64 / float32 / uint16 (bf16 bit patterns),
row-major [N,F].  Results are float64.  Functions that return sums also return ``S``, the sum
of absolute values of the terms, which is the scale tolerances are measured against.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liboracle.so")
_lib = None

SUM, MEAN, MAX, MIN = 0, 1, 2, 3
COPY_XJ, E_MUL_XJ, GAT_LOGIT, XI_SUB_XJ, XI_DOT_XJ = 0, 1, 2, 3, 4
OPS = {"sum": SUM, "mean": MEAN, "max": MAX, "min": MIN}


def build(force: bool = False) -> str:
    src = os.path.join(_HERE, "oracle.c")
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", src, "-o", _LIB_PATH, "-lm"])
    return _LIB_PATH


def _L():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB_PATH)
        _lib.oracle_coo_to_csr.restype = C.c_int
        _lib.oracle_get_threads.restype = C.c_int
    return _lib


def set_threads(t: int) -> None:
    _L().oracle_set_threads(C.c_int(int(t)))


def get_threads() -> int:
    return int(_L().oracle_get_threads())


def _dt(a):
    if a.dtype == np.float64:
        return 0
    if a.dtype == np.float32:
        return 1
    if a.dtype == np.uint16:
        return 2
    raise TypeError(f"unsupported dtype {a.dtype}")


def _c(a, dtype=None):
    a = np.ascontiguousarray(a) if dtype is None else np.ascontiguousarray(a, dtype=dtype)
    return a


def _ptr(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


def _op(op):
    return OPS[op] if isinstance(op, str) else int(op)


def _i32(a):
    return _c(a, np.int32)


def _f32_or_none(w):
    return None if w is None else _c(w, np.float32)


# ------------------------------------------------------------------ topology
def coo_to_csr(N, key, other):
    """Stable sparse form keyed by ``key`` -> (rowptr int64 [N+1], col int32 [E], eid int32 [E])."""
    key, other = _i32(key), _i32(other)
    E = key.shape[0]
    rowptr = np.empty(N + 1, np.int64)
    col = np.empty(E, np.int32)
    eid = np.empty(E, np.int32)
    rc = _L().oracle_coo_to_csr(C.c_int32(N), C.c_int64(E), _ptr(key), _ptr(other), _ptr(rowptr), _ptr(col), _ptr(eid))
    if rc != 0:
        raise IndexError("edge index outside [0, N)")
    return rowptr, col, eid


def t2f(eid, eidT):
    eid, eidT = _i32(eid), _i32(eidT)
    out = np.empty(eid.shape[0], np.int32)
    _L().oracle_t2f(C.c_int64(eid.shape[0]), _ptr(eid), _ptr(eidT), _ptr(out))
    return out


def degree(N, idx, w=None):
    idx = _i32(idx)
    w = _f32_or_none(w)
    di = np.empty(N, np.int64)
    dw = np.empty(N, np.float64)
    _L().oracle_degree(C.c_int32(N), C.c_int64(idx.shape[0]), _ptr(idx), _ptr(w), _ptr(di), _ptr(dw))
    return di, dw


def gcn_norm(N, src, dst, w=None):
    """Coefficients for an edge list that already contains the self-loops, COO order."""
    src, dst = _i32(src), _i32(dst)
    w = _f32_or_none(w)
    coef = np.empty(src.shape[0], np.float64)
    _L().oracle_gcn_norm(C.c_int32(N), C.c_int64(src.shape[0]), _ptr(src), _ptr(dst), _ptr(w), _ptr(coef))
    return coef


# ------------------------------------------------------------------ gather / apply / aggregate
def gather(idx, X):
    idx, X = _i32(idx), _c(X)
    F = X.shape[1]
    out = np.empty((idx.shape[0], F), np.float64)
    _L().oracle_gather(C.c_int64(idx.shape[0]), _ptr(idx), _ptr(X), C.c_int(_dt(X)), C.c_int(F), _ptr(out))
    return out


def apply_edges(msg, src, dst, X, Y=None, e=None, slope=0.2, H=1):
    """Per-edge messages, original edge order.  X: source-side node array (x_j; al for GAT_LOGIT); Y: target-side
    node array (x_i for XI_SUB_XJ / XI_DOT_XJ, ar for GAT_LOGIT).  XI_DOT_XJ returns [E,H] (one dot product per head)."""
    src, dst, X = _i32(src), _i32(dst), _c(X)
    E, F = src.shape[0], X.shape[1]
    Y = None if Y is None else _c(Y)
    ew = 0
    if e is not None:
        e = _c(e)
        if e.ndim == 1:
            e = e.reshape(-1, 1)
        ew = e.shape[1]
    if msg == XI_DOT_XJ:
        ew = H
    m = np.empty((E, H if msg == XI_DOT_XJ else F), np.float64)
    _L().oracle_apply_edges(C.c_int(msg), C.c_int64(E), _ptr(src), _ptr(dst), _ptr(X), C.c_int(_dt(X)),
                            _ptr(Y), C.c_int(_dt(Y) if Y is not None else 0),
                            _ptr(e), C.c_int(_dt(e) if e is not None else 0), C.c_int(ew), C.c_int(F),
                            C.c_double(slope), _ptr(m))
    return m


def apply_edges_backward(msg, N, src, dst, X, dm, Y=None, e=None, H=1, want=("dXj",)):
    """Backward of apply_edges for dL/dm = dm -> dict with the wanted ones of dXj, dXi [N,F], de [E,ew]
    and their magnitude sums SXj, SXi, Se."""
    src, dst, X = _i32(src), _i32(dst), _c(X)
    E, F = src.shape[0], X.shape[1]
    Y = None if Y is None else _c(Y)
    dm = _c(dm, np.float64)
    ew = 0
    if e is not None:
        e = _c(e)
        if e.ndim == 1:
            e = e.reshape(-1, 1)
        ew = e.shape[1]
    if msg == XI_DOT_XJ:
        ew = H
    o = {}
    for k, shape in (("dXj", (N, F)), ("dXi", (N, F)), ("de", (E, max(ew, 1)))):
        o[k] = np.empty(shape, np.float64) if k in want else None
        o["S" + k[1:]] = np.empty(shape, np.float64) if k in want else None
    _L().oracle_apply_edges_backward(C.c_int(msg), C.c_int32(N), C.c_int64(E), _ptr(src), _ptr(dst), _ptr(X), C.c_int(_dt(X)),
                                     _ptr(Y), C.c_int(_dt(Y) if Y is not None else 0), _ptr(e), C.c_int(_dt(e) if e is not None else 0),
                                     C.c_int(ew), C.c_int(F), _ptr(dm), _ptr(o["dXj"]), _ptr(o["SXj"]), _ptr(o["dXi"]), _ptr(o["SXi"]),
                                     _ptr(o["de"]), _ptr(o["Se"]))
    return o


def aggregate(op, N, dst, m):
    """-> (out [N,F], S [N,F], arg int64 [N,F] (edge index of the max/min winner, -1 if none))."""
    dst, m = _i32(dst), _c(m, np.float64)
    F = m.shape[1]
    out = np.empty((N, F), np.float64)
    S = np.empty((N, F), np.float64)
    arg = np.empty((N, F), np.int64)
    _L().oracle_aggregate(C.c_int(_op(op)), C.c_int32(N), C.c_int64(dst.shape[0]), _ptr(dst), _ptr(m), C.c_int(F),
                          _ptr(out), _ptr(S), _ptr(arg))
    return out, S, arg


def propagate(op, N, src, dst, X, w=None, rows=None):
    """Fused propagate: copy_xj (w None) or e_mul_xj (scalar edge weight) with op.
    rows: optional int array of target rows to compute (sampled checking) -> outputs [len(rows),F]."""
    src, dst, X = _i32(src), _i32(dst), _c(X)
    w = _f32_or_none(w)
    F = X.shape[1]
    slot, R = None, N
    if rows is not None:
        rows = np.asarray(rows, np.int64)
        slot = np.full(N, -1, np.int32)
        slot[rows] = np.arange(rows.shape[0], dtype=np.int32)
        R = rows.shape[0]
    out = np.empty((R, F), np.float64)
    S = np.empty((R, F), np.float64)
    arg = np.empty((R, F), np.int64)
    _L().oracle_propagate(C.c_int(_op(op)), C.c_int32(N), C.c_int64(src.shape[0]), _ptr(src), _ptr(dst), _ptr(X),
                          C.c_int(_dt(X)), _ptr(w), C.c_int(F), _ptr(slot), C.c_int32(R), _ptr(out), _ptr(S), _ptr(arg))
    return out, S, arg


def propagate_backward(op, N, src, dst, X, w, R, arg=None, rows=None, want_dX=True, want_dw=False):
    """-> dict(dX, SdX, dw, Sdw) for dL/dout = R.  rows: optional subset of SOURCE rows of dX."""
    src, dst, R = _i32(src), _i32(dst), _c(R)
    X = None if X is None else _c(X)
    w = _f32_or_none(w)
    F = R.shape[1]
    E = src.shape[0]
    slot, Rn = None, N
    if rows is not None:
        rows = np.asarray(rows, np.int64)
        slot = np.full(N, -1, np.int32)
        slot[rows] = np.arange(rows.shape[0], dtype=np.int32)
        Rn = rows.shape[0]
    dX = np.empty((Rn, F), np.float64) if want_dX else None
    SdX = np.empty((Rn, F), np.float64) if want_dX else None
    dw = np.empty(E, np.float64) if want_dw else None
    Sdw = np.empty(E, np.float64) if want_dw else None
    arg = None if arg is None else _c(arg, np.int64)
    _L().oracle_propagate_backward(C.c_int(_op(op)), C.c_int32(N), C.c_int64(E), _ptr(src), _ptr(dst),
                                   _ptr(X), C.c_int(_dt(X) if X is not None else 0), _ptr(w),
                                   _ptr(R), C.c_int(_dt(R)), _ptr(arg), C.c_int(F), _ptr(slot), C.c_int32(Rn),
                                   _ptr(dX), _ptr(SdX), _ptr(dw), _ptr(Sdw))
    return dict(dX=dX, SdX=SdX, dw=dw, Sdw=Sdw)


def gather_backward(N, idx, R):
    idx, R = _i32(idx), _c(R)
    F = R.shape[1]
    dX = np.empty((N, F), np.float64)
    S = np.empty((N, F), np.float64)
    _L().oracle_gather_backward(C.c_int32(N), C.c_int64(idx.shape[0]), _ptr(idx), _ptr(R), C.c_int(_dt(R)), C.c_int(F),
                                _ptr(dX), _ptr(S))
    return dX, S


def aggregate_backward(op, N, dst, R, arg=None):
    dst, R = _i32(dst), _c(R)
    F = R.shape[1]
    arg = None if arg is None else _c(arg, np.int64)
    dm = np.empty((dst.shape[0], F), np.float64)
    _L().oracle_aggregate_backward(C.c_int(_op(op)), C.c_int32(N), C.c_int64(dst.shape[0]), _ptr(dst), _ptr(R),
                                   C.c_int(_dt(R)), _ptr(arg), C.c_int(F), _ptr(dm))
    return dm


# ------------------------------------------------------------------ softmax / GAT
def edge_softmax(N, dst, s):
    dst, s = _i32(dst), _c(s)
    H = s.shape[1]
    alpha = np.empty(s.shape, np.float64)
    _L().oracle_edge_softmax(C.c_int32(N), C.c_int64(dst.shape[0]), _ptr(dst), _ptr(s), C.c_int(_dt(s)), C.c_int(H), _ptr(alpha))
    return alpha


def edge_softmax_backward(N, dst, alpha, dalpha):
    dst, alpha, dalpha = _i32(dst), _c(alpha), _c(dalpha)
    H = alpha.shape[1]
    ds = np.empty(alpha.shape, np.float64)
    S = np.empty(alpha.shape, np.float64)
    _L().oracle_edge_softmax_backward(C.c_int32(N), C.c_int64(dst.shape[0]), _ptr(dst), _ptr(alpha), C.c_int(_dt(alpha)),
                                      _ptr(dalpha), C.c_int(_dt(dalpha)), C.c_int(H), _ptr(ds), _ptr(S))
    return ds, S


def gat(N, src, dst, Wx, a_src, a_dst, H, Cw, slope=0.2):
    src, dst, Wx = _i32(src), _i32(dst), _c(Wx)
    a_src, a_dst = _c(a_src, np.float32), _c(a_dst, np.float32)
    E, F = src.shape[0], H * Cw
    al = np.empty((N, H), np.float64)
    ar = np.empty((N, H), np.float64)
    alpha = np.empty((E, H), np.float64)
    out = np.empty((N, F), np.float64)
    S = np.empty((N, F), np.float64)
    _L().oracle_gat(C.c_int32(N), C.c_int64(E), _ptr(src), _ptr(dst), _ptr(Wx), C.c_int(_dt(Wx)), _ptr(a_src), _ptr(a_dst),
                    C.c_int(H), C.c_int(Cw), C.c_double(slope), _ptr(al), _ptr(ar), _ptr(alpha), _ptr(out), _ptr(S))
    return dict(al=al, ar=ar, alpha=alpha, out=out, S=S)


def gat_backward(N, src, dst, Wx, a_src, a_dst, H, Cw, fwd, R, slope=0.2):
    src, dst, Wx, R = _i32(src), _i32(dst), _c(Wx), _c(R)
    a_src, a_dst = _c(a_src, np.float32), _c(a_dst, np.float32)
    E, F = src.shape[0], H * Cw
    dWx = np.empty((N, F), np.float64)
    SdWx = np.empty((N, F), np.float64)
    o = [np.empty((H, Cw), np.float64) for _ in range(4)]
    _L().oracle_gat_backward(C.c_int32(N), C.c_int64(E), _ptr(src), _ptr(dst), _ptr(Wx), C.c_int(_dt(Wx)), _ptr(a_src),
                             _ptr(a_dst), C.c_int(H), C.c_int(Cw), C.c_double(slope), _ptr(_c(fwd["al"])), _ptr(_c(fwd["ar"])),
                             _ptr(_c(fwd["alpha"])), _ptr(R), C.c_int(_dt(R)), _ptr(dWx), _ptr(SdWx),
                             _ptr(o[0]), _ptr(o[1]), _ptr(o[2]), _ptr(o[3]))
    return dict(dWx=dWx, SdWx=SdWx, da_src=o[0], da_dst=o[1], Sda_src=o[2], Sda_dst=o[3])


# ------------------------------------------------------------------ pooling / dense
def reduce_nodes(op, graph_ptr, X):
    graph_ptr, X = _i32(graph_ptr), _c(X)
    G, F = graph_ptr.shape[0] - 1, X.shape[1]
    out = np.empty((G, F), np.float64)
    S = np.empty((G, F), np.float64)
    arg = np.empty((G, F), np.int64)
    _L().oracle_reduce_nodes(C.c_int(_op(op)), C.c_int32(G), _ptr(graph_ptr), _ptr(X), C.c_int(_dt(X)), C.c_int(F),
                             _ptr(out), _ptr(S), _ptr(arg))
    return out, S, arg


def reduce_nodes_backward(op, graph_ptr, R, arg=None):
    graph_ptr, R = _i32(graph_ptr), _c(R)
    G, F = graph_ptr.shape[0] - 1, R.shape[1]
    N = int(graph_ptr[-1])
    arg = None if arg is None else _c(arg, np.int64)
    dX = np.zeros((N, F), np.float64)
    _L().oracle_reduce_nodes_backward(C.c_int(_op(op)), C.c_int32(G), _ptr(graph_ptr), _ptr(R), C.c_int(_dt(R)), _ptr(arg),
                                      C.c_int(F), _ptr(dX))
    return dX


def matmul(A, B, ta=False, tb=False):
    """Y = op(A) @ op(B) by a triple loop -> (Y, S)."""
    A, B = _c(A), _c(B)
    n, k = (A.shape[1], A.shape[0]) if ta else A.shape
    m = B.shape[0] if tb else B.shape[1]
    assert (B.shape[1] if tb else B.shape[0]) == k
    Y = np.empty((n, m), np.float64)
    S = np.empty((n, m), np.float64)
    _L().oracle_matmul(_ptr(A), C.c_int(_dt(A)), C.c_int(int(ta)), _ptr(B), C.c_int(_dt(B)), C.c_int(int(tb)),
                       C.c_int64(n), C.c_int64(k), C.c_int64(m), _ptr(Y), _ptr(S))
    return Y, S


# ------------------------------------------------------------------ compositions of the primitives above
# (Sec. 3 "Message Passing": propagate = apply_edges followed by aggregate_neighbors; Sec. 3 "Graph
# Convolutional Layers" names GINConv; Sec. 3 "Graph Data Structures" names heterogeneous and temporal graphs.)
def propagate_msg(msg, op, N, src, dst, Xj, Xi=None, e=None, H=1):
    """aggregate(op, apply_edges(msg)) for any message -> (out, S, arg)."""
    return aggregate(op, N, dst, apply_edges(msg, src, dst, Xj, Y=Xi, e=e, H=H))


def propagate_msg_backward(msg, op, N, src, dst, Xj, R, Xi=None, e=None, H=1, arg=None, want=("dXj",)):
    """Backward of propagate_msg for dL/dout = R: aggregate_backward, then apply_edges_backward."""
    dm = aggregate_backward(op, N, dst, R, arg)
    return apply_edges_backward(msg, N, src, dst, Xj, dm, Y=Xi, e=e, H=H, want=want)


def gin(N, src, dst, X, eps):
    """GIN aggregation: out[i,:] = (1 + eps) * x_i + sum over incoming edges of x_j -> (out, S)."""
    o, S, _ = propagate("sum", N, src, dst, X)
    from_self = (1.0 + float(eps)) * _to64(X)
    return from_self + o, np.abs(from_self) + S


def gin_backward(N, src, dst, X, eps, R):
    """-> dict(dX, SdX, deps): dX = (1+eps) * R + sum over outgoing edges of R[target]; deps = <R, X>."""
    bw = propagate_backward("sum", N, src, dst, None, None, R)
    R64 = _to64(R)
    return dict(dX=(1.0 + float(eps)) * R64 + bw["dX"], SdX=np.abs((1.0 + float(eps)) * R64) + bw["SdX"],
                deps=float((R64 * _to64(X)).sum()), Sdeps=float(np.abs(R64 * _to64(X)).sum()))


def gatv2_logits(src, dst, Xl, Xr, a, H, slope=0.2):
    """GATv2-style attention logits (the nonlinearity sits between the sum of the two transformed endpoints and
    the attention vector): s[k,h] = sum_c a[h,c] * LeakyReLU(Xl[src_k,h,c] + Xr[dst_k,h,c]).
    Composition: the element-wise GAT_LOGIT message over all H*C features, then one dot product per head with a.
    -> (s [E,H], S [E,H] sums of |terms|, m [E,F] the element-wise messages)."""
    m = apply_edges(GAT_LOGIT, src, dst, Xl, Y=Xr, slope=slope)
    E, F = m.shape
    a64 = _to64(a).reshape(H, F // H)
    m3 = m.reshape(E, H, F // H)
    return (m3 * a64[None]).sum(-1), (np.abs(m3) * np.abs(a64)[None]).sum(-1), m


def gatv2_logits_backward(N, src, dst, Xl, Xr, a, H, ds, slope=0.2):
    """For dL/ds = ds [E,H]: dm[k,h,c] = ds[k,h] * a[h,c] * LeakyReLU'(z) (slope at z <= 0), dXl = scatter-add of dm
    by source, dXr by target, da[h,c] = sum_k ds[k,h] * LeakyReLU(z)[k,h,c] -> dict(dXl, SXl, dXr, SXr, da, Sda)."""
    _, _, m = gatv2_logits(src, dst, Xl, Xr, a, H, slope)
    E, F = m.shape
    a64 = _to64(a).reshape(H, F // H)
    ds64 = np.asarray(ds, np.float64)
    dm = (ds64[:, :, None] * a64[None] * np.where(m.reshape(E, H, F // H) > 0, 1.0, float(slope))).reshape(E, F)
    dXl, SXl = gather_backward(N, src, dm)
    dXr, SXr = gather_backward(N, dst, dm)
    t = ds64[:, :, None] * m.reshape(E, H, F // H)
    return dict(dXl=dXl, SXl=SXl, dXr=dXr, SXr=SXr, da=t.sum(0), Sda=np.abs(t).sum(0))


def hetero_propagate(N_dst, relations):
    """Heterogeneous graph: relations = list of dict(src, dst, X, w (or None), op ('sum' | 'mean')); every
    relation sends from its own source node set (rows of its X) to the same target node set; the results are
    summed over relations in list order -> (out [N_dst,F], S)."""
    out = S = None
    for r in relations:
        n_src = r["X"].shape[0]
        n = max(N_dst, n_src)
        Xp = r["X"]
        if n_src < n:  # the edge-list routine takes one node count: pad the source side with unused rows
            Xp = np.concatenate([Xp, np.zeros((n - n_src, Xp.shape[1]), Xp.dtype)])
        o, s, _ = propagate(r["op"], n, r["src"], r["dst"], Xp, r.get("w"))
        out = o[:N_dst] if out is None else out + o[:N_dst]
        S = s[:N_dst] if S is None else S + s[:N_dst]
    return out, S


def epilogue(Z, bias=None, act=None):
    """Element-wise tail of a layer: Z + bias (per feature), then ReLU if act == 'relu' (float64 in, float64 out)."""
    Y = np.asarray(Z, np.float64) + (0.0 if bias is None else np.asarray(bias, np.float64)[None, :])
    return np.maximum(Y, 0.0) if act == "relu" else Y


def epilogue_backward(Y, R, act=None):
    """For Y = epilogue(Z): dZ = R * [Y > 0] (ReLU) or R; dbias = column sums of dZ -> (dZ, dbias, Sdbias)."""
    dZ = _to64(R) * ((np.asarray(Y) > 0) if act == "relu" else 1.0)
    return dZ, dZ.sum(axis=0), np.abs(dZ).sum(axis=0)


def _to64(a):
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)
