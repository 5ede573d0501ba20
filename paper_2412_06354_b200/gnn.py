"""ctypes binding of libgnn_b200.so: argument marshalling only.

Every function here has the name of the C entry point without the ``gnn_`` prefix, takes torch
CUDA tensors (torch is used for device memory and streams, nothing else), allocates outputs and
workspaces when they are not passed in, and raises ``GnnError`` on a non-zero status.  There is no
CPU path: loading fails if the CUDA library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgnn_b200.so")
_lib = None

SUM, MEAN, MAX, MIN = 0, 1, 2, 3
COPY_XJ, E_MUL_XJ, GAT_LOGIT, XI_SUB_XJ, XI_DOT_XJ = 0, 1, 2, 3, 4
SELF_ALWAYS, SELF_TIMES_DEGREE, SELF_IF_NONEMPTY = 0, 1, 2
F32, BF16 = 0, 1
OPS = {"sum": SUM, "mean": MEAN, "max": MAX, "min": MIN}
STATUS_NAMES = ["OK", "INVALID_ARG", "INDEX_OUT_OF_RANGE", "NOT_SORTED", "WORKSPACE_TOO_SMALL", "UNSUPPORTED", "CUDA", "TIMEOUT"]


class GnnError(RuntimeError):
    def __init__(self, status, msg):
        super().__init__(f"gnn status {status} ({STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else '?'}): {msg}")
        self.status = status


class CsrStruct(C.Structure):
    _fields_ = [("N", C.c_int32), ("E", C.c_int64), ("rowptr", C.c_void_p), ("col", C.c_void_p), ("eid", C.c_void_p),
                ("rowptrT", C.c_void_p), ("colT", C.c_void_p), ("eidT", C.c_void_p), ("t2f", C.c_void_p)]


class RowEpilogueStruct(C.Structure):
    _fields_ = [("Xself", C.c_void_p), ("self_coef", C.c_float), ("self_mode", C.c_int), ("bias", C.c_void_p), ("relu", C.c_int)]


class EdgeSegmentStruct(C.Structure):
    _fields_ = [("E", C.c_int64), ("src", C.c_void_p), ("dst", C.c_void_p), ("src_offset", C.c_int32), ("dst_offset", C.c_int32)]


_VP, _I32, _I64, _INT, _SZ, _F = C.c_void_p, C.c_int32, C.c_int64, C.c_int, C.c_size_t, C.c_float
_CSR = C.POINTER(CsrStruct)
_EPI = C.POINTER(RowEpilogueStruct)
_SEG = C.POINTER(EdgeSegmentStruct)

# name -> (restype, argtypes); mirrors include/gnn.h
SIGNATURES = {
    "gnn_status_string": (C.c_char_p, [_INT]),
    "gnn_last_error_string": (C.c_char_p, []),
    "gnn_version": (_INT, []),
    "gnn_coo_to_csr_workspace": (_SZ, [_I32, _I64]),
    "gnn_coo_to_csr": (_INT, [_I32, _I64, _VP, _VP, _CSR, _VP, _SZ, _VP]),
    "gnn_probe_gather_sink_floats": (_SZ, [_I64]),
    "gnn_probe_gather": (_INT, [_VP, _I64, _VP, _I32, _INT, _VP, _VP]),
    "gnn_csr_validate_workspace": (_SZ, [_I64]),
    "gnn_csr_validate": (_INT, [_CSR, _VP, _SZ, _VP]),
    "gnn_degree": (_INT, [_CSR, _INT, _VP, _VP, _VP]),
    "gnn_add_self_loops": (_INT, [_I32, _I64, _VP, _VP, _VP, _VP, _VP]),
    "gnn_gcn_norm": (_INT, [_CSR, _VP, _VP, _VP, _VP, _VP]),
    "gnn_permute_edge_data": (_INT, [_VP, _I64, _INT, _INT, _VP, _VP, _VP]),
    "gnn_propagate_fused_workspace": (_SZ, [_I64, _INT, _INT]),
    "gnn_propagate_fused": (_INT, [_CSR, _INT, _INT, _VP, _VP, _INT, _INT, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_propagate_fused_backward": (_INT, [_CSR, _INT, _INT, _VP, _VP, _VP, _VP, _INT, _INT, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_propagate_fused_static_max_bytes": (_SZ, []),
    "gnn_propagate_fused_static": (_INT, [_CSR, _INT, _INT, _VP, _VP, _INT, _INT, _VP, _VP, _VP]),
    "gnn_propagate_msg": (_INT, [_CSR, _INT, _INT, _VP, _VP, _VP, _INT, _INT, _INT, _EPI, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_propagate_msg_backward": (_INT, [_CSR, _INT, _INT, _VP, _VP, _VP, _INT, _VP, _INT, _INT, _EPI, _VP, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_row_epilogue_backward_workspace": (_SZ, [_I32, _INT]),
    "gnn_row_epilogue_backward": (_INT, [_VP, _VP, _I32, _INT, _INT, _INT, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_gin_workspace": (_SZ, [_I64, _INT]),
    "gnn_gin": (_INT, [_CSR, _VP, _F, _INT, _INT, _VP, _VP, _SZ, _VP]),
    "gnn_gin_backward": (_INT, [_CSR, _VP, _VP, _F, _INT, _INT, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_edge_dot": (_INT, [_CSR, _VP, _VP, _INT, _INT, _INT, _VP, _VP]),
    "gnn_edge_dot_backward_workspace": (_SZ, [_I64, _INT, _INT]),
    "gnn_edge_dot_backward": (_INT, [_CSR, _VP, _VP, _VP, _INT, _INT, _INT, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_gatv2_logits": (_INT, [_CSR, _VP, _VP, _VP, _INT, _INT, _INT, _F, _VP, _VP]),
    "gnn_gatv2_logits_backward_workspace": (_SZ, [_I32, _INT, _INT]),
    "gnn_gatv2_logits_backward": (_INT, [_CSR, _VP, _VP, _VP, _VP, _INT, _INT, _INT, _F, _VP, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_merge_edge_lists": (_INT, [_SEG, _INT, _VP, _VP, _VP, _VP]),
    "gnn_segment_coef": (_INT, [_CSR, _VP, _VP, _VP, _INT, _VP, _VP, _VP]),
    "gnn_gather": (_INT, [_VP, _I64, _VP, _I32, _INT, _INT, _VP, _VP]),
    "gnn_gather_backward": (_INT, [_CSR, _INT, _VP, _INT, _INT, _VP, _VP, _SZ, _VP]),
    "gnn_apply_edges": (_INT, [_CSR, _INT, _VP, _VP, _VP, _INT, _INT, _INT, _F, _VP, _VP]),
    "gnn_aggregate": (_INT, [_CSR, _INT, _VP, _INT, _INT, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_aggregate_backward": (_INT, [_CSR, _INT, _VP, _VP, _INT, _INT, _VP, _VP]),
    "gnn_axpby": (_INT, [_F, _VP, _F, _VP, _I64, _INT, _VP, _VP]),
    "gnn_edge_softmax": (_INT, [_CSR, _VP, _INT, _INT, _VP, _VP, _VP, _VP]),
    "gnn_edge_softmax_backward": (_INT, [_CSR, _VP, _VP, _INT, _INT, _VP, _VP]),
    "gnn_gat_fused_workspace": (_SZ, [_I32, _I64, _INT, _INT, _INT]),
    "gnn_gat_fused": (_INT, [_CSR, _VP, _VP, _VP, _INT, _INT, _INT, _F, _VP, _VP, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_gat_fused_backward": (_INT, [_CSR, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _INT, _INT, _INT, _F, _VP, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_graph_ptr_from_ids": (_INT, [_VP, _I32, _I32, _VP, _VP, _SZ, _VP]),
    "gnn_reduce_nodes": (_INT, [_VP, _I32, _I32, _INT, _VP, _INT, _INT, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_reduce_nodes_backward": (_INT, [_VP, _I32, _I32, _INT, _VP, _VP, _INT, _INT, _VP, _VP]),
    "gnn_linear_workspace": (_SZ, [_I32, _INT, _INT]),
    "gnn_linear": (_INT, [_VP, _VP, _I32, _INT, _INT, _INT, _VP, _VP, _SZ, _VP]),
    "gnn_linear_bias_act": (_INT, [_VP, _VP, _I32, _INT, _INT, _INT, _VP, _INT, _VP, _VP, _SZ, _VP]),
    "gnn_propagate_linear_workspace": (_SZ, [_I32, _I64, _INT, _INT]),
    "gnn_propagate_linear": (_INT, [_CSR, _INT, _INT, _VP, _VP, _VP, _INT, _INT, _INT, _VP, _INT, _VP, _VP, _SZ, _VP]),
    "gnn_propagate_linear_backward": (_INT, [_CSR, _INT, _INT, _VP, _VP, _VP, _VP, _INT, _INT, _INT, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_linear_backward": (_INT, [_VP, _VP, _VP, _I32, _INT, _INT, _INT, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_propagate_fused_host": (_INT, [_CSR, _INT, _INT, _VP, _VP, _INT, _INT, _VP, _VP, _VP, _VP, _VP, _SZ, _VP]),
    "gnn_propagate_fused_backward_host": (_INT, [_CSR, _INT, _INT, _VP, _VP, _VP, _INT, _INT, _VP, _VP, _VP, _VP, _SZ, _VP]),
}


def load(path: str = LIB_PATH):
    """Load the CUDA library (no GPU needed to load it) and set the prototypes."""
    global _lib
    if _lib is None:
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: build it with `python -m paper_2412_06354_b200.build` "
                              "(there is no CPU fallback)")
        lib = C.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _check(rc):
    if rc != 0:
        raise GnnError(rc, load().gnn_last_error_string().decode())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _p(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _pi(t, dtype, name):
    """Pointer of an index tensor, after checking its element type (the C ABI cannot)."""
    if t is None:
        return None
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if t.numel() and not t.is_contiguous():
        raise TypeError(f"{name} must be contiguous")
    return C.c_void_p(t.data_ptr())


def _pf32(t, name):
    return _pi(t, torch.float32, name)


def _dtype(t):
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported feature dtype {t.dtype}")


def _op(op):
    return OPS[op] if isinstance(op, str) else int(op)


def _dev(t):
    assert t.is_cuda and t.is_contiguous(), "CUDA contiguous tensor expected"
    return t


class Graph:
    """Both sparse forms of a graph on the device (see gnn_csr in gnn.h)."""

    def __init__(self, N, E, device):
        i64 = dict(dtype=torch.int64, device=device)
        i32 = dict(dtype=torch.int32, device=device)
        self.N, self.E = int(N), int(E)
        self.rowptr = torch.empty(N + 1, **i64)
        self.rowptrT = torch.empty(N + 1, **i64)
        n = max(self.E, 1)
        self.col, self.eid, self.colT, self.eidT, self.t2f = (torch.empty(n, **i32) for _ in range(5))
        self.c = CsrStruct(self.N, self.E, *(t.data_ptr() for t in (self.rowptr, self.col, self.eid, self.rowptrT, self.colT, self.eidT, self.t2f)))

    @property
    def ref(self):
        return C.byref(self.c)

    def nbytes(self):
        return sum(t.numel() * t.element_size() for t in (self.rowptr, self.col, self.eid, self.rowptrT, self.colT, self.eidT, self.t2f))


# ------------------------------------------------------------------ graph set-up
def coo_to_csr(N, src, dst, ws=None) -> Graph:
    src, dst = _dev(src), _dev(dst)
    E = src.numel()
    g = Graph(N, E, src.device)
    need = load().gnn_coo_to_csr_workspace(N, E)
    if ws is None:
        ws = torch.empty(need, dtype=torch.uint8, device=src.device)
    _check(load().gnn_coo_to_csr(N, E, _pi(src, torch.int32, "src"), _pi(dst, torch.int32, "dst"), g.ref, _p(ws), ws.numel(), _stream()))
    return g


def probe_gather(col, X, row_bytes, sink=None):
    """The bare gathers of one pass over col (see gnn_probe_gather): returns the sink buffer."""
    E = col.numel()
    if sink is None:
        sink = torch.empty(load().gnn_probe_gather_sink_floats(E), dtype=torch.float32, device=col.device)
    _check(load().gnn_probe_gather(_pi(col, torch.int32, "col"), E, _p(X), X.shape[0], int(row_bytes), _p(sink), _stream()))
    return sink


def csr_validate(g: Graph, ws=None):
    """Raises GnnError (INVALID_ARG, the failed checks in its text) unless g is a sound sparse form."""
    if ws is None:
        ws = torch.empty(load().gnn_csr_validate_workspace(g.E), dtype=torch.uint8, device=g.rowptr.device)
    _check(load().gnn_csr_validate(g.ref, _p(ws), ws.numel(), _stream()))


def degree(g: Graph, transposed=False, w=None):
    out = torch.empty(g.N, dtype=torch.int32 if w is None else torch.float32, device=g.rowptr.device)
    _check(load().gnn_degree(g.ref, int(transposed), _p(w), _p(out), _stream()))
    return out


def add_self_loops(N, src, dst):
    E = src.numel()
    so = torch.empty(E + N, dtype=torch.int32, device=src.device)
    do = torch.empty(E + N, dtype=torch.int32, device=src.device)
    _check(load().gnn_add_self_loops(N, E, _pi(src, torch.int32, "src"), _pi(dst, torch.int32, "dst"), _p(so), _p(do), _stream()))
    return so, do


def gcn_norm(g: Graph, w_csr=None, want_T=True):
    dev = g.rowptr.device
    deg = torch.empty(g.N, dtype=torch.float32, device=dev)
    coef = torch.empty(max(g.E, 1), dtype=torch.float32, device=dev)
    coefT = torch.empty(max(g.E, 1), dtype=torch.float32, device=dev) if want_T else None
    _check(load().gnn_gcn_norm(g.ref, _pf32(w_csr, "w_csr"), _p(deg), _p(coef), _p(coefT), _stream()))
    return deg, coef[:g.E], (coefT[:g.E] if want_T else None)


def permute_edge_data(perm, x, out=None):
    x = _dev(x)
    E = perm.numel()
    width = x.numel() // max(E, 1) if E else 1
    if out is None:
        out = torch.empty_like(x)
    _check(load().gnn_permute_edge_data(_pi(perm, torch.int32, "perm"), E, max(width, 1), x.element_size(), _p(x), _p(out), _stream()))
    return out


# ------------------------------------------------------------------ fused propagate
def propagate_fused_workspace(E, F, op="sum"):
    return load().gnn_propagate_fused_workspace(E, F, _op(op))


def propagate_fused(g: Graph, X, w_csr=None, op="sum", out=None, argmax=None, ws=None):
    """-> out, or (out, argmax) for max/min."""
    X = _dev(X)
    F = X.shape[1]
    opc = _op(op)
    if out is None:
        out = torch.empty((g.N, F), dtype=X.dtype, device=X.device)
    if opc in (MAX, MIN) and argmax is None:
        argmax = torch.empty((g.N, F), dtype=torch.int32, device=X.device)
    if ws is None:
        ws = torch.empty(propagate_fused_workspace(g.E, F, opc), dtype=torch.uint8, device=X.device)
    msg = COPY_XJ if w_csr is None else E_MUL_XJ
    _check(load().gnn_propagate_fused(g.ref, msg, opc, _p(X), _pf32(w_csr, "w_csr"), F, _dtype(X), _p(out), _pi(argmax, torch.int32, "argmax"), _p(ws), ws.numel(), _stream()))
    return (out, argmax) if opc in (MAX, MIN) else out


def propagate_fused_backward(g: Graph, dOut, op="sum", X=None, w_csrT=None, argmax=None, want_dX=True, want_dW=False,
                             dX=None, dW=None, ws=None):
    """-> (dX or None, dW or None)."""
    dOut = _dev(dOut)
    F = dOut.shape[1]
    opc = _op(op)
    if want_dX and dX is None:
        dX = torch.empty((g.N, F), dtype=dOut.dtype, device=dOut.device)
    if want_dW and dW is None:
        dW = torch.empty(max(g.E, 1), dtype=torch.float32, device=dOut.device)
    if ws is None:
        ws = torch.empty(propagate_fused_workspace(g.E, F, opc), dtype=torch.uint8, device=dOut.device)
    msg = COPY_XJ if (w_csrT is None) else E_MUL_XJ
    _check(load().gnn_propagate_fused_backward(g.ref, msg, opc, _p(dOut), _p(X), _pf32(w_csrT, "w_csrT"), _pi(argmax, torch.int32, "argmax"), F, _dtype(dOut),
                                               _p(dX if want_dX else None), _p(dW if want_dW else None), _p(ws), ws.numel(), _stream()))
    return (dX if want_dX else None), (dW[:g.E] if want_dW else None)


def propagate_fused_host(g: Graph, h_X, w_csr, op, h_out, d_in, d_out, ws, argmax=None):
    """Host-buffer forward: h_X, h_out are (pinned) host tensors; d_in, d_out device staging."""
    F = h_X.shape[1]
    msg = COPY_XJ if w_csr is None else E_MUL_XJ
    _check(load().gnn_propagate_fused_host(g.ref, msg, _op(op), _p(h_X), _pf32(w_csr, "w_csr"), F, _dtype(h_X), _p(h_out), _pi(argmax, torch.int32, "argmax"),
                                           _p(d_in), _p(d_out), _p(ws), ws.numel(), _stream()))
    return h_out


def propagate_fused_backward_host(g: Graph, h_dOut, op, w_csrT, h_dX, d_in, d_out, ws, argmax=None):
    F = h_dOut.shape[1]
    msg = COPY_XJ if w_csrT is None else E_MUL_XJ
    _check(load().gnn_propagate_fused_backward_host(g.ref, msg, _op(op), _p(h_dOut), _pf32(w_csrT, "w_csrT"), _pi(argmax, torch.int32, "argmax"), F, _dtype(h_dOut),
                                                    _p(h_dX), _p(d_in), _p(d_out), _p(ws), ws.numel(), _stream()))
    return h_dX


# ------------------------------------------------------------------ more (message, op) pairs, GIN, XI_DOT_XJ
def _epi(epi):
    """dict(Xself=, self_coef=, self_mode=, bias=, relu=) -> (struct or None, the tensors it points to)."""
    if epi is None:
        return None, ()
    xs, b = epi.get("Xself"), epi.get("bias")
    st = RowEpilogueStruct(xs.data_ptr() if xs is not None else None, float(epi.get("self_coef", 0.0)),
                           int(epi.get("self_mode", SELF_ALWAYS)), _pf32(b, "bias").value if b is not None else None,
                           int(bool(epi.get("relu", False))))
    return C.byref(st), (st, xs, b)


def propagate_msg(g: Graph, msg, Xj, Xi=None, e_csr=None, op="sum", epi=None, out=None, argmax=None, ws=None):
    """gnn_propagate_msg -> out, or (out, argmax) for max/min.  e_csr: float32 [E] or [E,width] in CSR order."""
    Xj = _dev(Xj)
    F = Xj.shape[1]
    opc = _op(op)
    ew = 0 if e_csr is None else (1 if e_csr.dim() == 1 else e_csr.shape[1])
    if out is None:
        out = torch.empty((g.N, F), dtype=Xj.dtype, device=Xj.device)
    if opc in (MAX, MIN) and argmax is None:
        argmax = torch.empty((g.N, F), dtype=torch.int32, device=Xj.device)
    ws = _ws(g.E, F, opc, Xj.device, ws)
    ep, keep = _epi(epi)
    _check(load().gnn_propagate_msg(g.ref, msg, opc, _p(Xj), _p(Xi), _pf32(e_csr, "e_csr"), ew, F, _dtype(Xj), ep, _p(out),
                                    _pi(argmax, torch.int32, "argmax"), _p(ws), ws.numel(), _stream()))
    del keep
    return (out, argmax) if opc in (MAX, MIN) else out


def propagate_msg_backward(g: Graph, msg, dOut, op="sum", Xj=None, e_csrT=None, e_width=0, argmax=None, self_grad=None,
                           want_dXj=True, want_dXi=False, want_de=False, ws=None):
    """gnn_propagate_msg_backward -> dict(dXj, dXi, de) with None for the outputs not asked for."""
    dOut = _dev(dOut)
    F = dOut.shape[1]
    opc = _op(op)
    ew = e_width or (0 if e_csrT is None else (1 if e_csrT.dim() == 1 else e_csrT.shape[1]))
    dev = dOut.device
    dXj = torch.empty((g.N, F), dtype=dOut.dtype, device=dev) if want_dXj else None
    dXi = torch.empty((g.N, F), dtype=dOut.dtype, device=dev) if want_dXi else None
    de = torch.empty((max(g.E, 1), max(ew, 1)), dtype=torch.float32, device=dev) if want_de else None
    ws = _ws(g.E, F, opc, dev, ws)
    sg, keep = _epi(self_grad)
    _check(load().gnn_propagate_msg_backward(g.ref, msg, opc, _p(dOut), _p(Xj), _pf32(e_csrT, "e_csrT"), ew, _pi(argmax, torch.int32, "argmax"),
                                             F, _dtype(dOut), sg, _p(dXj), _p(dXi), _p(de), _p(ws), ws.numel(), _stream()))
    del keep
    return dict(dXj=dXj, dXi=dXi, de=None if de is None else de[:g.E])


def row_epilogue_backward(Y, dY, relu=True, want_dbias=True, dZ=None, ws=None):
    """-> (dZ, dbias or None)"""
    dY = _dev(dY)
    N, F = dY.shape
    if dZ is None:
        dZ = torch.empty_like(dY)
    dbias = torch.empty(F, dtype=torch.float32, device=dY.device) if want_dbias else None
    if ws is None:
        ws = torch.empty(load().gnn_row_epilogue_backward_workspace(N, F), dtype=torch.uint8, device=dY.device)
    _check(load().gnn_row_epilogue_backward(_p(Y), _p(dY), N, F, _dtype(dY), int(bool(relu)), _p(dZ), _p(dbias), _p(ws), ws.numel(), _stream()))
    return dZ, dbias


def gin(g: Graph, X, eps, out=None, ws=None):
    X = _dev(X)
    F = X.shape[1]
    if out is None:
        out = torch.empty((g.N, F), dtype=X.dtype, device=X.device)
    if ws is None:
        ws = torch.empty(load().gnn_gin_workspace(g.E, F), dtype=torch.uint8, device=X.device)
    _check(load().gnn_gin(g.ref, _p(X), float(eps), F, _dtype(X), _p(out), _p(ws), ws.numel(), _stream()))
    return out


def gin_backward(g: Graph, dOut, eps, X=None, want_deps=False, ws=None):
    """-> (dX, deps as a float32 device tensor of one element, or None)"""
    dOut = _dev(dOut)
    F = dOut.shape[1]
    dX = torch.empty((g.N, F), dtype=dOut.dtype, device=dOut.device)
    deps = torch.empty(1, dtype=torch.float32, device=dOut.device) if want_deps else None
    if ws is None:
        ws = torch.empty(load().gnn_gin_workspace(g.E, F), dtype=torch.uint8, device=dOut.device)
    _check(load().gnn_gin_backward(g.ref, _p(dOut), _p(X), float(eps), F, _dtype(dOut), _p(dX), _p(deps), _p(ws), ws.numel(), _stream()))
    return dX, deps


def edge_dot(g: Graph, Xj, Xi, H=1):
    """s[p,h] = <Xi[row(p),h,:], Xj[col[p],h,:]> -> float32 [E,H], CSR order."""
    Xj, Xi = _dev(Xj), _dev(Xi)
    F = Xj.shape[1]
    s = torch.empty((max(g.E, 1), H), dtype=torch.float32, device=Xj.device)
    _check(load().gnn_edge_dot(g.ref, _p(Xj), _p(Xi), H, F // H, _dtype(Xj), _p(s), _stream()))
    return s[:g.E]


def edge_dot_backward(g: Graph, Xj, Xi, ds_csr, H=1, want_dXj=True, want_dXi=True, ws=None):
    Xj, Xi = _dev(Xj), _dev(Xi)
    N, F = Xj.shape
    dXj = torch.empty_like(Xj) if want_dXj else None
    dXi = torch.empty_like(Xi) if want_dXi else None
    if ws is None:
        ws = torch.empty(load().gnn_edge_dot_backward_workspace(g.E, H, F // H), dtype=torch.uint8, device=Xj.device)
    _check(load().gnn_edge_dot_backward(g.ref, _p(Xj), _p(Xi), _pf32(ds_csr, "ds_csr"), H, F // H, _dtype(Xj), _p(dXj), _p(dXi), _p(ws), ws.numel(), _stream()))
    return dXj, dXi


def gatv2_logits(g: Graph, Xl, Xr, a, H, slope=0.2):
    """s[p,h] = sum_c a[h,c] * LeakyReLU(Xl[col[p],h,c] + Xr[row(p),h,c]) -> float32 [E,H], CSR order."""
    Xl, Xr = _dev(Xl), _dev(Xr)
    F = Xl.shape[1]
    s = torch.empty((max(g.E, 1), H), dtype=torch.float32, device=Xl.device)
    _check(load().gnn_gatv2_logits(g.ref, _p(Xl), _p(Xr), _pf32(a, "a"), H, F // H, _dtype(Xl), float(slope), _p(s), _stream()))
    return s[:g.E]


def gatv2_logits_backward(g: Graph, Xl, Xr, a, ds_csr, H, slope=0.2, ws=None):
    """-> (dXl, dXr, da)"""
    Xl, Xr = _dev(Xl), _dev(Xr)
    N, F = Xl.shape
    dXl, dXr = torch.empty_like(Xl), torch.empty_like(Xr)
    da = torch.empty((H, F // H), dtype=torch.float32, device=Xl.device)
    if ws is None:
        ws = torch.empty(load().gnn_gatv2_logits_backward_workspace(N, H, F // H), dtype=torch.uint8, device=Xl.device)
    _check(load().gnn_gatv2_logits_backward(g.ref, _p(Xl), _p(Xr), _pf32(a, "a"), _pf32(ds_csr, "ds_csr"), H, F // H, _dtype(Xl), float(slope),
                                            _p(dXl), _p(dXr), _p(da), _p(ws), ws.numel(), _stream()))
    return dXl, dXr, da


# ------------------------------------------------------------------ heterogeneous / temporal graphs
def merge_edge_lists(segments):
    """segments: list of (src, dst, src_offset, dst_offset) with int32 device tensors -> (src, dst, seg) of the merged list."""
    S = len(segments)
    arr = (EdgeSegmentStruct * S)()
    total = 0
    for k, (src, dst, so, do) in enumerate(segments):
        arr[k] = EdgeSegmentStruct(src.numel(), _pi(src, torch.int32, "src").value if src.numel() else None,
                                   _pi(dst, torch.int32, "dst").value if dst.numel() else None, int(so), int(do))
        total += src.numel()
    dev = segments[0][0].device
    so_, do_, sg_ = (torch.empty(max(total, 1), dtype=torch.int32, device=dev) for _ in range(3))
    _check(load().gnn_merge_edge_lists(arr, S, _p(so_), _p(do_), _p(sg_), _stream()))
    return so_[:total], do_[:total], sg_[:total]


def segment_coef(g: Graph, seg_csr, seg_is_mean, w_csr=None, want_T=True):
    """-> (coef_csr, coef_csrT or None): per-position multipliers of a merged multi-relation / multi-snapshot form."""
    dev = g.rowptr.device
    coef = torch.empty(max(g.E, 1), dtype=torch.float32, device=dev)
    coefT = torch.empty(max(g.E, 1), dtype=torch.float32, device=dev) if want_T else None
    _check(load().gnn_segment_coef(g.ref, _pi(seg_csr, torch.int32, "seg_csr"), _pf32(w_csr, "w_csr"), _pi(seg_is_mean, torch.int32, "seg_is_mean"),
                                   seg_is_mean.numel(), _p(coef), _p(coefT), _stream()))
    return coef[:g.E], (coefT[:g.E] if want_T else None)


# ------------------------------------------------------------------ unfused primitives
def _ws(E, F, op, device, ws):
    if ws is None:
        ws = torch.empty(propagate_fused_workspace(E, F, op), dtype=torch.uint8, device=device)
    return ws


def gather(idx, X, out=None):
    X = _dev(X)
    E, F = idx.numel(), X.shape[1]
    if out is None:
        out = torch.empty((E, F), dtype=X.dtype, device=X.device)
    _check(load().gnn_gather(_pi(idx, torch.int32, "idx"), E, _p(X), X.shape[0], F, _dtype(X), _p(out), _stream()))
    return out


def gather_backward(g: Graph, dOut_EF, by_src=False, ws=None):
    dOut_EF = _dev(dOut_EF)
    F = dOut_EF.shape[1]
    dX = torch.empty((g.N, F), dtype=dOut_EF.dtype, device=dOut_EF.device)
    ws = _ws(g.E, F, SUM, dOut_EF.device, ws)
    _check(load().gnn_gather_backward(g.ref, int(by_src), _p(dOut_EF), F, _dtype(dOut_EF), _p(dX), _p(ws), ws.numel(), _stream()))
    return dX


def apply_edges(g: Graph, msg, X, ar=None, e=None, slope=0.2):
    """COPY_XJ / E_MUL_XJ: X [N,F], e float32 [E] or [E,w] (CSR order) -> m [E,F] of X.dtype.
    GAT_LOGIT: X = al, ar float32 [N,H] -> float32 [E,H]."""
    X = _dev(X)
    F = X.shape[1]
    ew = 0 if e is None else (1 if e.dim() == 1 else e.shape[1])
    m = torch.empty((max(g.E, 1), F), dtype=X.dtype, device=X.device)
    _check(load().gnn_apply_edges(g.ref, msg, _p(X), _p(ar), _p(e), ew, F, _dtype(X), float(slope), _p(m), _stream()))
    return m[:g.E]


def aggregate(g: Graph, m_EF, op="sum", ws=None):
    m_EF = _dev(m_EF)
    F = m_EF.shape[1]
    opc = _op(op)
    out = torch.empty((g.N, F), dtype=m_EF.dtype, device=m_EF.device)
    argmax = torch.empty((g.N, F), dtype=torch.int32, device=m_EF.device) if opc in (MAX, MIN) else None
    ws = _ws(g.E, F, opc, m_EF.device, ws)
    _check(load().gnn_aggregate(g.ref, opc, _p(m_EF), F, _dtype(m_EF), _p(out), _pi(argmax, torch.int32, "argmax"), _p(ws), ws.numel(), _stream()))
    return (out, argmax) if opc in (MAX, MIN) else out


def aggregate_backward(g: Graph, dOut, op="sum", argmax=None):
    dOut = _dev(dOut)
    F = dOut.shape[1]
    dm = torch.empty((max(g.E, 1), F), dtype=dOut.dtype, device=dOut.device)
    _check(load().gnn_aggregate_backward(g.ref, _op(op), _p(dOut), _pi(argmax, torch.int32, "argmax"), F, _dtype(dOut), _p(dm), _stream()))
    return dm[:g.E]


def edge_softmax(g: Graph, logits, want_stats=False):
    logits = _dev(logits)
    H = logits.shape[1]
    alpha = torch.empty_like(logits)
    rmax = torch.empty((g.N, H), dtype=torch.float32, device=logits.device) if want_stats else None
    rsum = torch.empty((g.N, H), dtype=torch.float32, device=logits.device) if want_stats else None
    _check(load().gnn_edge_softmax(g.ref, _p(logits), H, _dtype(logits), _p(alpha), _p(rmax), _p(rsum), _stream()))
    return (alpha, rmax, rsum) if want_stats else alpha


def edge_softmax_backward(g: Graph, alpha, dalpha):
    alpha, dalpha = _dev(alpha), _dev(dalpha)
    ds = torch.empty_like(alpha)
    _check(load().gnn_edge_softmax_backward(g.ref, _p(alpha), _p(dalpha), alpha.shape[1], _dtype(alpha), _p(ds), _stream()))
    return ds


# ------------------------------------------------------------------ pooling
def graph_ptr_from_ids(graph_id, G):
    N = graph_id.numel()
    gptr = torch.empty(G + 1, dtype=torch.int64, device=graph_id.device)
    ws = torch.empty(256, dtype=torch.uint8, device=graph_id.device)
    _check(load().gnn_graph_ptr_from_ids(_pi(graph_id, torch.int32, "graph_id"), N, G, _p(gptr), _p(ws), ws.numel(), _stream()))
    return gptr


def reduce_nodes(graph_ptr, X, op="mean", ws=None):
    X = _dev(X)
    G, (N, F) = graph_ptr.numel() - 1, X.shape
    opc = _op(op)
    out = torch.empty((G, F), dtype=X.dtype, device=X.device)
    argmax = torch.empty((G, F), dtype=torch.int32, device=X.device) if opc in (MAX, MIN) else None
    ws = _ws(N, F, opc, X.device, ws)
    _check(load().gnn_reduce_nodes(_pi(graph_ptr, torch.int64, "graph_ptr"), G, N, opc, _p(X), F, _dtype(X), _p(out), _pi(argmax, torch.int32, "argmax"), _p(ws), ws.numel(), _stream()))
    return (out, argmax) if opc in (MAX, MIN) else out


def reduce_nodes_backward(graph_ptr, dOut, N, op="mean", argmax=None):
    dOut = _dev(dOut)
    G, F = dOut.shape
    dX = torch.empty((N, F), dtype=dOut.dtype, device=dOut.device)
    _check(load().gnn_reduce_nodes_backward(_pi(graph_ptr, torch.int64, "graph_ptr"), G, N, _op(op), _p(dOut), _pi(argmax, torch.int32, "argmax"), F, _dtype(dOut), _p(dX), _stream()))
    return dX


# ------------------------------------------------------------------ GAT
def gat_fused(g: Graph, Wx, a_src, a_dst, H, slope=0.2, ws=None):
    """Wx [N, H*C] -> dict(out, alpha (float32 [E,H], CSR order), al, ar (float32 [N,H]))."""
    Wx = _dev(Wx)
    N, F = Wx.shape
    Cw = F // H
    dev = Wx.device
    out = torch.empty_like(Wx)
    alpha = torch.empty((max(g.E, 1), H), dtype=torch.float32, device=dev)
    al = torch.empty((N, H), dtype=torch.float32, device=dev)
    ar = torch.empty((N, H), dtype=torch.float32, device=dev)
    if ws is None:
        ws = torch.empty(load().gnn_gat_fused_workspace(N, g.E, H, Cw, 0), dtype=torch.uint8, device=dev)
    _check(load().gnn_gat_fused(g.ref, _p(Wx), _p(a_src), _p(a_dst), H, Cw, _dtype(Wx), float(slope), _p(out), _p(alpha),
                                _p(al), _p(ar), _p(ws), ws.numel(), _stream()))
    return dict(out=out, alpha=alpha[:g.E], al=al, ar=ar)


def gat_fused_backward(g: Graph, Wx, a_src, a_dst, fwd, dOut, H, slope=0.2, ws=None):
    Wx, dOut = _dev(Wx), _dev(dOut)
    N, F = Wx.shape
    Cw = F // H
    dev = Wx.device
    dWx = torch.empty_like(Wx)
    da_src = torch.empty((H, Cw), dtype=torch.float32, device=dev)
    da_dst = torch.empty((H, Cw), dtype=torch.float32, device=dev)
    if ws is None:
        ws = torch.empty(load().gnn_gat_fused_workspace(N, g.E, H, Cw, 1), dtype=torch.uint8, device=dev)
    _check(load().gnn_gat_fused_backward(g.ref, _p(Wx), _p(a_src), _p(a_dst), _p(fwd["alpha"]), _p(fwd["al"]), _p(fwd["ar"]),
                                         _p(dOut), H, Cw, _dtype(Wx), float(slope), _p(dWx), _p(da_src), _p(da_dst),
                                         _p(ws), ws.numel(), _stream()))
    return dict(dWx=dWx, da_src=da_src, da_dst=da_dst)


def propagate_fused_static(g: Graph, X, w_csr=None, op="sum", out=None, argmax=None):
    """gnn_propagate_fused_static: the fused propagate with the library's built-in 8 MiB scratch, for
    embedders that may not allocate device memory.  The caller passes `out` (and `argmax` for max/min);
    nothing is allocated here when they are given."""
    X = _dev(X)
    F = X.shape[1]
    opc = _op(op)
    if out is None:
        out = torch.empty((g.N, F), dtype=X.dtype, device=X.device)
    if opc in (MAX, MIN) and argmax is None:
        argmax = torch.empty((g.N, F), dtype=torch.int32, device=X.device)
    msg = COPY_XJ if w_csr is None else E_MUL_XJ
    _check(load().gnn_propagate_fused_static(g.ref, msg, opc, _p(X), _pf32(w_csr, "w_csr"), F, _dtype(X), _p(out), _pi(argmax, torch.int32, "argmax"), _stream()))
    return (out, argmax) if opc in (MAX, MIN) else out


# ------------------------------------------------------------------ dense transform
def linear(X, W, ws=None, return_ws=False):
    X, W = _dev(X), _dev(W)
    (N, K), M = X.shape, W.shape[1]
    Y = torch.empty((N, M), dtype=X.dtype, device=X.device)
    if ws is None:
        ws = torch.empty(load().gnn_linear_workspace(N, K, M), dtype=torch.uint8, device=X.device)
    _check(load().gnn_linear(_p(X), _p(W), N, K, M, _dtype(X), _p(Y), _p(ws), ws.numel(), _stream()))
    return (Y, ws) if return_ws else Y


def linear_bias_act(X, W, bias=None, relu=False, ws=None):
    """Y = act(X W + bias) with the tail inside the product kernel's epilogue."""
    X, W = _dev(X), _dev(W)
    (N, K), M = X.shape, W.shape[1]
    Y = torch.empty((N, M), dtype=X.dtype, device=X.device)
    if ws is None:
        ws = torch.empty(load().gnn_linear_workspace(N, K, M), dtype=torch.uint8, device=X.device)
    _check(load().gnn_linear_bias_act(_p(X), _p(W), N, K, M, _dtype(X), _pf32(bias, "bias"), int(bool(relu)), _p(Y), _p(ws), ws.numel(), _stream()))
    return Y


def propagate_linear(g: Graph, X, W, w_csr=None, op="sum", bias=None, relu=False, ws=None, return_ws=False):
    """Y = act((op over incoming edges of w * X[source]) W + bias) in one kernel."""
    X, W = _dev(X), _dev(W)
    K, M = W.shape
    Y = torch.empty((g.N, M), dtype=X.dtype, device=X.device)
    if ws is None:
        ws = torch.empty(load().gnn_propagate_linear_workspace(g.N, g.E, K, M), dtype=torch.uint8, device=X.device)
    msg = COPY_XJ if w_csr is None else E_MUL_XJ
    _check(load().gnn_propagate_linear(g.ref, msg, _op(op), _p(X), _pf32(w_csr, "w_csr"), _p(W), K, M, _dtype(X), _pf32(bias, "bias"),
                                       int(bool(relu)), _p(Y), _p(ws), ws.numel(), _stream()))
    return (Y, ws) if return_ws else Y


def propagate_linear_backward(g: Graph, dY, X, W, w_csrT=None, op="sum", want_dX=True, want_dW=True, ws=None):
    """-> (dX or None, dW or None)"""
    dY, W = _dev(dY), _dev(W)
    K, M = W.shape
    dX = torch.empty((g.N, K), dtype=dY.dtype, device=dY.device) if want_dX else None
    dW = torch.empty((K, M), dtype=dY.dtype, device=dY.device) if want_dW else None
    if ws is None:
        ws = torch.empty(load().gnn_propagate_linear_workspace(g.N, g.E, K, M), dtype=torch.uint8, device=dY.device)
    msg = COPY_XJ if w_csrT is None else E_MUL_XJ
    _check(load().gnn_propagate_linear_backward(g.ref, msg, _op(op), _p(dY), _p(X), _pf32(w_csrT, "w_csrT"), _p(W), K, M, _dtype(dY),
                                                _p(dX), _p(dW), _p(ws), ws.numel(), _stream()))
    return dX, dW


def linear_backward(X, W, dY, want_dX=True, want_dW=True, ws=None, return_ws=False):
    dY = _dev(dY)
    N, M = dY.shape
    K = W.shape[0] if W is not None else X.shape[1]
    dX = torch.empty((N, K), dtype=dY.dtype, device=dY.device) if want_dX else None
    dW = torch.empty((K, M), dtype=dY.dtype, device=dY.device) if want_dW else None
    if ws is None:
        ws = torch.empty(load().gnn_linear_workspace(N, K, M), dtype=torch.uint8, device=dY.device)
    _check(load().gnn_linear_backward(_p(X), _p(W), _p(dY), N, K, M, _dtype(dY), _p(dX), _p(dW), _p(ws), ws.numel(), _stream()))
    return (dX, dW, ws) if return_ws else (dX, dW)


def axpby(alpha, a, beta, b, out=None):
    a, b = _dev(a), _dev(b)
    if out is None:
        out = torch.empty_like(a)
    _check(load().gnn_axpby(float(alpha), _p(a), float(beta), _p(b), a.numel(), _dtype(a), _p(out), _stream()))
    return out
