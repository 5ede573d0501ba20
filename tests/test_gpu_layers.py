"""Layer-level runs of the workload configurations, composed from the C-ABI primitives only (no torch
arithmetic): GCN layer on the small random graph, GraphConv + mean pooling on the batch of small graphs,
SAGE (mean and max) on the power-law graph.  Each stage is checked against the CPU checker applied to the
device's own input of that stage (so storage rounding between stages is modelled exactly), and the final
output against the all-fp64 composition norm-wise."""
import numpy as np
import pytest

import oracle
from paper_2412_06354_b200 import synth
from util import assert_close, bits, f64_to_dtype_bits, to_dev, to_host64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gnn():
    from paper_2412_06354_b200 import gnn as g
    g.load()
    oracle.set_threads(8)
    yield g
    oracle.set_threads(1)


def host(t):
    """device tensor -> host array in the representation the checker reads (f32 array or bf16 bits)."""
    import torch
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def normwise(got, ref):
    return np.abs(got - ref).max() / np.abs(ref).max()


def as_dtype(a32, dtype):
    import torch
    if dtype == "f32":
        return a32
    return torch.from_numpy(a32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_gcn_layer_small_graph(gnn):
    """Y = D^-1/2 (A+I) D^-1/2 X W, fp32, forward and backward (dX, dW)."""
    wl = synth.workload_gcn_small()
    n, X, W = wl["N"], wl["X"], wl["W"]
    so, do = gnn.add_self_loops(n, to_dev(wl["src"]), to_dev(wl["dst"]))
    g = gnn.coo_to_csr(n, so, do)
    _, coef, coefT = gnn.gcn_norm(g)
    hs, hd = synth.with_self_loops(n, wl["src"], wl["dst"])
    eid = g.eid[:g.E].cpu().numpy()
    c32 = np.empty(len(hs), np.float32)
    c32[eid] = coef.cpu().numpy()
    XW = gnn.linear(to_dev(X), to_dev(W))
    o, S = oracle.matmul(X, W)
    assert_close(to_host64(XW), o, S, "f32", "X*W")
    Y = gnn.propagate_fused(g, XW, coef, "sum")
    o, S, _ = oracle.propagate("sum", n, hs, hd, host(XW), c32)
    assert_close(to_host64(Y), o, S, "f32", "propagate(X*W)")
    # against the all-fp64 layer
    c64 = oracle.gcn_norm(n, hs, hd)
    ref = oracle.aggregate("sum", n, hd, c64[:, None] * oracle.gather(hs, oracle.matmul(X, W)[0]))[0]
    assert normwise(to_host64(Y), ref) < 1e-5
    # backward
    R = synth.normal_f32(Y.shape, 31)
    dH, _ = gnn.propagate_fused_backward(g, to_dev(R), "sum", w_csrT=coefT)
    bw = oracle.propagate_backward("sum", n, hs, hd, None, c32, R)
    assert_close(to_host64(dH), bw["dX"], bw["SdX"], "f32", "dH")
    dX, dW = gnn.linear_backward(to_dev(X), to_dev(W), dH)
    o, S = oracle.matmul(host(dH), W, tb=True)
    assert_close(to_host64(dX), o, S, "f32", "dX")
    o, S = oracle.matmul(X, host(dH), ta=True)
    assert_close(to_host64(dW), o, S, "f32", "dW")


def test_graphconv_and_pooling_on_batch(gnn):
    """H = X W1 + mean_j(x_j) W2 on 512 block-diagonal graphs, P = mean-pool(H) [512,128]; fp32; fwd + bwd."""
    wl = synth.workload_batched()
    n, G, F, gp = wl["N"], wl["G"], wl["F"], wl["graph_ptr"]
    src, dst, X, W1, W2 = wl["src"], wl["dst"], wl["X"], wl["W1"], wl["W2"]
    g = gnn.coo_to_csr(n, to_dev(src), to_dev(dst))
    gptr = to_dev(gp.astype(np.int64))
    Xd = to_dev(X)
    A = gnn.propagate_fused(g, Xd, None, "mean")
    H1 = gnn.linear(Xd, to_dev(W1))
    H2 = gnn.linear(A, to_dev(W2))
    H = gnn.axpby(1.0, H1, 1.0, H2)
    P = gnn.reduce_nodes(gptr, H, "mean")
    # stage-wise
    o, S, _ = oracle.propagate("mean", n, src, dst, X)
    assert_close(to_host64(A), o, S, "f32", "mean aggregation")
    o, S = oracle.matmul(host(A), W2)
    assert_close(to_host64(H2), o, S, "f32", "agg*W2")
    h1, h2 = to_host64(H1), to_host64(H2)
    assert_close(to_host64(H), h1 + h2, np.abs(h1) + np.abs(h2), "f32", "sum of the two terms")
    o, S, _ = oracle.reduce_nodes("mean", gp, host(H))
    assert_close(to_host64(P), o, S, "f32", "pooling")
    # all-fp64 reference
    agg = oracle.propagate("mean", n, src, dst, X)[0]
    Href = oracle.matmul(X, W1)[0] + oracle.matmul(agg, W2)[0]
    Pref = oracle.reduce_nodes("mean", gp, Href)[0]
    assert P.shape == (512, 128) and normwise(to_host64(P), Pref) < 1e-5
    # backward for dL/dP = R
    R = synth.normal_f32((G, F), 32)
    dH = gnn.reduce_nodes_backward(gptr, to_dev(R), n, "mean")
    assert_close(to_host64(dH), oracle.reduce_nodes_backward("mean", gp, R), np.abs(oracle.reduce_nodes_backward("mean", gp, R)), "f32", "dH")
    dX1, dW1 = gnn.linear_backward(Xd, to_dev(W1), dH)
    dA, dW2 = gnn.linear_backward(A, to_dev(W2), dH)
    dX2, _ = gnn.propagate_fused_backward(g, dA, "mean")
    dX = gnn.axpby(1.0, dX1, 1.0, dX2)
    bw = oracle.propagate_backward("mean", n, src, dst, None, None, host(dA))
    assert_close(to_host64(dX2), bw["dX"], bw["SdX"], "f32", "dX through the aggregation")
    dHref = oracle.reduce_nodes_backward("mean", gp, R)
    dXref = oracle.matmul(dHref, W1, tb=True)[0] + oracle.propagate_backward("mean", n, src, dst, None, None, oracle.matmul(dHref, W2, tb=True)[0])["dX"]
    assert normwise(to_host64(dX), dXref) < 1e-5
    assert normwise(to_host64(dW2), oracle.matmul(agg, dHref, ta=True)[0]) < 1e-5
    assert normwise(to_host64(dW1), oracle.matmul(X, dHref, ta=True)[0]) < 1e-5


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("op", ["mean", "max"])
def test_sage_layer_powerlaw(gnn, dtype, op):
    """H = X W_self + agg_j(x_j) W_neigh on the 170k-node power-law graph, F = 128, agg = mean or max."""
    wl = synth.workload_powerlaw(dtype=dtype)
    n, F, src, dst, X = wl["N"], wl["F"], wl["src"], wl["dst"], wl["X"]
    Ws, Wn = as_dtype(wl["W_self"], dtype), as_dtype(wl["W_neigh"], dtype)
    g = gnn.coo_to_csr(n, to_dev(src), to_dev(dst))
    eid = g.eid[:g.E].cpu().numpy()
    Xd = to_dev(X)
    if op == "max":
        A, arg = gnn.propagate_fused(g, Xd, None, "max")
        o, _, a = oracle.propagate("max", n, src, dst, X)
        assert np.array_equal(bits(A), f64_to_dtype_bits(o, dtype))
    else:
        A, arg = gnn.propagate_fused(g, Xd, None, "mean"), None
        o, S, _ = oracle.propagate("mean", n, src, dst, X)
        assert_close(to_host64(A), o, S, dtype, "aggregation")
    H1, H2 = gnn.linear(Xd, to_dev(Ws)), gnn.linear(A, to_dev(Wn))
    H = gnn.axpby(1.0, H1, 1.0, H2)
    rows = np.random.default_rng(5).choice(n, 4000, replace=False)
    o, S = oracle.matmul(host(A)[rows], Wn)
    assert_close(to_host64(H2)[rows], o, S, dtype, "agg*W_neigh (sampled rows)")
    o, S = oracle.matmul(X[rows], Ws)
    assert_close(to_host64(H1)[rows], o, S, dtype, "X*W_self (sampled rows)")
    h1, h2 = to_host64(H1), to_host64(H2)
    assert_close(to_host64(H), h1 + h2, np.abs(h1) + np.abs(h2), dtype, "sum of the two terms")
    # backward
    R = synth.normal((n, F), dtype, 33)
    Rd = to_dev(R)
    dX1, dWs = gnn.linear_backward(Xd, to_dev(Ws), Rd)
    dA, dWn = gnn.linear_backward(A, to_dev(Wn), Rd)
    dX2, _ = gnn.propagate_fused_backward(g, dA, op, argmax=arg)
    dX = gnn.axpby(1.0, dX1, 1.0, dX2)
    bw = oracle.propagate_backward(op, n, src, dst, X, None, host(dA), arg=(a if op == "max" else None))
    assert_close(to_host64(dX2), bw["dX"], bw["SdX"], dtype, "dX through the aggregation")
    o, S = oracle.matmul(host(A), R, ta=True)
    assert_close(to_host64(dWn), o, S, dtype, "dW_neigh")
    o, S = oracle.matmul(R[rows], Wn, tb=True)
    assert_close(to_host64(dA)[rows], o, S, dtype, "dA (sampled rows)")
    d1, d2 = to_host64(dX1), to_host64(dX2)
    assert_close(to_host64(dX), d1 + d2, np.abs(d1) + np.abs(d2), dtype, "dX")
