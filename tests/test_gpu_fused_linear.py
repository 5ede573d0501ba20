"""GPU parity of the aggregate -> transform fusion (one kernel for propagate followed by the layer weight) and of
the bias / relu epilogue of the dense transform, against the CPU checker: the checker aggregates, rounds the
aggregated matrix to the storage type where the device does (bf16), and multiplies by a triple loop."""
import numpy as np
import pytest

import oracle
from paper_2412_06354_b200 import synth
from test_gpu_propagate import build_graph, feats, host_csr, ragged_graph
from util import assert_close, bits, to_dev, to_host64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gnn():
    import torch
    from paper_2412_06354_b200 import gnn as g
    g.load()
    assert torch.cuda.is_available()
    oracle.set_threads(8)
    yield g
    oracle.set_threads(1)


def to_bf16_bits(a64):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a64)).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def weights(K, M, dtype, seed):
    W = synth.glorot_f32(K, M, seed)
    return W if dtype == "f32" else to_bf16_bits(W.astype(np.float64))


def reference(dtype, H, SH, W):
    """(Y, S, extra) for Y = H * W where H is the aggregated matrix in fp64 and SH its magnitude sums.
    bf16: the device rounds each aggregated value to bf16 once; where the fp64 value lies within the fp32
    accumulation error of a rounding boundary the device may round the other way, which moves Y by one bf16
    step of that value times |W|: that is the per-element allowance `extra`.  fp32: the aggregated value enters
    the product exactly as accumulated, so its accumulation error 1e-5 * SH carries through |W|."""
    Wabs = np.abs(synth.to_f64(W))
    if dtype == "f32":
        Y, S = oracle.matmul(H, synth.to_f64(W))
        return Y, oracle.matmul(SH, Wabs)[0], None
    Hq = to_bf16_bits(H)
    Y, S = oracle.matmul(Hq, W)
    hq = synth.to_f64(Hq)
    step = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(H), 1e-300))) - 7)  # spacing of bf16 values around H
    near = np.abs(np.abs(H - hq) - 0.5 * step) <= 1e-5 * SH + 1e-30
    extra = oracle.matmul(near * step, Wabs)[0] + 1e-5 * oracle.matmul(SH, Wabs)[0]
    return Y, S, extra


SHAPES = [("bf16", 64, 64), ("bf16", 128, 128), ("bf16", 256, 256), ("bf16", 128, 48), ("bf16", 32, 256),
          ("f32", 64, 64), ("f32", 128, 128), ("f32", 16, 32), ("f32", 128, 64)]


@pytest.mark.parametrize("dtype,K,M", SHAPES)
@pytest.mark.parametrize("op,weighted", [("sum", True), ("mean", False)])
def test_fused_forward(gnn, dtype, K, M, op, weighted):
    n, src, dst = ragged_graph(110 + K + M)  # one 6000-edge hub (split over warps), short rows, rows without edges
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    X = feats((n, K), dtype, 1100 + K)
    W = weights(K, M, dtype, 1101 + M)
    w = synth.uniform_f32((len(src),), 0.0, 1.0, 18) if weighted else None
    w_csr = to_dev(w[ref["eid"]]) if weighted else None
    Y = gnn.propagate_linear(g, to_dev(X), to_dev(W), w_csr=w_csr, op=op)
    H, SH, _ = oracle.propagate(op, n, src, dst, X, w)
    o, S, extra = reference(dtype, H, SH, W)
    assert_close(to_host64(Y), o, S, dtype, f"fused {op} K={K} M={M}", extra=extra)
    again = gnn.propagate_linear(g, to_dev(X), to_dev(W), w_csr=w_csr, op=op)
    assert np.array_equal(bits(Y), bits(again)), "not bit-reproducible"
    # the unfused sequence gives the same result up to the rounding of the stored intermediate
    Hd = gnn.propagate_fused(g, to_dev(X), w_csr, op)
    Yu = gnn.linear(Hd, to_dev(W))
    assert_close(to_host64(Yu), o, S, dtype, "unfused sequence", extra=extra)


@pytest.mark.parametrize("dtype,K,M", [("bf16", 128, 128), ("bf16", 256, 64), ("f32", 64, 64), ("f32", 128, 128)])
def test_fused_forward_with_bias_and_relu(gnn, dtype, K, M):
    n, src, dst = ragged_graph(120 + K + M)
    g = build_graph(gnn, n, src, dst)
    X = feats((n, K), dtype, 1200 + K)
    W = weights(K, M, dtype, 1201 + M)
    bias = synth.uniform_f32((M,), -0.3, 0.3, 19)
    Y = gnn.propagate_linear(g, to_dev(X), to_dev(W), op="mean", bias=to_dev(bias), relu=True)
    H, SH, _ = oracle.propagate("mean", n, src, dst, X)
    z, S, extra = reference(dtype, H, SH, W)
    extra = (0.0 if extra is None else extra) + (1e-5 if dtype == "f32" else 0.0) * 0
    assert_close(to_host64(Y), oracle.epilogue(z, bias, "relu"), S + np.abs(bias)[None, :], dtype, "fused + bias + relu",
                 extra=None if dtype == "f32" else extra)


@pytest.mark.parametrize("dtype,K,M", [("bf16", 128, 128), ("bf16", 64, 256), ("f32", 64, 64), ("f32", 128, 128)])
@pytest.mark.parametrize("op", ["sum", "mean"])
@pytest.mark.parametrize("want_dW", [False, True])
def test_fused_backward(gnn, dtype, K, M, op, want_dW):
    n, src, dst = ragged_graph(130 + K + M)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    X = feats((n, K), dtype, 1300 + K)
    W = weights(K, M, dtype, 1301 + M)
    R = feats((n, M), dtype, 1302 + M, stream=1)
    w = synth.uniform_f32((len(src),), 0.0, 1.0, 20)
    dX, dW = gnn.propagate_linear_backward(g, to_dev(R), to_dev(X), to_dev(W), w_csrT=to_dev(w[ref["eidT"]]), op=op, want_dW=want_dW)
    bw = oracle.propagate_backward(op, n, src, dst, None, w, R)  # G = A^T dY
    G, SG = bw["dX"], bw["SdX"]
    Wt = np.ascontiguousarray(W.T)
    o, S, extra = reference(dtype, G, SG, Wt)
    assert_close(to_host64(dX), o, S, dtype, f"dX {op}", extra=extra)
    if want_dW:
        # dW = X^T G with G stored in the call's dtype by the device
        Gq = G if dtype == "f32" else to_bf16_bits(G)
        o, S = oracle.matmul(X, Gq, ta=True)
        slack = oracle.matmul(np.abs(synth.to_f64(X)), (1e-5 if dtype == "f32" else 2.0 ** -8) * SG, ta=True)[0]
        assert_close(to_host64(dW), o, S, dtype, f"dW {op}", extra=slack)


@pytest.mark.parametrize("dtype,N,K,M", [("bf16", 5000, 128, 128), ("bf16", 300, 64, 256), ("f32", 4000, 128, 128), ("f32", 1000, 64, 64),
                                         ("f32", 700, 20, 12), ("bf16", 900, 24, 40), ("f32", 513, 256, 256)])
def test_linear_bias_relu_epilogue(gnn, dtype, N, K, M):
    """The dense transform with its bias / relu tail, on the tensor-core paths (epilogue inside the kernel) and on the
    shapes that fall to the other kernels (one more pass)."""
    X = feats((N, K), dtype, 1400 + K)
    W = weights(K, M, dtype, 1401 + M)
    bias = synth.uniform_f32((M,), -0.5, 0.5, 21)
    Y = gnn.linear_bias_act(to_dev(X), to_dev(W), to_dev(bias), relu=True)
    z, S = oracle.matmul(X, W)
    assert_close(to_host64(Y), oracle.epilogue(z, bias, "relu"), S + np.abs(bias)[None, :], dtype, "X*W + bias, relu")
    Yb = gnn.linear_bias_act(to_dev(X), to_dev(W), to_dev(bias), relu=False)
    assert_close(to_host64(Yb), oracle.epilogue(z, bias, None), S + np.abs(bias)[None, :], dtype, "X*W + bias")
    # backward of the tail, then of the product
    R = feats((N, M), dtype, 1402 + M, stream=1)
    dZ, dbias = gnn.row_epilogue_backward(Y, to_dev(R), relu=True)
    rz, rb, rS = oracle.epilogue_backward(to_host64(Y), R, "relu")
    assert np.array_equal(to_host64(dZ), rz)
    assert_close(to_host64(dbias)[None, :], rb[None, :], rS[None, :], "f32", "dbias")
