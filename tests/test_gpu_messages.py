"""GPU parity of the further fused (message, op) pairs: x_i - x_j, edge factors per head and per feature,
GIN, the bias / relu row epilogue, and the per-head dot-product message, forward and backward, against
the CPU checker through the C ABI."""
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
    return g


def eid_of(arg, eid):
    a = arg.cpu().numpy()
    return np.where(a >= 0, eid[np.maximum(a, 0)], -1)


def absval(a):
    """|a| for float32 arrays and for bf16 bit patterns."""
    return (a & np.uint16(0x7FFF)) if a.dtype == np.uint16 else np.abs(a)


# rows up to 512 bytes take the position-first kernel on these graphs, wider rows the row-walking one
SUB_SHAPES = [("f32", 64), ("f32", 256), ("bf16", 32), ("bf16", 128), ("bf16", 1024)]


@pytest.mark.parametrize("dtype,F", SUB_SHAPES)
@pytest.mark.parametrize("op", ["sum", "mean", "max", "min"])
def test_xi_sub_xj(gnn, dtype, F, op):
    n, src, dst = ragged_graph(60 + F)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    Xj = feats((n, F), dtype, 600 + F)
    Xi = feats((n, F), dtype, 601 + F, stream=1)
    R = feats((n, F), dtype, 602 + F, stream=2)
    res = gnn.propagate_msg(g, gnn.XI_SUB_XJ, to_dev(Xj), Xi=to_dev(Xi), op=op)
    o, S, a = oracle.propagate_msg(oracle.XI_SUB_XJ, op, n, src, dst, Xj, Xi=Xi)
    arg = None
    if op in ("max", "min"):
        out, arg = res
        # the winner is unique: first edge of the row among equal differences
        assert np.array_equal(eid_of(arg, ref["eid"]), a), "winner differs"
        S = np.abs(o)  # one subtraction, rounded once
    else:
        out = res
        # the device forms c(i) * x_i - (sum or mean of x_j): the scale of its rounding error is the sum of
        # the magnitudes of those terms
        deg = np.bincount(dst, minlength=n).astype(np.float64)[:, None]
        sj = oracle.propagate(op, n, src, dst, absval(Xj))[0]
        S = sj + (deg if op == "sum" else (deg > 0)) * synth.to_f64(absval(Xi))
    assert_close(to_host64(out), o, S, dtype, f"x_i - x_j {op}")
    again = gnn.propagate_msg(g, gnn.XI_SUB_XJ, to_dev(Xj), Xi=to_dev(Xi), op=op)
    assert np.array_equal(bits(out), bits(again[0] if arg is not None else again)), "not bit-reproducible"
    # backward: both inputs separately
    bw = gnn.propagate_msg_backward(g, gnn.XI_SUB_XJ, to_dev(R), op=op, argmax=arg, want_dXi=True)
    rb = oracle.propagate_msg_backward(oracle.XI_SUB_XJ, op, n, src, dst, Xj, R, Xi=Xi, arg=a if arg is not None else None, want=("dXj", "dXi"))
    assert_close(to_host64(bw["dXj"]), rb["dXj"], rb["SXj"], dtype, f"dXj {op}")
    assert_close(to_host64(bw["dXi"]), rb["dXi"], rb["SXi"], dtype, f"dXi {op}")
    # one tensor on both sides: the self gradient joins the same pass
    mode = gnn.SELF_TIMES_DEGREE if op == "sum" else gnn.SELF_IF_NONEMPTY
    Rd = to_dev(R)
    both = gnn.propagate_msg_backward(g, gnn.XI_SUB_XJ, Rd, op=op, argmax=arg, self_grad=dict(Xself=Rd, self_coef=1.0, self_mode=mode))
    assert_close(to_host64(both["dXj"]), rb["dXj"] + rb["dXi"], rb["SXj"] + rb["SXi"], dtype, f"dX (shared tensor) {op}")


@pytest.mark.parametrize("dtype,F,H", [("f32", 64, 4), ("f32", 256, 8), ("bf16", 64, 2), ("bf16", 256, 8), ("bf16", 512, 4)])
@pytest.mark.parametrize("width", ["H", "F"])
@pytest.mark.parametrize("op", ["sum", "mean"])
def test_edge_factors_per_head_and_per_feature(gnn, dtype, F, H, width, op):
    n, src, dst = ragged_graph(70 + F)
    E = len(src)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    ew = H if width == "H" else F
    X = feats((n, F), dtype, 700 + F)
    R = feats((n, F), dtype, 701 + F, stream=1)
    e = synth.uniform_f32((E, ew), -1.0, 1.0, 13)
    e_csr, e_csrT = to_dev(e[ref["eid"]]), to_dev(e[ref["eidT"]])
    out = gnn.propagate_msg(g, gnn.E_MUL_XJ, to_dev(X), e_csr=e_csr, op=op)
    o, S, _ = oracle.propagate_msg(oracle.E_MUL_XJ, op, n, src, dst, X, e=e)
    assert_close(to_host64(out), o, S, dtype, f"e_mul_xj width {ew} {op}")
    assert np.array_equal(bits(out), bits(gnn.propagate_msg(g, gnn.E_MUL_XJ, to_dev(X), e_csr=e_csr, op=op))), "not bit-reproducible"
    bw = gnn.propagate_msg_backward(g, gnn.E_MUL_XJ, to_dev(R), op=op, Xj=to_dev(X), e_csrT=e_csrT, want_de=True)
    rb = oracle.propagate_msg_backward(oracle.E_MUL_XJ, op, n, src, dst, X, R, e=e, want=("dXj", "de"))
    assert_close(to_host64(bw["dXj"]), rb["dXj"], rb["SXj"], dtype, f"dXj width {ew} {op}")
    assert_close(to_host64(bw["de"]), rb["de"][ref["eid"]], rb["Se"][ref["eid"]], "f32", f"de width {ew} {op}")


def test_edge_factors_on_the_row_walking_kernel_for_narrow_rows(gnn):
    """Narrow rows reach the row-walking kernel only on graphs of 8 Mi edges and more: per-feature and per-head
    factors there, sampled against the checker on the rows of a node subset."""
    n, e = 60_000, 8_500_000
    rng = np.random.default_rng(77)
    src = rng.integers(0, n, e).astype(np.int32)
    dst = rng.integers(0, n, e).astype(np.int32)
    dst[:300_000] = 11  # a hub cut by hundreds of chunks
    g = build_graph(gnn, n, src, dst)
    eid = g.eid[:g.E].cpu().numpy()
    F, H = 32, 4
    X = feats((n, F), "bf16", 78)
    rows = np.unique(np.concatenate([[0, 11, n - 1], rng.integers(0, n, 500)]))
    keep = np.isin(dst, rows)
    oracle.set_threads(8)
    try:
        for ew in (H, F):
            ev = synth.uniform_f32((e, ew), -1.0, 1.0, 14 + ew)
            out = gnn.propagate_msg(g, gnn.E_MUL_XJ, to_dev(X), e_csr=to_dev(ev[eid]), op="sum")
            o, S, _ = oracle.propagate_msg(oracle.E_MUL_XJ, "sum", n, src[keep], dst[keep], X, e=ev[keep])
            assert_close(to_host64(out)[rows], o[rows], S[rows], "bf16", f"width {ew} on the row-walking kernel")
    finally:
        oracle.set_threads(1)


@pytest.mark.parametrize("dtype,F", [("f32", 64), ("f32", 256), ("bf16", 128), ("bf16", 512)])
def test_gin(gnn, dtype, F):
    n, src, dst = ragged_graph(80 + F)
    g = build_graph(gnn, n, src, dst)
    X = feats((n, F), dtype, 800 + F)
    R = feats((n, F), dtype, 801 + F, stream=1)
    eps = 0.25
    out = gnn.gin(g, to_dev(X), eps)
    o, S = oracle.gin(n, src, dst, X, eps)
    assert_close(to_host64(out), o, S, dtype, "gin forward")
    dX, deps = gnn.gin_backward(g, to_dev(R), eps, X=to_dev(X), want_deps=True)
    rb = oracle.gin_backward(n, src, dst, X, eps, R)
    assert_close(to_host64(dX), rb["dX"], rb["SdX"], dtype, "gin dX")
    assert abs(float(deps.cpu()[0]) - rb["deps"]) <= 1e-5 * rb["Sdeps"], "gin deps"
    dX2, deps2 = gnn.gin_backward(g, to_dev(R), eps, X=to_dev(X), want_deps=True)
    assert np.array_equal(bits(dX), bits(dX2)) and np.array_equal(bits(deps), bits(deps2)), "not bit-reproducible"


@pytest.mark.parametrize("dtype,F", [("f32", 64), ("f32", 256), ("bf16", 128), ("bf16", 1024)])
@pytest.mark.parametrize("op", ["sum", "mean", "max"])
def test_bias_relu_epilogue(gnn, dtype, F, op):
    n, src, dst = ragged_graph(90 + F)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    X = feats((n, F), dtype, 900 + F)
    R = feats((n, F), dtype, 901 + F, stream=1)
    bias = synth.uniform_f32((F,), -0.5, 0.5, 15)
    w = synth.uniform_f32((len(src),), 0.0, 1.0, 16)
    res = gnn.propagate_msg(g, gnn.E_MUL_XJ, to_dev(X), e_csr=to_dev(w[ref["eid"]]), op=op, epi=dict(bias=to_dev(bias), relu=True))
    Y = res[0] if op == "max" else res
    z, S, _ = oracle.propagate(op, n, src, dst, X, w)
    o = oracle.epilogue(z, bias, "relu")
    assert_close(to_host64(Y), o, (np.abs(z) if op == "max" else S) + np.abs(bias)[None, :], dtype, f"bias + relu after {op}")
    # backward of the epilogue: the mask is taken from the output the device produced
    dZ, dbias = gnn.row_epilogue_backward(Y, to_dev(R), relu=True)
    rz, rb, rS = oracle.epilogue_backward(to_host64(Y), R, "relu")
    assert np.array_equal(to_host64(dZ), rz), "masked gradient differs"
    assert_close(to_host64(dbias)[None, :], rb[None, :], rS[None, :], "f32", "dbias")
    dZ2, dbias2 = gnn.row_epilogue_backward(Y, to_dev(R), relu=True)
    assert np.array_equal(bits(dbias), bits(dbias2)), "dbias not bit-reproducible"
    # without relu the mask is all ones and no Y is needed
    dZ3, dbias3 = gnn.row_epilogue_backward(None, to_dev(R), relu=False)
    _, rb3, rS3 = oracle.epilogue_backward(None, R, None)
    assert np.array_equal(bits(dZ3), bits(to_dev(R)))
    assert_close(to_host64(dbias3)[None, :], rb3[None, :], rS3[None, :], "f32", "dbias without relu")


@pytest.mark.parametrize("dtype,H,C", [("f32", 1, 64), ("f32", 4, 16), ("f32", 2, 128), ("bf16", 1, 128), ("bf16", 8, 32), ("bf16", 4, 256)])
def test_xi_dot_xj(gnn, dtype, H, C):
    n, src, dst = ragged_graph(100 + H * C)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    F = H * C
    Xj = feats((n, F), dtype, 1000 + F)
    Xi = feats((n, F), dtype, 1001 + F, stream=1)
    s = gnn.edge_dot(g, to_dev(Xj), to_dev(Xi), H)
    o = oracle.apply_edges(oracle.XI_DOT_XJ, src, dst, Xj, Y=Xi, H=H)
    S = oracle.apply_edges(oracle.XI_DOT_XJ, src, dst, absval(Xj), Y=absval(Xi), H=H)
    assert_close(to_host64(s), o[ref["eid"]], S[ref["eid"]], "f32", "x_i . x_j")
    ds = synth.normal_f32((len(src), H), 17)
    dXj, dXi = gnn.edge_dot_backward(g, to_dev(Xj), to_dev(Xi), to_dev(ds[ref["eid"]]), H)
    rb = oracle.apply_edges_backward(oracle.XI_DOT_XJ, n, src, dst, Xj, ds, Y=Xi, H=H, want=("dXj", "dXi"))
    assert_close(to_host64(dXj), rb["dXj"], rb["SXj"], dtype, "x_i . x_j: dXj")
    assert_close(to_host64(dXi), rb["dXi"], rb["SXi"], dtype, "x_i . x_j: dXi")


def test_message_argument_errors(gnn):
    import torch
    n, src, dst = ragged_graph(3, n=200, e=2000, hub=100, empty_from=190)
    g = build_graph(gnn, n, src, dst)
    X = to_dev(feats((n, 64), "f32", 1))
    e = torch.zeros((g.E, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(gnn.GnnError) as err:  # wide factors with max
        gnn.propagate_msg(g, gnn.E_MUL_XJ, X, e_csr=e, op="max")
    assert err.value.status == 5
    with pytest.raises(gnn.GnnError) as err:  # x_i - x_j without x_i
        gnn.propagate_msg(g, gnn.XI_SUB_XJ, X)
    assert err.value.status == 1
    with pytest.raises(gnn.GnnError) as err:  # the self slot is taken by x_i
        gnn.propagate_msg(g, gnn.XI_SUB_XJ, X, Xi=X, epi=dict(Xself=X, self_coef=1.0))
    assert err.value.status == 5
    with pytest.raises(gnn.GnnError) as err:  # width that does not divide F
        gnn.propagate_msg(g, gnn.E_MUL_XJ, X, e_csr=torch.zeros((g.E, 5), dtype=torch.float32, device="cuda"))
    assert err.value.status == 1
    with pytest.raises(gnn.GnnError) as err:  # GAT logits are not a propagate message
        gnn.propagate_msg(g, gnn.GAT_LOGIT, X)
    assert err.value.status == 5


@pytest.mark.parametrize("dtype,H,C", [("f32", 1, 64), ("f32", 4, 16), ("f32", 8, 16), ("bf16", 8, 32), ("bf16", 2, 64), ("bf16", 1, 40)])
def test_gatv2_logits_forward_backward(gnn, dtype, H, C):
    n, src, dst = ragged_graph(140 + H * C)  # a 6000-edge hub (block tier of the backward), short rows, empty rows
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    F = H * C
    Xl = feats((n, F), dtype, 1500 + F)
    Xr = feats((n, F), dtype, 1501 + F, stream=1)
    a = synth.uniform_f32((H, C), -1.0, 1.0, 26)
    s = gnn.gatv2_logits(g, to_dev(Xl), to_dev(Xr), to_dev(a), H)
    o, S, _ = oracle.gatv2_logits(src, dst, Xl, Xr, a, H)
    assert_close(to_host64(s), o[ref["eid"]], S[ref["eid"]], "f32", "GATv2 logits")
    ds = synth.normal_f32((len(src), H), 27)
    dXl, dXr, da = gnn.gatv2_logits_backward(g, to_dev(Xl), to_dev(Xr), to_dev(a), to_dev(ds[ref["eid"]]), H)
    rb = oracle.gatv2_logits_backward(n, src, dst, Xl, Xr, a, H, ds)
    assert_close(to_host64(dXl), rb["dXl"], rb["SXl"], dtype, "GATv2 dXl")
    assert_close(to_host64(dXr), rb["dXr"], rb["SXr"], dtype, "GATv2 dXr")
    assert_close(to_host64(da), rb["da"], rb["Sda"], "f32", "GATv2 da")
    again = gnn.gatv2_logits_backward(g, to_dev(Xl), to_dev(Xr), to_dev(a), to_dev(ds[ref["eid"]]), H)
    assert all(np.array_equal(bits(x), bits(y)) for x, y in zip((dXl, dXr, da), again)), "not bit-reproducible"


@pytest.mark.parametrize("dtype,H,C", [("f32", 4, 16), ("bf16", 8, 32), ("f32", 1, 128)])
def test_gatv2_backward_hub_rows_of_both_orientations(gnn, dtype, H, C):
    """Several rows of thousands of positions and a band of rows of 257 ... 2000 positions (the block tier), in the
    target and in the source orientation, among 80000 mostly short rows."""
    rng = np.random.default_rng(77 + H)
    n, e = 80000, 300000
    src = rng.integers(0, n, e).astype(np.int32)
    dst = rng.integers(0, n, e).astype(np.int32)
    dst[:9000] = 7
    dst[9000:12001] = 7 + 37
    dst[12001:14050] = 79999            # the last row
    for k in range(30):                 # block-tier rows of 257 ... 2000 positions
        dst[20000 + 2000 * k:20000 + 2000 * k + 257 + 60 * k] = 100 + k
    src[90000:95000] = 79990
    for k in range(20):
        src[100000 + 1000 * k:100000 + 1000 * k + 300 + 30 * k] = 200 + 3 * k
    perm = rng.permutation(e)
    src, dst = src[perm].copy(), dst[perm].copy()
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    F = H * C
    Xl = feats((n, F), dtype, 1600 + F)
    Xr = feats((n, F), dtype, 1601 + F, stream=1)
    a = synth.uniform_f32((H, C), -1.0, 1.0, 28)
    ds = synth.normal_f32((e, H), 29)
    dXl, dXr, da = gnn.gatv2_logits_backward(g, to_dev(Xl), to_dev(Xr), to_dev(a), to_dev(ds[ref["eid"]]), H)
    rb = oracle.gatv2_logits_backward(n, src, dst, Xl, Xr, a, H, ds)
    assert_close(to_host64(dXl), rb["dXl"], rb["SXl"], dtype, "GATv2 dXl")
    assert_close(to_host64(dXr), rb["dXr"], rb["SXr"], dtype, "GATv2 dXr")
    assert_close(to_host64(da), rb["da"], rb["Sda"], "f32", "GATv2 da")
    again = gnn.gatv2_logits_backward(g, to_dev(Xl), to_dev(Xr), to_dev(a), to_dev(ds[ref["eid"]]), H)
    assert all(np.array_equal(bits(x), bits(y)) for x, y in zip((dXl, dXr, da), again)), "not bit-reproducible"
