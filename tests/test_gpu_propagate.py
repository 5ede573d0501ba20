"""GPU parity: graph set-up and fused propagate (forward and backward) against the CPU checker,
element by element on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_2412_06354_b200 import synth
from util import assert_close, bits, f64_to_dtype_bits, host_bits, to_dev, to_host64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gnn():
    import torch
    from paper_2412_06354_b200 import gnn as g
    g.load()
    assert torch.cuda.is_available()
    return g


def ragged_graph(seed, n=1500, e=30000, hub=6000, empty_from=1400):
    """Random multigraph with one hub row spanning many chunks, short rows, duplicate edges,
    self-loops and a block of nodes without incoming edges."""
    rng = np.random.default_rng(seed)
    src = rng.integers(0, n, e).astype(np.int32)
    dst = rng.integers(0, empty_from, e).astype(np.int32)
    dst[:hub] = 7
    perm = rng.permutation(e)
    return n, src[perm].copy(), dst[perm].copy()


def host_csr(n, src, dst):
    rowptr, col, eid = oracle.coo_to_csr(n, dst, src)
    rowptrT, colT, eidT = oracle.coo_to_csr(n, src, dst)
    return dict(rowptr=rowptr, col=col, eid=eid, rowptrT=rowptrT, colT=colT, eidT=eidT, t2f=oracle.t2f(eid, eidT))


def build_graph(gnn, n, src, dst):
    return gnn.coo_to_csr(n, to_dev(src), to_dev(dst))


def feats(shape, dtype, seed, stream=0):
    return synth.normal(shape, dtype, seed, stream)


# ---------------------------------------------------------------- set-up: bit-exact
@pytest.mark.parametrize("case", ["ragged", "tiny", "empty", "one_node", "big_ids"])
def test_coo_to_csr_bit_exact(gnn, case):
    if case == "ragged":
        n, src, dst = ragged_graph(1)
    elif case == "tiny":
        n, src, dst = 5, np.array([0, 4, 4, 2], np.int32), np.array([4, 0, 0, 2], np.int32)
    elif case == "empty":
        n, src, dst = 7, np.zeros(0, np.int32), np.zeros(0, np.int32)
    elif case == "one_node":
        n, src, dst = 1, np.zeros(300, np.int32), np.zeros(300, np.int32)
    else:  # ids above 2^16 exercise the third radix pass; more than one tile of edges
        rng = np.random.default_rng(5)
        n = 70_001
        src = rng.integers(0, n, 20_000).astype(np.int32)
        dst = rng.integers(0, n, 20_000).astype(np.int32)
        src[:4] = [70_000, 65_536, 65_535, 0]
        dst[:4] = [0, 70_000, 65_536, 65_535]
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    E = len(src)
    for k, v in ref.items():
        got = getattr(g, k).cpu().numpy()
        got = got if k.startswith("rowptr") else got[:E]
        assert np.array_equal(got, v), k
    deg_in = gnn.degree(g).cpu().numpy()
    deg_out = gnn.degree(g, transposed=True).cpu().numpy()
    assert np.array_equal(deg_in, oracle.degree(n, dst)[0])
    assert np.array_equal(deg_out, oracle.degree(n, src)[0])


def test_coo_to_csr_rejects_out_of_range(gnn):
    src = to_dev(np.array([0, 1, 5], np.int32))
    dst = to_dev(np.array([1, 0, 0], np.int32))
    with pytest.raises(gnn.GnnError) as e:
        gnn.coo_to_csr(5, src, dst)
    assert e.value.status == 2
    with pytest.raises(gnn.GnnError) as e:
        gnn.coo_to_csr(6, to_dev(np.array([0, -1], np.int32)), to_dev(np.array([0, 0], np.int32)))
    assert e.value.status == 2
    import torch
    with pytest.raises(gnn.GnnError) as e:  # workspace too small
        gnn.coo_to_csr(6, src, dst, ws=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4


def test_self_loops_gcn_norm_permute_weighted_degree(gnn):
    import torch
    n, src, dst = ragged_graph(2, n=800, e=9000, hub=900, empty_from=800)
    so, do = gnn.add_self_loops(n, to_dev(src), to_dev(dst))
    hs, hd = synth.with_self_loops(n, src, dst)
    assert np.array_equal(so.cpu().numpy(), hs) and np.array_equal(do.cpu().numpy(), hd)
    g = gnn.coo_to_csr(n, so, do)
    ref = host_csr(n, hs, hd)
    # unweighted
    deg, coef, coefT = gnn.gcn_norm(g)
    c = oracle.gcn_norm(n, hs, hd)
    assert_close(to_host64(coef), c[ref["eid"]], np.abs(c[ref["eid"]]), "f32", "gcn coef (CSR order)")
    assert_close(to_host64(coefT), c[ref["eidT"]], np.abs(c[ref["eidT"]]), "f32", "gcn coef (CSR^T order)")
    assert np.array_equal(to_host64(deg), oracle.degree(n, hd)[1])
    # weighted, weights given in COO order and permuted on the device
    w = synth.uniform_f32((len(hs),), 0.1, 2.0, 9)
    w_csr = gnn.permute_edge_data(g.eid[:g.E], to_dev(w))
    assert np.array_equal(w_csr.cpu().numpy(), w[ref["eid"]])
    deg, coef, coefT = gnn.gcn_norm(g, w_csr)
    cw = oracle.gcn_norm(n, hs, hd, w)
    dw = oracle.degree(n, hd, w)[1]
    assert_close(to_host64(deg), dw, dw, "f32", "weighted degree")
    assert_close(to_host64(coef), cw[ref["eid"]], np.abs(cw[ref["eid"]]), "f32", "weighted gcn coef")
    assert_close(to_host64(gnn.degree(g, w=w_csr)), dw, dw, "f32", "gnn_degree weighted")
    # 2-wide and bf16 edge data
    e2 = synth.normal_bf16((len(hs), 2), 3)
    got = gnn.permute_edge_data(g.t2f[:g.E], gnn.permute_edge_data(g.eid[:g.E], to_dev(e2)))
    assert np.array_equal(bits(got), host_bits(e2[ref["eidT"]]))


# ---------------------------------------------------------------- forward
SHAPES = [("f32", 4), ("f32", 32), ("f32", 64), ("f32", 100), ("f32", 128), ("f32", 256), ("f32", 512),
          ("bf16", 8), ("bf16", 32), ("bf16", 64), ("bf16", 128), ("bf16", 200), ("bf16", 256), ("bf16", 512), ("bf16", 1024)]


@pytest.mark.parametrize("dtype,F", SHAPES)
@pytest.mark.parametrize("weighted", [False, True])
def test_propagate_sum_mean(gnn, dtype, F, weighted):
    n, src, dst = ragged_graph(10 + F)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    X = feats((n, F), dtype, 100 + F)
    w = synth.uniform_f32((len(src),), 0.0, 1.0, 7) if weighted else None
    w_csr = to_dev(w[ref["eid"]]) if weighted else None
    Xd = to_dev(X)
    for op in ("sum", "mean"):
        out = gnn.propagate_fused(g, Xd, w_csr, op)
        o, S, _ = oracle.propagate(op, n, src, dst, X, w)
        assert_close(to_host64(out), o, S, dtype, f"propagate {op} F={F} {dtype} weighted={weighted}")
        again = gnn.propagate_fused(g, Xd, w_csr, op)
        assert np.array_equal(bits(out), bits(again)), "not bit-reproducible"


@pytest.mark.parametrize("dtype,F", [("f32", 4), ("f32", 64), ("f32", 128), ("f32", 512), ("bf16", 32), ("bf16", 128), ("bf16", 256), ("bf16", 1024)])
@pytest.mark.parametrize("op", ["max", "min"])
def test_propagate_max_min_bit_exact(gnn, dtype, F, op):
    n, src, dst = ragged_graph(20 + F)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    X = feats((n, F), dtype, 200 + F)  # bf16 N(0,1) on the hub row ties often: tie-break is exercised
    out, arg = gnn.propagate_fused(g, to_dev(X), None, op)
    o, _, a = oracle.propagate(op, n, src, dst, X)
    assert np.array_equal(bits(out), f64_to_dtype_bits(o, dtype)), "values differ"
    got_arg = arg.cpu().numpy()
    eid_of = np.where(got_arg >= 0, ref["eid"][np.maximum(got_arg, 0)], -1)
    assert np.array_equal(eid_of, a), "winner differs"


@pytest.mark.parametrize("dtype,F", [("f32", 64), ("f32", 512), ("bf16", 32), ("bf16", 128), ("bf16", 1024)])
@pytest.mark.parametrize("op", ["max", "min"])
def test_propagate_weighted_max_min(gnn, dtype, F, op):
    """e_mul_xj with max/min: the message w*x is rounded once to fp32 and compared in fp32 (the checker does
    the same), so values and winners are bit-exact; signed weights, both kernels (rows up to 512 bytes take the
    position-first kernel here, wider rows the row-walking one); then the routing backward with the weights."""
    n, src, dst = ragged_graph(50 + F)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    X = feats((n, F), dtype, 500 + F)
    R = feats((n, F), dtype, 501 + F, stream=1)
    w = synth.uniform_f32((len(src),), -1.0, 1.0, 12)
    out, arg = gnn.propagate_fused(g, to_dev(X), to_dev(w[ref["eid"]]), op)
    o, _, a = oracle.propagate(op, n, src, dst, X, w)
    assert np.array_equal(bits(out), f64_to_dtype_bits(o, dtype)), "values differ"
    got_arg = arg.cpu().numpy()
    assert np.array_equal(np.where(got_arg >= 0, ref["eid"][np.maximum(got_arg, 0)], -1), a), "winner differs"
    dX, _ = gnn.propagate_fused_backward(g, to_dev(R), op, w_csrT=to_dev(w[ref["eidT"]]), argmax=arg)
    bw = oracle.propagate_backward(op, n, src, dst, X, w, R, arg=a)
    assert_close(to_host64(dX), bw["dX"], bw["SdX"], dtype, f"weighted dX {op}")


# ---------------------------------------------------------------- backward
@pytest.mark.parametrize("dtype,F", [("f32", 16), ("f32", 64), ("f32", 128), ("f32", 512), ("bf16", 32), ("bf16", 64), ("bf16", 128), ("bf16", 512)])
@pytest.mark.parametrize("op", ["sum", "mean"])
def test_propagate_backward_sum_mean(gnn, dtype, F, op):
    n, src, dst = ragged_graph(30 + F)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    X = feats((n, F), dtype, 300 + F)
    R = feats((n, F), dtype, 301 + F, stream=1)
    w = synth.uniform_f32((len(src),), 0.0, 1.0, 8)
    w_csrT = to_dev(w[ref["eidT"]])
    dX, dW = gnn.propagate_fused_backward(g, to_dev(R), op, X=to_dev(X), w_csrT=w_csrT, want_dW=True)
    bw = oracle.propagate_backward(op, n, src, dst, X, w, R, want_dw=True)
    assert_close(to_host64(dX), bw["dX"], bw["SdX"], dtype, f"dX {op}")
    assert_close(to_host64(dW), bw["dw"][ref["eid"]], bw["Sdw"][ref["eid"]], "f32", f"dW {op}")
    # unweighted (copy_xj)
    dX, _ = gnn.propagate_fused_backward(g, to_dev(R), op)
    bw = oracle.propagate_backward(op, n, src, dst, X, None, R)
    assert_close(to_host64(dX), bw["dX"], bw["SdX"], dtype, f"dX {op} copy")


@pytest.mark.parametrize("dtype,F", [("f32", 64), ("f32", 128), ("bf16", 32), ("bf16", 128), ("bf16", 512)])
@pytest.mark.parametrize("op", ["max", "min"])
def test_propagate_backward_max_min(gnn, dtype, F, op):
    n, src, dst = ragged_graph(40 + F)
    g = build_graph(gnn, n, src, dst)
    X = feats((n, F), dtype, 400 + F)
    R = feats((n, F), dtype, 401 + F, stream=1)
    out, arg = gnn.propagate_fused(g, to_dev(X), None, op)
    dX, _ = gnn.propagate_fused_backward(g, to_dev(R), op, argmax=arg)
    _, _, a = oracle.propagate(op, n, src, dst, X)
    bw = oracle.propagate_backward(op, n, src, dst, X, None, R, arg=a)
    assert_close(to_host64(dX), bw["dX"], bw["SdX"], dtype, f"dX {op}")


# ---------------------------------------------------------------- degenerate shapes
def test_edge_cases(gnn):
    import torch
    F = 64
    # no edges at all: zeros, argmax -1
    g = build_graph(gnn, 9, np.zeros(0, np.int32), np.zeros(0, np.int32))
    X = to_dev(feats((9, F), "f32", 1))
    assert torch.count_nonzero(gnn.propagate_fused(g, X, None, "sum")) == 0
    out, arg = gnn.propagate_fused(g, X, None, "max")
    assert torch.count_nonzero(out) == 0 and bool((arg == -1).all())
    dX, _ = gnn.propagate_fused_backward(g, X, "mean")
    assert torch.count_nonzero(dX) == 0
    # rows that end exactly on chunk boundaries (256 edges each) and trailing empty rows
    n = 12
    dst = np.repeat(np.arange(8, dtype=np.int32), 256)
    src = (np.arange(len(dst)) % n).astype(np.int32)
    g = build_graph(gnn, n, src, dst)
    Xh = feats((n, F), "f32", 2)
    o, S, _ = oracle.propagate("sum", n, src, dst, Xh)
    assert_close(to_host64(gnn.propagate_fused(g, to_dev(Xh), None, "sum")), o, S, "f32", "aligned rows")
    # one row holding every edge, more than one block of chunks
    e = 5000
    src = (np.arange(e) * 7 % n).astype(np.int32)
    dst = np.full(e, 3, np.int32)
    g = build_graph(gnn, n, src, dst)
    for op in ("sum", "mean", "max"):
        o, S, a = oracle.propagate(op, n, src, dst, Xh)
        got = gnn.propagate_fused(g, to_dev(Xh), None, op)
        got = got[0] if op == "max" else got
        assert_close(to_host64(got), o, S, "f32", f"single hub {op}")
    # single node with a self-loop
    g = build_graph(gnn, 1, np.zeros(1, np.int32), np.zeros(1, np.int32))
    X1 = to_dev(feats((1, F), "f32", 3))
    assert torch.equal(gnn.propagate_fused(g, X1, None, "mean"), X1)


def test_unsupported_and_bad_arguments(gnn):
    import torch
    n, src, dst = ragged_graph(3, n=50, e=200, hub=20, empty_from=50)
    g = build_graph(gnn, n, src, dst)
    with pytest.raises(gnn.GnnError) as e:  # 3 floats = 12 bytes per row
        gnn.propagate_fused(g, torch.zeros((n, 3), device="cuda"))
    assert e.value.status == 5
    with pytest.raises(gnn.GnnError) as e:  # 1024 floats = 4096 bytes per row
        gnn.propagate_fused(g, torch.zeros((n, 1024), device="cuda"))
    assert e.value.status == 5
    with pytest.raises(gnn.GnnError) as e:
        gnn.propagate_fused(g, torch.zeros((n, 64), device="cuda"), ws=torch.empty(32, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4
    with pytest.raises(gnn.GnnError) as e:  # max backward without argmax
        gnn.propagate_fused_backward(g, torch.zeros((n, 64), device="cuda"), "max")
    assert e.value.status == 1


# ---------------------------------------------------------------- workload-shaped cases
def test_gcn_small_workload(gnn):
    """N=2000, 10000 edges + self-loops, F=64 f32: normalised propagate, forward and backward."""
    wl = synth.workload_gcn_small()
    n, F = wl["N"], wl["F"]
    so, do = gnn.add_self_loops(n, to_dev(wl["src"]), to_dev(wl["dst"]))
    g = gnn.coo_to_csr(n, so, do)
    _, coef, coefT = gnn.gcn_norm(g)
    hs, hd = synth.with_self_loops(n, wl["src"], wl["dst"])
    c32 = np.empty(len(hs), np.float32)
    c32[g.eid[:g.E].cpu().numpy()] = coef.cpu().numpy()  # the device's own coefficients, COO order
    out = gnn.propagate_fused(g, to_dev(wl["X"]), coef, "sum")
    o, S, _ = oracle.propagate("sum", n, hs, hd, wl["X"], c32)
    assert_close(to_host64(out), o, S, "f32", "gcn propagate")
    # end to end against fp64 coefficients: coefficient rounding (1e-7) stays inside 1e-5*S
    o64 = oracle.aggregate("sum", n, hd, oracle.gcn_norm(n, hs, hd)[:, None] * oracle.gather(hs, wl["X"]))
    assert_close(to_host64(out), o64[0], o64[1], "f32", "gcn propagate vs fp64 coefficients")
    R = feats((n, F), "f32", 77)
    dX, _ = gnn.propagate_fused_backward(g, to_dev(R), "sum", w_csrT=coefT)
    bw = oracle.propagate_backward("sum", n, hs, hd, wl["X"], c32, R)
    assert_close(to_host64(dX), bw["dX"], bw["SdX"], "f32", "gcn dX")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_powerlaw_workload_full_size(gnn, dtype):
    """Preferential-attachment graph, N=170000, 1359980 edges, F=128: mean, max (+argmax), GCN-weighted sum."""
    wl = synth.workload_powerlaw(dtype=dtype)
    n, F, src, dst, X = wl["N"], wl["F"], wl["src"], wl["dst"], wl["X"]
    g = build_graph(gnn, n, src, dst)
    eid = g.eid[:g.E].cpu().numpy()
    eidT = g.eidT[:g.E].cpu().numpy()
    Xd = to_dev(X)
    oracle.set_threads(8)
    try:
        out = gnn.propagate_fused(g, Xd, None, "mean")
        o, S, _ = oracle.propagate("mean", n, src, dst, X)
        assert_close(to_host64(out), o, S, dtype, "mean")
        out, arg = gnn.propagate_fused(g, Xd, None, "max")
        o, _, a = oracle.propagate("max", n, src, dst, X)
        assert np.array_equal(bits(out), f64_to_dtype_bits(o, dtype))
        ga = arg.cpu().numpy()
        assert np.array_equal(np.where(ga >= 0, eid[np.maximum(ga, 0)], -1), a)
        R = feats((n, F), dtype, 78)
        dX, _ = gnn.propagate_fused_backward(g, to_dev(R), "max", argmax=arg)
        bw = oracle.propagate_backward("max", n, src, dst, X, None, R, arg=a)
        assert_close(to_host64(dX), bw["dX"], bw["SdX"], dtype, "max backward")
        w = synth.uniform_f32((len(src),), 0.0, 1.0, 9)
        out = gnn.propagate_fused(g, Xd, to_dev(w[eid]), "sum")
        o, S, _ = oracle.propagate("sum", n, src, dst, X, w)
        assert_close(to_host64(out), o, S, dtype, "weighted sum")
        dX, dW = gnn.propagate_fused_backward(g, to_dev(R), "sum", X=Xd, w_csrT=to_dev(w[eidT]), want_dW=True)
        bw = oracle.propagate_backward("sum", n, src, dst, X, w, R, want_dw=True)
        assert_close(to_host64(dX), bw["dX"], bw["SdX"], dtype, "weighted dX")
        assert_close(to_host64(dW), bw["dw"][eid], bw["Sdw"][eid], "f32", "dW")
    finally:
        oracle.set_threads(1)


@pytest.mark.parametrize("e,dtype,F", [(200_000, "f32", 32), (200_000, "bf16", 8), (600_000, "bf16", 64), (600_000, "f32", 12),
                                       (70_000, "bf16", 128), (130_000, "f32", 128)])
def test_chunk_regimes_with_empty_rows_everywhere(gnn, e, dtype, F):
    """Edge counts on both sides of the chunk-size thresholds (64 / 128 / 256 positions per warp), rows
    without edges at the front, in the middle and at the end, a hub cut by many chunks, every lane layout."""
    n = 5000
    rng = np.random.default_rng(e + F)
    # targets only in [300, 4000) and never a multiple of 7: empty rows lead, trail and are interspersed
    dst = rng.integers(300, 4000, e).astype(np.int32)
    dst[dst % 7 == 0] += 1
    dst[: e // 20] = 1234  # hub
    src = rng.integers(0, n, e).astype(np.int32)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    eid, eidT = ref["eid"], ref["eidT"]
    X = feats((n, F), dtype, 300 + F)
    w = synth.uniform_f32((e,), 0.0, 1.0, 11)
    Xd = to_dev(X)
    for op, weighted in (("sum", True), ("mean", False)):
        out = gnn.propagate_fused(g, Xd, to_dev(w[eid]) if weighted else None, op)
        o, S, _ = oracle.propagate(op, n, src, dst, X, w if weighted else None)
        assert_close(to_host64(out), o, S, dtype, f"{op} E={e}")
        R = feats((n, F), dtype, 301 + F)
        dX, _ = gnn.propagate_fused_backward(g, to_dev(R), op, w_csrT=to_dev(w[eidT]) if weighted else None)
        bw = oracle.propagate_backward(op, n, src, dst, X, w if weighted else None, R)
        assert_close(to_host64(dX), bw["dX"], bw["SdX"], dtype, f"{op} backward E={e}")
    for op in ("max", "min"):
        out, arg = gnn.propagate_fused(g, Xd, None, op)
        o, _, a = oracle.propagate(op, n, src, dst, X)
        assert np.array_equal(bits(out), f64_to_dtype_bits(o, dtype))
        ga = arg.cpu().numpy()
        assert np.array_equal(np.where(ga >= 0, eid[np.maximum(ga, 0)], -1), a)
        R = feats((n, F), dtype, 302 + F)
        dX, _ = gnn.propagate_fused_backward(g, to_dev(R), op, argmax=arg)
        bw = oracle.propagate_backward(op, n, src, dst, X, None, R, arg=a)
        assert_close(to_host64(dX), bw["dX"], bw["SdX"], dtype, f"{op} backward E={e}")


@pytest.mark.parametrize("dtype,F", [("bf16", 64), ("f32", 16), ("bf16", 512)])
def test_long_runs_of_rows_without_edges(gnn, dtype, F):
    """A bipartite-like graph: 200000 nodes of which only 2000 in the middle receive edges, with one more
    run of 40000 empty rows between two of them.  Both the short-row kernel (F*s <= 512 bytes) and the
    row-walking kernel (wider rows) must jump over the runs and still zero every empty row."""
    n, e = 200_000, 50_000
    rng = np.random.default_rng(F)
    dst = rng.integers(90_000, 92_000, e).astype(np.int32)
    dst[dst >= 91_000] += 40_000
    src = rng.integers(0, n, e).astype(np.int32)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    X = feats((n, F), dtype, 400 + F)
    Xd = to_dev(X)
    for op in ("sum", "mean"):
        out = gnn.propagate_fused(g, Xd, None, op)
        o, S, _ = oracle.propagate(op, n, src, dst, X)
        assert_close(to_host64(out), o, S, dtype, f"{op} with long empty runs")
    out, arg = gnn.propagate_fused(g, Xd, None, "max")
    o, _, a = oracle.propagate("max", n, src, dst, X)
    assert np.array_equal(bits(out), f64_to_dtype_bits(o, dtype))
    ga = arg.cpu().numpy()
    assert np.array_equal(np.where(ga >= 0, ref["eid"][np.maximum(ga, 0)], -1), a)
    # the transposed form has the runs elsewhere (sources are spread over all nodes)
    R = feats((n, F), dtype, 401 + F)
    dX, _ = gnn.propagate_fused_backward(g, to_dev(R), "sum")
    bw = oracle.propagate_backward("sum", n, src, dst, X, None, R)
    assert_close(to_host64(dX), bw["dX"], bw["SdX"], dtype, "backward with long empty runs")
    # edge-weight gradient: one dot product per edge, rows found across the runs
    _, dW = gnn.propagate_fused_backward(g, to_dev(R), "sum", X=Xd, want_dX=False, want_dW=True)
    bw = oracle.propagate_backward("sum", n, src, dst, X, np.ones(e, np.float32), R, want_dX=False, want_dw=True)
    assert_close(to_host64(dW), bw["dw"][ref["eid"]], bw["Sdw"][ref["eid"]], "f32", "dW with long empty runs")


@pytest.mark.parametrize("dtype,F", [("bf16", 32), ("f32", 64), ("f32", 128), ("bf16", 128)])
def test_low_mean_degree_above_8mi_edges_takes_positions_first(gnn, dtype, F):
    """Graphs of 8 Mi edges and more whose mean degree is a handful run sums on one-slab chunks (positions first)
    instead of the row walk: forward sum, mean and the backward of the mean, on sampled rows, with a hub cut by
    hundreds of chunks, rows without edges and a ragged last chunk."""
    import torch
    n, e = 2_300_000, 8_600_037
    rng = np.random.default_rng(91)
    src = rng.integers(0, n, e).astype(np.int32)
    dst = rng.integers(0, n - 50_000, e).astype(np.int32)  # the last rows receive nothing
    dst[:70_000] = 13
    g = build_graph(gnn, n, src, dst)
    X = feats((n, F), dtype, 92 + F)
    R = feats((n, F), dtype, 93 + F, stream=1)
    w = synth.uniform_f32((e,), 0.0, 1.0, 94)
    eid = g.eid[:g.E].cpu().numpy()
    rows = np.unique(np.concatenate([[0, 13, n - 50_001, n - 1], rng.integers(0, n, 3000)]))
    dev_rows = torch.from_numpy(rows).cuda()
    oracle.set_threads(8)
    try:
        out = gnn.propagate_fused(g, to_dev(X), to_dev(w[eid]), "sum")
        o, S, _ = oracle.propagate("sum", n, src, dst, X, w, rows=rows)
        assert_close(to_host64(out[dev_rows]), o, S, dtype, "weighted sum")
        assert np.array_equal(bits(out), bits(gnn.propagate_fused(g, to_dev(X), to_dev(w[eid]), "sum"))), "not bit-reproducible"
        assert torch.count_nonzero(out[n - 50_000:]) == 0
        out = gnn.propagate_fused(g, to_dev(X), None, "mean")
        o, S, _ = oracle.propagate("mean", n, src, dst, X, None, rows=rows)
        assert_close(to_host64(out[dev_rows]), o, S, dtype, "mean")
        # backward of the mean: rows of the transposed form, each gathered row divided by its target's degree
        dX, _ = gnn.propagate_fused_backward(g, to_dev(R), "mean")
        srows = np.unique(np.concatenate([[0, n - 1], rng.integers(0, n, 3000)]))
        bw = oracle.propagate_backward("mean", n, src, dst, None, None, R, rows=srows)
        assert_close(to_host64(dX[torch.from_numpy(srows).cuda()]), bw["dX"], bw["SdX"], dtype, "backward of the mean")
    finally:
        oracle.set_threads(1)
