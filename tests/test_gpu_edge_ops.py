"""GPU parity: the unfused primitives (gather, apply_edges, aggregate), edge softmax and batched
pooling against the CPU checker, through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_2412_06354_b200 import synth
from util import assert_close, bits, f64_to_dtype_bits, host_bits, to_dev, to_host64
from test_gpu_propagate import build_graph, feats, host_csr, ragged_graph

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gnn():
    from paper_2412_06354_b200 import gnn as g
    g.load()
    return g


@pytest.mark.parametrize("dtype,F", [("f32", 4), ("f32", 100), ("bf16", 8), ("bf16", 128)])
def test_gather_and_its_backward(gnn, dtype, F):
    n, src, dst = ragged_graph(50 + F)
    g = build_graph(gnn, n, src, dst)
    X = feats((n, F), dtype, 500 + F)
    for idx in (src, dst):
        out = gnn.gather(to_dev(idx), to_dev(X))
        assert np.array_equal(bits(out), host_bits(X[idx])), "gather is a bit-exact copy"
    R = feats((len(src), F), dtype, 501 + F)  # one row per edge, original edge order
    for by_src, idx in ((False, dst), (True, src)):
        dX = gnn.gather_backward(g, to_dev(R), by_src=by_src)
        ref, S = oracle.gather_backward(n, idx, R)
        assert_close(to_host64(dX), ref, S, dtype, f"gather_backward by_src={by_src}")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_apply_edges_messages(gnn, dtype):
    H, C = 4, 16
    F = H * C
    n, src, dst = ragged_graph(60)
    g = build_graph(gnn, n, src, dst)
    ref = host_csr(n, src, dst)
    eid = ref["eid"]
    X = feats((n, F), dtype, 600)
    Xd = to_dev(X)
    m = gnn.apply_edges(g, gnn.COPY_XJ, Xd)
    assert np.array_equal(bits(m), host_bits(X[src[eid]]))
    for ew in (1, H, F):
        e = synth.uniform_f32((len(src), ew), -1.0, 1.0, 601 + ew)
        m = gnn.apply_edges(g, gnn.E_MUL_XJ, Xd, e=to_dev(e[eid]))
        mo = oracle.apply_edges(oracle.E_MUL_XJ, src, dst, X, e=e)[eid]
        assert_close(to_host64(m), mo, np.abs(mo), dtype, f"e_mul_xj width {ew}")
    if dtype == "f32":
        al = synth.normal_f32((n, H), 610)
        ar = synth.normal_f32((n, H), 611)
        s = gnn.apply_edges(g, gnn.GAT_LOGIT, to_dev(al), ar=to_dev(ar), slope=0.2)
        so = oracle.apply_edges(oracle.GAT_LOGIT, src, dst, al, Y=ar, slope=0.2)[eid]
        # a two-term sum: the scale is |al| + |ar| (times the slope on the negative side)
        scale = np.abs(al[src[eid]].astype(np.float64)) + np.abs(ar[dst[eid]].astype(np.float64))
        assert_close(to_host64(s), so, scale, "f32", "gat logit")


@pytest.mark.parametrize("dtype,F", [("f32", 64), ("bf16", 128), ("bf16", 40)])
def test_aggregate_matches_checker_and_fused_path(gnn, dtype, F):
    n, src, dst = ragged_graph(70 + F)
    g = build_graph(gnn, n, src, dst)
    eid = host_csr(n, src, dst)["eid"]
    X = feats((n, F), dtype, 700 + F)
    w = synth.uniform_f32((len(src),), 0.0, 1.0, 701)
    m = gnn.apply_edges(g, gnn.E_MUL_XJ, to_dev(X), e=to_dev(w[eid]))  # CSR order, stored dtype
    m_host = np.empty((len(src), F), np.float64)
    m_host[eid] = to_host64(m)  # the device's own messages, back in original edge order
    for op in ("sum", "mean", "max", "min"):
        got = gnn.aggregate(g, m, op)
        o, S, a = oracle.aggregate(op, n, dst, m_host)
        if op in ("max", "min"):
            out, arg = got
            assert np.array_equal(bits(out), f64_to_dtype_bits(o, dtype))
            ga = arg.cpu().numpy()
            assert np.array_equal(np.where(ga >= 0, eid[np.maximum(ga, 0)], -1), a)
            R = feats((n, F), dtype, 702)
            dm = gnn.aggregate_backward(g, to_dev(R), op, argmax=arg)
            dmo = oracle.aggregate_backward(op, n, dst, R, a)[eid]
            assert np.array_equal(bits(dm), f64_to_dtype_bits(dmo, dtype))
        else:
            assert_close(to_host64(got), o, S, dtype, f"aggregate {op}")
            R = feats((n, F), dtype, 703)
            dm = gnn.aggregate_backward(g, to_dev(R), op)
            dmo = oracle.aggregate_backward(op, n, dst, R)[eid]
            assert_close(to_host64(dm), dmo, np.abs(dmo), dtype, f"aggregate_backward {op}")
    # propagate == aggregate(apply_edges): fused and unfused agree (the unfused path rounds each
    # message to the storage dtype first, so agreement is within tolerance, not bitwise)
    fused = gnn.propagate_fused(g, to_dev(X), to_dev(w[eid]), "sum")
    o, S, _ = oracle.propagate("sum", n, src, dst, X, w)
    if dtype == "f32":  # bf16 messages carry a 2^-9 rounding each, which the fused path does not have
        assert_close(to_host64(gnn.aggregate(g, m, "sum")), o, S, dtype, "unfused vs checker")
    assert_close(to_host64(fused), o, S, dtype, "fused vs checker")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("H", [1, 3, 4, 8, 16, 32])
def test_edge_softmax_forward_backward(gnn, dtype, H):
    n, src, dst = ragged_graph(80 + H)  # hub row of 6000 edges takes the block-per-row path
    g = build_graph(gnn, n, src, dst)
    eid = host_csr(n, src, dst)["eid"]
    E = len(src)
    s = feats((E, H), dtype, 800 + H)
    if dtype == "f32":
        s = (s * 3).astype(np.float32)
    alpha, rmax, rsum = gnn.edge_softmax(g, to_dev(s[eid]), want_stats=True)
    ao = oracle.edge_softmax(n, dst, s)
    assert_close(to_host64(alpha), ao[eid], ao[eid], dtype, "alpha")
    tot = np.zeros((n, H))
    np.add.at(tot, dst, to_host64(alpha)[np.argsort(eid)])
    deg = np.bincount(dst, minlength=n)
    assert np.allclose(tot[deg > 0], 1.0, atol=2e-2 if dtype == "bf16" else 1e-5)
    smax = np.full((n, H), -np.inf)
    np.maximum.at(smax, dst, synth.to_f64(s))
    assert np.array_equal(to_host64(rmax)[deg > 0], smax[deg > 0])
    assert np.all(to_host64(rmax)[deg == 0] == 0) and np.all(to_host64(rsum)[deg == 0] == 0)
    # backward, from the device's own (rounded) alpha
    a_host = np.empty((E, H), np.float64)
    a_host[eid] = to_host64(alpha)
    R = feats((E, H), dtype, 801 + H)
    ds = gnn.edge_softmax_backward(g, alpha, to_dev(R[eid]))
    dso, S = oracle.edge_softmax_backward(n, dst, a_host, R)
    assert_close(to_host64(ds), dso[eid], S[eid], dtype, "dlogits")
    again = gnn.edge_softmax(g, to_dev(s[eid]))
    assert np.array_equal(bits(again), bits(alpha))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("H", [1, 4, 8, 32])
def test_edge_softmax_rows_of_tens_of_thousands_of_positions(gnn, dtype, H):
    """Three rows above 8192 positions (shared by a cluster of blocks when H is 4, 8, 16 or 32), two of them in one
    scan window, one a single position above the threshold; a band of rows of 513 ... 3000 positions (a block each)."""
    rng = np.random.default_rng(31 + H)
    n, e = 3000, 120000
    src = rng.integers(0, n, e).astype(np.int32)
    dst = rng.integers(0, n, e).astype(np.int32)
    dst[:20000] = 7
    dst[20000:29000] = 9
    dst[29000:37193] = 2990
    at = 40000
    for k in range(12):
        dst[at:at + 513 + 220 * k] = 300 + 5 * k
        at += 513 + 220 * k
    perm = rng.permutation(e)
    src, dst = src[perm].copy(), dst[perm].copy()
    g = build_graph(gnn, n, src, dst)
    eid = host_csr(n, src, dst)["eid"]
    s = feats((e, H), dtype, 900 + H)
    if dtype == "f32":
        s = (s * 3).astype(np.float32)
    alpha, rmax, rsum = gnn.edge_softmax(g, to_dev(s[eid]), want_stats=True)
    ao = oracle.edge_softmax(n, dst, s)
    assert_close(to_host64(alpha), ao[eid], ao[eid], dtype, "alpha")
    deg = np.bincount(dst, minlength=n)
    smax = np.full((n, H), -np.inf)
    np.maximum.at(smax, dst, synth.to_f64(s))
    assert np.array_equal(to_host64(rmax)[deg > 0], smax[deg > 0])
    ssum = np.zeros((n, H))
    np.add.at(ssum, dst, np.exp(synth.to_f64(s) - smax[dst]))
    assert np.allclose(to_host64(rsum)[deg > 0], ssum[deg > 0], rtol=1e-4)
    a_host = np.empty((e, H), np.float64)
    a_host[eid] = to_host64(alpha)
    R = feats((e, H), dtype, 901 + H)
    ds = gnn.edge_softmax_backward(g, alpha, to_dev(R[eid]))
    dso, S = oracle.edge_softmax_backward(n, dst, a_host, R)
    assert_close(to_host64(ds), dso[eid], S[eid], dtype, "dlogits")
    again = gnn.edge_softmax(g, to_dev(s[eid]))
    assert np.array_equal(bits(again), bits(alpha))
    assert np.array_equal(bits(gnn.edge_softmax_backward(g, alpha, to_dev(R[eid]))), bits(ds))


def test_edge_softmax_degenerate(gnn):
    import torch
    # one edge -> 1; equal logits -> 1/deg; huge logits do not overflow
    src = np.array([0, 1, 2, 3, 1], np.int32)
    dst = np.array([4, 4, 4, 0, 0], np.int32)
    g = build_graph(gnn, 5, src, dst)
    eid = g.eid[:5].cpu().numpy()
    s = np.array([[1000.0], [1000.0], [1000.0], [-50.0], [30.0]], np.float32)
    a = to_host64(gnn.edge_softmax(g, to_dev(s[eid])))
    back = np.empty_like(a)
    back[eid] = a
    assert np.allclose(back[:3, 0], 1 / 3, rtol=1e-6) and abs(back[3, 0] - np.exp(-80.0)) < 1e-40 and abs(back[4, 0] - 1) < 1e-6
    g0 = build_graph(gnn, 3, np.zeros(0, np.int32), np.zeros(0, np.int32))
    gnn.edge_softmax(g0, torch.empty((0, 4), device="cuda"))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_batched_pooling(gnn, dtype):
    """512 graphs of 10-40 nodes, F=128: mean-aggregation layer on the batch, then pooling."""
    wl = synth.workload_batched()
    n, G, F, gp = wl["N"], wl["G"], wl["F"], wl["graph_ptr"]
    X = wl["X"] if dtype == "f32" else synth.normal_bf16((n, F), synth.BASE_SEED + 2, 10)
    gid = np.repeat(np.arange(G), np.diff(gp)).astype(np.int32)
    gptr = gnn.graph_ptr_from_ids(to_dev(gid), G)
    assert np.array_equal(gptr.cpu().numpy(), gp.astype(np.int64))
    g = build_graph(gnn, n, wl["src"], wl["dst"])
    h = gnn.propagate_fused(g, to_dev(X), None, "mean")
    ho, S, _ = oracle.propagate("mean", n, wl["src"], wl["dst"], X)
    assert_close(to_host64(h), ho, S, dtype, "mean layer on the batch")
    R = feats((G, F), dtype, 900)
    for op in ("sum", "mean", "max", "min"):
        got = gnn.reduce_nodes(gptr, to_dev(X), op)
        o, S, a = oracle.reduce_nodes(op, gp, X)
        if op in ("max", "min"):
            out, arg = got
            assert np.array_equal(bits(out), f64_to_dtype_bits(o, dtype))
            assert np.array_equal(arg.cpu().numpy(), a)
            dX = gnn.reduce_nodes_backward(gptr, to_dev(R), n, op, argmax=arg)
            assert np.array_equal(bits(dX), f64_to_dtype_bits(oracle.reduce_nodes_backward(op, gp, R, a), dtype))
        else:
            assert_close(to_host64(got), o, S, dtype, f"reduce_nodes {op}")
            dX = gnn.reduce_nodes_backward(gptr, to_dev(R), n, op)
            ref = oracle.reduce_nodes_backward(op, gp, R)
            assert_close(to_host64(dX), ref, np.abs(ref), dtype, f"reduce_nodes_backward {op}")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_pooling_over_graphs_of_a_million_nodes(gnn, dtype):
    """Two graphs of 700000 and 499980 nodes around one of 20: a graph spans thousands of chunks of the reduction,
    so its partial results are combined by the block-per-row pass, for max / min with the winning positions."""
    import torch
    sizes = [700_000, 20, 499_980]
    gp = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    n, F = int(gp[-1]), 32
    X = feats((n, F), dtype, 1234)
    p0 = int(oracle.reduce_nodes("max", gp, X)[2][0, 0])  # the winner of column 0 in the first graph ...
    X[(p0 + 350_000) % 700_000] = X[p0]                   # ... now has a twin far away: the smaller position wins
    gptr = to_dev(gp)
    R = feats((3, F), dtype, 1235)
    for op in ("mean", "max", "min"):
        got = gnn.reduce_nodes(gptr, to_dev(X), op)
        o, S, a = oracle.reduce_nodes(op, gp, X)
        if op in ("max", "min"):
            out, arg = got
            assert np.array_equal(bits(out), f64_to_dtype_bits(o, dtype))
            assert np.array_equal(arg.cpu().numpy(), a)
            again = gnn.reduce_nodes(gptr, to_dev(X), op)
            assert torch.equal(again[1], arg)
        else:
            assert_close(to_host64(got), o, S, dtype, f"reduce_nodes {op}")


def test_pooling_edge_cases(gnn):
    import torch
    # an empty graph in the middle of the batch, and unsorted ids
    gid = to_dev(np.array([0, 0, 2, 2, 2], np.int32))
    gptr = gnn.graph_ptr_from_ids(gid, 4)
    assert gptr.cpu().tolist() == [0, 2, 2, 5, 5]
    X = to_dev(feats((5, 8), "f32", 1))
    out, arg = gnn.reduce_nodes(gptr, X, "max")
    assert torch.count_nonzero(out[1]) == 0 and bool((arg[1] == -1).all()) and bool((arg[3] == -1).all())
    assert torch.equal(out[0], torch.maximum(X[0], X[1]))
    with pytest.raises(gnn.GnnError) as e:
        gnn.graph_ptr_from_ids(to_dev(np.array([0, 2, 1], np.int32)), 3)
    assert e.value.status == 3
    with pytest.raises(gnn.GnnError) as e:
        gnn.graph_ptr_from_ids(to_dev(np.array([0, 1, 5], np.int32)), 3)
    assert e.value.status == 3
