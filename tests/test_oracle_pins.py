"""Pins for the CPU checker: each of its functions is tied to something other than itself --
closed forms, dense brute force with numpy, invariants, fp64 finite differences -- so that a
dropped term, a wrong sign or index, or a swapped source/target fails here.  CPU only."""
import os

import numpy as np
import pytest

import oracle
from paper_2412_06354_b200 import synth

RNG = np.random.default_rng(20241206)
GOLD = os.path.join(os.path.dirname(__file__), "golden", "gcn_closed_forms.txt")


def rand_graph(n, e, rng=RNG, loops=True):
    src = rng.integers(0, n, e).astype(np.int32)
    dst = rng.integers(0, n, e).astype(np.int32)
    if not loops:
        dst = np.where(dst == src, (dst + 1) % n, dst).astype(np.int32)
    return src, dst


def dense_adj(n, src, dst, w=None):
    """A[j, i] = (weighted) multiplicity of edge j -> i."""
    A = np.zeros((n, n))
    np.add.at(A, (src, dst), 1.0 if w is None else w.astype(np.float64))
    return A


def undirected(pairs):
    s = [u for u, v in pairs] + [v for u, v in pairs]
    d = [v for u, v in pairs] + [u for u, v in pairs]
    return np.array(s, np.int32), np.array(d, np.int32)


def golden():
    out = {}
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        out[k] = float(v)
    return out


# ---------------------------------------------------------------- direction and topology
def test_direction_source_to_target():
    X = np.array([[3.0, -2.0], [7.0, 11.0]])
    out, S, arg = oracle.propagate("sum", 2, [0], [1], X)
    assert np.array_equal(out[1], X[0]) and np.array_equal(out[0], [0.0, 0.0])
    m = oracle.apply_edges(oracle.COPY_XJ, [0], [1], X)
    assert np.array_equal(m[0], X[0])
    out2, _, _ = oracle.aggregate("sum", 2, [1], m)
    assert np.array_equal(out2, out)


def test_coo_to_csr_invariants_and_bruteforce():
    n, e = 37, 400
    src, dst = rand_graph(n, e)
    rowptr, col, eid = oracle.coo_to_csr(n, dst, src)
    assert rowptr[0] == 0 and rowptr[-1] == e
    assert np.array_equal(np.diff(rowptr), np.bincount(dst, minlength=n))
    assert np.array_equal(np.sort(eid), np.arange(e))
    assert np.all(np.diff(dst[eid]) >= 0)
    for i in range(n):
        seg = eid[rowptr[i]:rowptr[i + 1]]
        assert np.all(np.diff(seg) > 0) and np.all(dst[seg] == i)
    assert np.array_equal(col, src[eid])
    # python's sort is stable: an independent statement of the same order
    ref = np.array(sorted(range(e), key=lambda k: dst[k]), np.int32)
    assert np.array_equal(eid, ref)
    # three encodings of one graph: COO -> sparse -> dense == COO -> dense
    A = np.zeros((n, n))
    for i in range(n):
        for p in range(rowptr[i], rowptr[i + 1]):
            A[col[p], i] += 1
    assert np.array_equal(A, dense_adj(n, src, dst))
    # transposed form and the position map between the two
    rowptrT, colT, eidT = oracle.coo_to_csr(n, src, dst)
    t2f = oracle.t2f(eid, eidT)
    assert np.array_equal(eid[t2f], eidT)
    assert np.array_equal(colT, dst[eidT])


def test_coo_to_csr_rejects_bad_index():
    with pytest.raises(IndexError):
        oracle.coo_to_csr(3, [0, 3], [1, 1])
    with pytest.raises(IndexError):
        oracle.coo_to_csr(3, [0, 1], [-1, 1])


def test_degree_closed_forms():
    n = 6
    s, d = undirected([(0, i) for i in range(1, n)])  # star
    di, dw = oracle.degree(n, d)
    assert di.tolist() == [n - 1] + [1] * (n - 1) and di.sum() == len(d)
    do, _ = oracle.degree(n, s)
    assert np.array_equal(di, do)  # symmetric graph: in == out
    s, d = undirected([(0, 1), (1, 2), (2, 3)])  # path
    assert oracle.degree(4, d)[0].tolist() == [1, 2, 2, 1]
    w = np.array([0.5, 2.0, 1.0], np.float32)
    _, dw = oracle.degree(3, [2, 2, 0], w)  # duplicates counted
    assert dw.tolist() == [1.0, 0.0, 2.5]
    di, _ = oracle.degree(3, [2, 2, 0])
    assert di.tolist() == [1, 0, 2]


# ---------------------------------------------------------------- GCN closed forms + dense
def gcn_propagate_ones(n, pairs):
    s, d = undirected(pairs)
    s, d = synth.with_self_loops(n, s, d)
    c = oracle.gcn_norm(n, s, d)
    out, _, _ = oracle.propagate("sum", n, s, d, np.ones((n, 1)), c.astype(np.float32))
    out64 = oracle.aggregate("sum", n, d, c[:, None] * np.ones((len(s), 1)))[0]
    return out[:, 0], out64[:, 0]


@pytest.mark.parametrize("n", [5, 8])
def test_gcn_star_closed_form(n):
    g = golden()
    y32, y = gcn_propagate_ones(n, [(0, i) for i in range(1, n)])
    assert abs(y[0] - g[f"star{n}_hub"]) < 1e-14
    assert np.all(np.abs(y[1:] - g[f"star{n}_leaf"]) < 1e-14)
    assert np.allclose(y32, y, rtol=1e-7)  # coefficients rounded to f32 on the way in


def test_gcn_path_closed_form():
    g = golden()
    _, y = gcn_propagate_ones(4, [(0, 1), (1, 2), (2, 3)])
    assert np.allclose(y, [g["path4_end"], g["path4_inner"], g["path4_inner"], g["path4_end"]], atol=1e-14, rtol=0)


def test_gcn_dense_bruteforce_and_eigenvector():
    n, F = 40, 5
    src, dst = synth.gnm(n, 90, 7)
    s, d = synth.with_self_loops(n, src, dst)
    X = RNG.standard_normal((n, F))
    W = RNG.standard_normal((F, 3))
    c = oracle.gcn_norm(n, s, d)
    A = dense_adj(n, src, dst) + np.eye(n)
    deg = A.sum(axis=0)
    Dm = np.diag(deg ** -0.5)
    ref = (Dm @ A.T @ Dm) @ X @ W
    m = c[:, None] * oracle.gather(s, X)
    agg = oracle.aggregate("sum", n, d, m)[0]
    Y, _ = oracle.matmul(agg, W)
    assert np.allclose(Y, ref, atol=1e-12)
    # sqrt(d) is a fixed vector of the normalised operator
    v = oracle.aggregate("sum", n, d, c[:, None] * np.sqrt(deg)[s][:, None])[0][:, 0]
    assert np.allclose(v, np.sqrt(deg), atol=1e-12)


def test_gcn_norm_weighted_and_zero_degree():
    # directed, weighted, node 2 has no incoming edge -> coefficient 0 for edges leaving it
    src = np.array([0, 1, 2, 0], np.int32)
    dst = np.array([1, 0, 0, 0], np.int32)
    w = np.array([2.0, 0.5, 1.0, 4.0], np.float32)
    c = oracle.gcn_norm(3, src, dst, w)
    d = np.array([0.5 + 1.0 + 4.0, 2.0, 0.0])
    exp = [2.0 / np.sqrt(d[1] * d[0]), 0.5 / np.sqrt(d[0] * d[1]), 0.0, 4.0 / np.sqrt(d[0] * d[0])]
    assert np.allclose(c, exp, atol=1e-15)


# ---------------------------------------------------------------- gather / apply_edges
def test_gather_is_a_copy():
    X = synth.normal_f32((9, 4), 1)
    idx = np.array([8, 0, 0, 3], np.int32)
    assert np.array_equal(oracle.gather(idx, X), X[idx].astype(np.float64))
    Xb = synth.normal_bf16((9, 8), 2)
    assert np.array_equal(oracle.gather(idx, Xb), synth.to_f64(Xb)[idx])


def test_apply_edges_messages():
    n, e, H, Cw = 11, 50, 2, 3
    F = H * Cw
    src, dst = rand_graph(n, e)
    X = RNG.standard_normal((n, F))
    assert np.array_equal(oracle.apply_edges(oracle.COPY_XJ, src, dst, X), X[src])
    ones = np.ones(e)
    assert np.array_equal(oracle.apply_edges(oracle.E_MUL_XJ, src, dst, X, e=ones), X[src])
    w1 = RNG.standard_normal(e)
    assert np.array_equal(oracle.apply_edges(oracle.E_MUL_XJ, src, dst, X, e=w1), w1[:, None] * X[src])
    wh = RNG.standard_normal((e, H))
    ref = (wh[:, :, None] * X[src].reshape(e, H, Cw)).reshape(e, F)
    assert np.array_equal(oracle.apply_edges(oracle.E_MUL_XJ, src, dst, X, e=wh), ref)
    wf = RNG.standard_normal((e, F))
    assert np.array_equal(oracle.apply_edges(oracle.E_MUL_XJ, src, dst, X, e=wf), wf * X[src])
    al, ar = RNG.standard_normal((n, H)), RNG.standard_normal((n, H))
    z = al[src] + ar[dst]
    ref = np.where(z > 0, z, 0.2 * z)
    assert np.allclose(oracle.apply_edges(oracle.GAT_LOGIT, src, dst, al, Y=ar, slope=0.2), ref, atol=1e-15)
    # slope is honoured and the negative side is scaled, not clipped
    got = oracle.apply_edges(oracle.GAT_LOGIT, [0], [1], np.array([[-1.0], [0.0]]), Y=np.array([[0.0], [-1.0]]), slope=0.5)
    assert got[0, 0] == -1.0


# ---------------------------------------------------------------- aggregate / propagate
@pytest.mark.parametrize("weighted", [False, True])
def test_sum_equals_dense_product(weighted):
    n, e, F = 48, 600, 7
    src, dst = rand_graph(n, e)
    X = RNG.standard_normal((n, F))
    w = RNG.random(e).astype(np.float32) if weighted else None
    out, S, _ = oracle.propagate("sum", n, src, dst, X, w)
    assert np.allclose(out, dense_adj(n, src, dst, w).T @ X, atol=1e-12)
    assert np.allclose(S, dense_adj(n, src, dst, None if w is None else np.abs(w)).T @ np.abs(X), atol=1e-12)
    # fused == aggregate(apply_edges)
    msg = oracle.E_MUL_XJ if weighted else oracle.COPY_XJ
    m = oracle.apply_edges(msg, src, dst, X, e=w)
    out2, S2, _ = oracle.aggregate("sum", n, dst, m)
    assert np.allclose(out, out2, atol=1e-13) and np.allclose(S, S2, atol=1e-13)


def test_mean_keeps_constants_and_bounds():
    n, e, F = 30, 120, 4
    src, dst = rand_graph(n, e)
    deg = np.bincount(dst, minlength=n)
    Xc = np.full((n, F), 3.25)
    out, _, _ = oracle.propagate("mean", n, src, dst, Xc)
    assert np.all(out[deg > 0] == 3.25) and np.all(out[deg == 0] == 0.0)
    X = RNG.standard_normal((n, F))
    mean = oracle.propagate("mean", n, src, dst, X)[0]
    summ = oracle.propagate("sum", n, src, dst, X)[0]
    mx, _, amx = oracle.propagate("max", n, src, dst, X)
    mn, _, amn = oracle.propagate("min", n, src, dst, X)
    nz = deg > 0
    assert np.allclose(mean[nz], summ[nz] / deg[nz][:, None], atol=1e-14)
    assert np.all(mn[nz] <= mean[nz] + 1e-15) and np.all(mean[nz] <= mx[nz] + 1e-15)
    # brute force per row, and the winner index points at the winning value
    for i in range(n):
        ks = np.nonzero(dst == i)[0]
        if len(ks) == 0:
            assert np.all(mx[i] == 0) and np.all(amx[i] == -1) and np.all(amn[i] == -1)
            continue
        assert np.array_equal(mx[i], X[src[ks]].max(axis=0))
        assert np.array_equal(mn[i], X[src[ks]].min(axis=0))
        for f in range(F):
            assert dst[amx[i, f]] == i and X[src[amx[i, f]], f] == mx[i, f]
            assert dst[amn[i, f]] == i and X[src[amn[i, f]], f] == mn[i, f]
    # aggregate path agrees with fused path for max (values and winners)
    m = oracle.apply_edges(oracle.COPY_XJ, src, dst, X)
    mx2, _, amx2 = oracle.aggregate("max", n, dst, m)
    assert np.array_equal(mx, mx2) and np.array_equal(amx, amx2)


def test_max_min_tie_break_first_edge_and_signed_zero():
    # three edges into node 0 with equal values: the first edge wins
    X = np.array([[0.0], [5.0], [5.0], [5.0], [-0.0]])
    src = np.array([2, 1, 3], np.int32)
    dst = np.zeros(3, np.int32)
    for op in ("max", "min"):
        v, _, a = oracle.propagate(op, 5, src, dst, X)
        assert v[0, 0] == 5.0 and a[0, 0] == 0
    # +0 and -0 compare equal: first stays, and its sign bit is what is returned
    v, _, a = oracle.propagate("max", 5, [4, 0], [1, 1], X)
    assert a[1, 0] == 0 and np.signbit(v[1, 0])
    v, _, a = oracle.propagate("min", 5, [0, 4], [1, 1], X)
    assert a[1, 0] == 0 and not np.signbit(v[1, 0])


def test_propagate_row_subset_matches_full():
    n, e, F = 50, 700, 6
    src, dst = rand_graph(n, e)
    X = synth.normal_f32((n, F), 3)
    w = RNG.random(e).astype(np.float32)
    rows = np.array([49, 0, 7, 23])
    for op in ("sum", "mean", "max"):
        full = oracle.propagate(op, n, src, dst, X, w)
        part = oracle.propagate(op, n, src, dst, X, w, rows=rows)
        for a, b in zip(full, part):
            assert np.array_equal(a[rows], b)


def test_propagate_backward_source_row_subset_matches_full():
    """The rows= path of the backward (a slot per SOURCE row) against the full result, which the finite
    differences below pin; rows unsorted, first and last row included, directed graph so that a slot
    looked up through the wrong endpoint lands in another row."""
    n, e, F = 50, 700, 6
    src, dst = rand_graph(n, e)
    X = synth.normal_f32((n, F), 5)
    R = synth.normal_f32((n, F), 6)
    w = RNG.random(e).astype(np.float32)
    rows = np.array([49, 0, 31, 7, 23])
    outdeg = np.bincount(src, minlength=n)
    assert (outdeg[rows] > 0).all() and len(set(src[:20]) - set(dst[:20])) > 0
    for op in ("sum", "mean", "max", "min"):
        arg = oracle.propagate(op, n, src, dst, X, w)[2] if op in ("max", "min") else None
        full = oracle.propagate_backward(op, n, src, dst, X, w, R, arg=arg)
        part = oracle.propagate_backward(op, n, src, dst, X, w, R, arg=arg, rows=rows)
        assert part["dX"].shape == (len(rows), F)
        assert np.array_equal(full["dX"][rows], part["dX"]) and np.array_equal(full["SdX"][rows], part["SdX"])
        assert np.abs(part["dX"]).sum() > 0
    # and against the definition written out for the subset: dX[j] = sum over edges out of j
    part = oracle.propagate_backward("mean", n, src, dst, X, w, R, rows=rows)
    indeg = np.bincount(dst, minlength=n)
    for t, j in enumerate(rows):
        ref = np.zeros(F)
        for k in np.nonzero(src == j)[0]:
            ref += float(w[k]) / indeg[dst[k]] * R[dst[k]].astype(np.float64)
        assert np.allclose(part["dX"][t], ref, rtol=1e-13, atol=1e-15)


def test_weighted_max_compares_messages_rounded_to_f32():
    """Stored (fp32) features: the winner is decided on w*x rounded once to fp32, the precision a
    device compares in; two exact products that differ below fp32 resolution tie and the first
    edge wins.  fp64 features are compared exactly."""
    u = 2.0 ** -23
    X32 = np.array([[1.0 + 2 * u], [1.0 + u], [0.0]], np.float32)   # nodes 0, 1 feed node 2
    w = np.array([1.0, 1.0 + u], np.float32)
    src, dst = np.array([0, 1], np.int32), np.array([2, 2], np.int32)
    p0, p1 = float(w[0]) * float(X32[0, 0]), float(w[1]) * float(X32[1, 0])
    assert p1 > p0 and np.float32(p1) == np.float32(p0)
    v, _, a = oracle.propagate("max", 3, src, dst, X32, w)
    assert a[2, 0] == 0 and v[2, 0] == float(np.float32(p0))
    v, _, a = oracle.propagate("max", 3, src, dst, X32.astype(np.float64), w)
    assert a[2, 0] == 1 and v[2, 0] == p1
    v, _, a = oracle.propagate("min", 3, src[::-1].copy(), dst, X32, w[::-1].copy())
    assert a[2, 0] == 0   # the same tie under min, other edge first


@pytest.mark.parametrize("op", ["max", "min"])
def test_weighted_max_backward_finite_differences(op):
    n, e, F = 20, 150, 4
    src, dst = rand_graph(n, e)
    X = RNG.standard_normal((n, F))
    w = (RNG.random(e) + 0.5).astype(np.float32) * np.where(RNG.random(e) < 0.3, -1, 1).astype(np.float32)
    R = RNG.standard_normal((n, F))
    arg = oracle.propagate(op, n, src, dst, X, w)[2]
    bw = oracle.propagate_backward(op, n, src, dst, X, w, R, arg=arg)
    loss = lambda: (oracle.propagate(op, n, src, dst, X, w)[0] * R).sum()
    ids = RNG.choice(X.size, 60, replace=False)
    assert np.allclose(fd(loss, X, ids, h=1e-7), bw["dX"].reshape(-1)[ids], rtol=1e-6, atol=1e-8)
    # fused == apply_edges + aggregate for the weighted message
    m = oracle.apply_edges(oracle.E_MUL_XJ, src, dst, X, e=w)
    v2, _, a2 = oracle.aggregate(op, n, dst, m)
    v1, _, a1 = oracle.propagate(op, n, src, dst, X, w)
    assert np.array_equal(v1, v2) and np.array_equal(a1, a2)


def test_thread_count_does_not_change_results():
    n, e, F = 64, 2000, 8
    src, dst = rand_graph(n, e)
    X = synth.normal_f32((n, F), 4)
    w = RNG.random(e).astype(np.float32)
    R = RNG.standard_normal((n, F))
    oracle.set_threads(1)
    a = oracle.propagate("sum", n, src, dst, X, w)
    ab = oracle.propagate_backward("sum", n, src, dst, X, w, R, want_dw=True)
    oracle.set_threads(5)
    b = oracle.propagate("sum", n, src, dst, X, w)
    bb = oracle.propagate_backward("sum", n, src, dst, X, w, R, want_dw=True)
    oracle.set_threads(1)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))
    assert all(np.array_equal(ab[k], bb[k]) for k in ab)


# ---------------------------------------------------------------- backward passes
def fd(fun, x, idxs, h=1e-6):
    g = np.empty(len(idxs))
    flat = x.reshape(-1)
    for t, i in enumerate(idxs):
        old = flat[i]
        flat[i] = old + h
        fp = fun()
        flat[i] = old - h
        fm = fun()
        flat[i] = old
        g[t] = (fp - fm) / (2 * h)
    return g


@pytest.mark.parametrize("op", ["sum", "mean"])
def test_propagate_backward_adjoint_and_finite_differences(op):
    n, e, F = 25, 160, 5
    src, dst = rand_graph(n, e)
    X = RNG.standard_normal((n, F))
    w32 = RNG.random(e).astype(np.float32) + 0.1
    R = RNG.standard_normal((n, F))
    bw = oracle.propagate_backward(op, n, src, dst, X, w32, R, want_dw=True)
    out = oracle.propagate(op, n, src, dst, X, w32)[0]
    # adjoint identity <P(X), R> = <X, P^T(R)>
    assert abs((out * R).sum() - (X * bw["dX"]).sum()) < 1e-11
    loss = lambda: (oracle.propagate(op, n, src, dst, X, w32)[0] * R).sum()
    ids = RNG.choice(X.size, 60, replace=False)
    g = fd(loss, X, ids)
    assert np.allclose(g, bw["dX"].reshape(-1)[ids], rtol=1e-6, atol=1e-8)
    # edge-weight gradient: the loss is linear in w, so a float32 step is exact enough
    w = w32.copy()
    for k in RNG.choice(e, 40, replace=False):
        wp, wm = w.copy(), w.copy()
        wp[k] += 0.25
        wm[k] -= 0.25
        step = float(wp[k]) - float(wm[k])  # the float32 steps actually taken
        num = ((oracle.propagate(op, n, src, dst, X, wp)[0] * R).sum() - (oracle.propagate(op, n, src, dst, X, wm)[0] * R).sum()) / step
        assert abs(num - bw["dw"][k]) < 1e-9 * max(1.0, abs(num))


@pytest.mark.parametrize("op", ["max", "min"])
def test_max_backward_routes_to_winner(op):
    n, e, F = 20, 150, 4
    src, dst = rand_graph(n, e)
    X = RNG.standard_normal((n, F))  # fp64 random: no ties
    R = RNG.standard_normal((n, F))
    out, _, arg = oracle.propagate(op, n, src, dst, X)
    bw = oracle.propagate_backward(op, n, src, dst, X, None, R, arg=arg)
    deg = np.bincount(dst, minlength=n)
    assert np.allclose(bw["dX"].sum(axis=0), R[deg > 0].sum(axis=0), atol=1e-12)
    loss = lambda: (oracle.propagate(op, n, src, dst, X)[0] * R).sum()
    ids = RNG.choice(X.size, 50, replace=False)
    assert np.allclose(fd(loss, X, ids, h=1e-7), bw["dX"].reshape(-1)[ids], rtol=1e-6, atol=1e-8)
    # w.r.t. the message tensor
    dm = oracle.aggregate_backward(op, n, dst, R, arg)
    ref = np.zeros((e, F))
    for i in range(n):
        for f in range(F):
            if arg[i, f] >= 0:
                ref[arg[i, f], f] = R[i, f]
    assert np.array_equal(dm, ref)


def test_gather_and_aggregate_backward_are_transposes():
    n, e, F = 17, 90, 3
    src, dst = rand_graph(n, e)
    X = RNG.standard_normal((n, F))
    Re = RNG.standard_normal((e, F))
    dX, S = oracle.gather_backward(n, src, Re)
    assert abs((oracle.gather(src, X) * Re).sum() - (X * dX).sum()) < 1e-11
    ref = np.zeros((n, F))
    np.add.at(ref, src, Re)
    assert np.allclose(dX, ref, atol=1e-13)
    Rn = RNG.standard_normal((n, F))
    m = RNG.standard_normal((e, F))
    for op in ("sum", "mean"):
        dm = oracle.aggregate_backward(op, n, dst, Rn)
        assert abs((oracle.aggregate(op, n, dst, m)[0] * Rn).sum() - (m * dm).sum()) < 1e-11


# ---------------------------------------------------------------- edge softmax / GAT
def test_edge_softmax_invariants():
    n, e, H = 15, 120, 3
    src, dst = rand_graph(n, e)
    s = RNG.standard_normal((e, H)) * 3
    a = oracle.edge_softmax(n, dst, s)
    tot = np.zeros((n, H))
    np.add.at(tot, dst, a)
    deg = np.bincount(dst, minlength=n)
    assert np.allclose(tot[deg > 0], 1.0, atol=1e-14) and np.all(tot[deg == 0] == 0)
    shift = RNG.standard_normal((n, H)) * 10
    assert np.allclose(oracle.edge_softmax(n, dst, s + shift[dst]), a, atol=1e-13)
    eq = oracle.edge_softmax(n, dst, np.full((e, H), 1.7))
    assert np.allclose(eq, 1.0 / deg[dst][:, None], atol=1e-15)
    # one edge -> 1 ; two edges -> logistic of the difference
    assert oracle.edge_softmax(2, [1], np.array([[123.0]]))[0, 0] == 1.0
    two = oracle.edge_softmax(2, [1, 1], np.array([[0.3], [-1.1]]))
    assert abs(two[0, 0] - 1 / (1 + np.exp(-(0.3 + 1.1)))) < 1e-15
    # large logits do not overflow (the row maximum is subtracted)
    big = oracle.edge_softmax(2, [1, 1], np.array([[1000.0], [999.0]]))
    assert np.isfinite(big).all() and abs(big.sum() - 1) < 1e-15


def test_edge_softmax_backward():
    n, e, H = 12, 80, 2
    src, dst = rand_graph(n, e)
    s = RNG.standard_normal((e, H))
    Rm = RNG.standard_normal((e, H))
    a = oracle.edge_softmax(n, dst, s)
    ds, S = oracle.edge_softmax_backward(n, dst, a, Rm)
    tot = np.zeros((n, H))
    np.add.at(tot, dst, ds)
    assert np.allclose(tot, 0, atol=1e-14)
    loss = lambda: (oracle.edge_softmax(n, dst, s) * Rm).sum()
    ids = RNG.choice(s.size, 60, replace=False)
    assert np.allclose(fd(loss, s, ids), ds.reshape(-1)[ids], rtol=1e-6, atol=1e-9)
    assert np.all(S >= np.abs(ds) - 1e-15)


def test_gat_reductions_and_composition():
    n, e, H, Cw = 30, 260, 2, 4
    F = H * Cw
    src, dst = rand_graph(n, e)
    Wx = RNG.standard_normal((n, F))
    zero = np.zeros((H, Cw), np.float32)
    g0 = oracle.gat(n, src, dst, Wx, zero, zero, H, Cw)
    assert np.allclose(g0["out"], oracle.propagate("mean", n, src, dst, Wx)[0], atol=1e-13)
    a_s = RNG.standard_normal((H, Cw)).astype(np.float32)
    a_d = RNG.standard_normal((H, Cw)).astype(np.float32)
    g = oracle.gat(n, src, dst, Wx, a_s, a_d, H, Cw)
    al = np.einsum("nhc,hc->nh", Wx.reshape(n, H, Cw), a_s.astype(np.float64))
    ar = np.einsum("nhc,hc->nh", Wx.reshape(n, H, Cw), a_d.astype(np.float64))
    assert np.allclose(g["al"], al, atol=1e-13) and np.allclose(g["ar"], ar, atol=1e-13)
    s = oracle.apply_edges(oracle.GAT_LOGIT, src, dst, al, Y=ar, slope=0.2)
    alpha = oracle.edge_softmax(n, dst, s)
    assert np.allclose(g["alpha"], alpha, atol=1e-14)
    m = oracle.apply_edges(oracle.E_MUL_XJ, src, dst, Wx, e=alpha)
    assert np.allclose(g["out"], oracle.aggregate("sum", n, dst, m)[0], atol=1e-13)
    # one dominant logit selects that source
    Wd = np.zeros((3, 2))
    Wd[0] = [50.0, 1.0]
    Wd[1] = [-50.0, 2.0]
    sel = oracle.gat(3, [0, 1], [2, 2], Wd, np.array([[1.0, 0.0]], np.float32), np.zeros((1, 2), np.float32), 1, 2)
    assert np.allclose(sel["out"][2], Wd[0], atol=1e-12)


def test_gat_backward_finite_differences():
    n, e, H, Cw = 14, 90, 2, 3
    F = H * Cw
    src, dst = rand_graph(n, e)
    Wx = RNG.standard_normal((n, F))
    a_s = RNG.standard_normal((H, Cw)).astype(np.float32)
    a_d = RNG.standard_normal((H, Cw)).astype(np.float32)
    R = RNG.standard_normal((n, F))
    fwd = oracle.gat(n, src, dst, Wx, a_s, a_d, H, Cw)
    bw = oracle.gat_backward(n, src, dst, Wx, a_s, a_d, H, Cw, fwd, R)
    loss = lambda: (oracle.gat(n, src, dst, Wx, a_s, a_d, H, Cw)["out"] * R).sum()
    ids = RNG.choice(Wx.size, 60, replace=False)
    assert np.allclose(fd(loss, Wx, ids), bw["dWx"].reshape(-1)[ids], rtol=2e-6, atol=1e-8)
    # attention vectors are float32 inputs: step in float32, compare to the analytic slope
    for name, arr in (("da_src", a_s), ("da_dst", a_d)):
        for i in range(arr.size):
            old = arr.reshape(-1)[i]
            h = np.float32(2.0 ** -10)
            arr.reshape(-1)[i] = old + h
            fp = loss()
            hp = float(arr.reshape(-1)[i]) - float(old)
            arr.reshape(-1)[i] = old - h
            fm = loss()
            hm = float(old) - float(arr.reshape(-1)[i])
            arr.reshape(-1)[i] = old
            num = (fp - fm) / (hp + hm)
            assert abs(num - bw[name].reshape(-1)[i]) < 2e-4 * max(1.0, abs(num))
    assert np.all(bw["SdWx"] >= np.abs(bw["dWx"]) - 1e-12)


# ---------------------------------------------------------------- pooling, batching, dense
def test_reduce_nodes_and_batch_equivalence():
    wl = synth.workload_batched(G=9, F=6)
    n, gp, X = wl["N"], wl["graph_ptr"], wl["X"]
    out, S, arg = oracle.reduce_nodes("mean", gp, X)
    for g in range(9):
        assert np.allclose(out[g], X[gp[g]:gp[g + 1]].astype(np.float64).mean(axis=0), atol=1e-14)
    # pooling == aggregation over the node -> graph bipartite edge list
    gid = np.repeat(np.arange(9), np.diff(gp)).astype(np.int32)
    for op in ("sum", "mean", "max", "min"):
        a = oracle.reduce_nodes(op, gp, X)
        b = oracle.aggregate(op, 9, gid, synth.to_f64(X))
        assert np.allclose(a[0], b[0], atol=1e-14) and np.array_equal(a[2], b[2])
    const = np.full((n, 2), -1.5)
    assert np.all(oracle.reduce_nodes("mean", gp, const)[0] == -1.5)
    # a layer on the batched graph == the layer on each member, concatenated
    full = oracle.propagate("mean", n, wl["src"], wl["dst"], X)[0]
    for g in range(9):
        a, b = gp[g], gp[g + 1]
        sel = (wl["dst"] >= a) & (wl["dst"] < b)
        part = oracle.propagate("mean", b - a, wl["src"][sel] - a, wl["dst"][sel] - a, X[a:b])[0]
        assert np.array_equal(full[a:b], part)
    # backward
    R = RNG.standard_normal((9, 6))
    for op in ("sum", "mean"):
        dX = oracle.reduce_nodes_backward(op, gp, R)
        assert abs((oracle.reduce_nodes(op, gp, X)[0] * R).sum() - (X * dX).sum()) < 1e-10
    _, _, amx = oracle.reduce_nodes("max", gp, X)
    dX = oracle.reduce_nodes_backward("max", gp, R, amx)
    assert np.allclose(dX.sum(axis=0), R.sum(axis=0), atol=1e-13)
    assert np.count_nonzero(dX) == R.size
    # empty graph in the batch
    o, _, a = oracle.reduce_nodes("max", np.array([0, 2, 2, 3], np.int32), np.array([[1.0], [2.0], [3.0]]))
    assert o[:, 0].tolist() == [2.0, 0.0, 3.0] and a[:, 0].tolist() == [1, -1, 2]


def test_matmul_matches_numpy():
    A = RNG.standard_normal((13, 7))
    B = RNG.standard_normal((7, 5))
    Y, S = oracle.matmul(A, B)
    assert np.allclose(Y, A @ B, atol=1e-13) and np.allclose(S, np.abs(A) @ np.abs(B), atol=1e-13)
    Dy = RNG.standard_normal((13, 5))
    assert np.allclose(oracle.matmul(Dy, B, tb=True)[0], Dy @ B.T, atol=1e-13)
    assert np.allclose(oracle.matmul(A, Dy, ta=True)[0], A.T @ Dy, atol=1e-13)
    Ab = synth.normal_bf16((4, 8), 5)
    Bf = synth.normal_f32((8, 3), 6)
    assert np.allclose(oracle.matmul(Ab, Bf)[0], synth.to_f64(Ab) @ Bf.astype(np.float64), atol=1e-13)


def test_bf16_and_f32_inputs_are_widened_exactly():
    # 0x3FC0 = 1.5, 0xC000 = -2.0, 0x3F81 = 1 + 2^-7
    Xb = np.array([[0x3FC0, 0xC000], [0x3F81, 0x0000]], np.uint16)
    out, _, _ = oracle.propagate("sum", 2, [0, 1], [1, 1], Xb)
    assert out[1].tolist() == [1.5 + 1.0078125, -2.0]


# ---------------------------------------------------------------- further messages, GIN, heterogeneous sums
def test_xi_sub_xj_and_xi_dot_xj_messages_against_dense_algebra():
    n, e, H, Cw = 23, 140, 2, 3
    F = H * Cw
    src, dst = rand_graph(n, e)
    Xj, Xi = RNG.standard_normal((n, F)), RNG.standard_normal((n, F))
    A = dense_adj(n, src, dst)                       # A[j, i] = multiplicity of j -> i
    deg = A.sum(axis=0)
    o, _, _ = oracle.propagate_msg(oracle.XI_SUB_XJ, "sum", n, src, dst, Xj, Xi=Xi)
    assert np.allclose(o, deg[:, None] * Xi - A.T @ Xj, atol=1e-12)
    m = oracle.apply_edges(oracle.XI_DOT_XJ, src, dst, Xj, Y=Xi, H=H)
    for h in range(H):
        G = Xi[:, h * Cw:(h + 1) * Cw] @ Xj[:, h * Cw:(h + 1) * Cw].T      # G[i, j]
        assert np.allclose(m[:, h], G[dst, src], atol=1e-12)
    # direction: on the single edge 0 -> 1 the message is x_i - x_j with i = 1, j = 0
    m = oracle.apply_edges(oracle.XI_SUB_XJ, [0], [1], Xj, Y=Xi)
    assert np.array_equal(m[0], Xi[1] - Xj[0])
    # max over x_i - x_j is x_i minus the smallest x_j
    o, _, a = oracle.propagate_msg(oracle.XI_SUB_XJ, "max", n, src, dst, Xj, Xi=Xi)
    mn, _, amn = oracle.propagate("min", n, src, dst, Xj)
    has = deg > 0
    assert np.allclose(o[has], (Xi - mn)[has], atol=1e-12) and np.array_equal(a, amn)


@pytest.mark.parametrize("msg", ["copy", "emul1", "emulH", "emulF", "sub", "dot"])
def test_apply_edges_backward_finite_differences(msg):
    n, e, H, Cw = 15, 70, 2, 4
    F = H * Cw
    src, dst = rand_graph(n, e)
    Xj, Xi = RNG.standard_normal((n, F)), RNG.standard_normal((n, F))
    code = {"copy": oracle.COPY_XJ, "emul1": oracle.E_MUL_XJ, "emulH": oracle.E_MUL_XJ, "emulF": oracle.E_MUL_XJ,
            "sub": oracle.XI_SUB_XJ, "dot": oracle.XI_DOT_XJ}[msg]
    ev = {"emul1": RNG.standard_normal((e, 1)), "emulH": RNG.standard_normal((e, H)), "emulF": RNG.standard_normal((e, F))}.get(msg)
    Y = Xi if msg in ("sub", "dot") else None
    dm = RNG.standard_normal((e, H if msg == "dot" else F))
    loss = lambda: (oracle.apply_edges(code, src, dst, Xj, Y=Y, e=ev, H=H) * dm).sum()
    want = ("dXj",) + (("dXi",) if Y is not None else ()) + (("de",) if ev is not None else ())
    bw = oracle.apply_edges_backward(code, n, src, dst, Xj, dm, Y=Y, e=ev, H=H, want=want)
    ids = RNG.choice(Xj.size, 40, replace=False)
    assert np.allclose(fd(loss, Xj, ids), bw["dXj"].reshape(-1)[ids], rtol=1e-6, atol=1e-8)
    if Y is not None:
        assert np.allclose(fd(loss, Xi, ids), bw["dXi"].reshape(-1)[ids], rtol=1e-6, atol=1e-8)
    if ev is not None:
        ide = RNG.choice(ev.size, 40, replace=False)
        assert np.allclose(fd(loss, ev, ide), bw["de"].reshape(-1)[ide], rtol=1e-6, atol=1e-8)
    # magnitude sums bound the results
    assert (np.abs(bw["dXj"]) <= bw["SXj"] + 1e-15).all()


def test_gin_closed_form_dense_form_and_gradient():
    # star with hub 0 and n-1 leaves, all features 1: hub = (1+eps) + (n-1), leaf = (1+eps) + 1
    n, eps = 6, 0.25
    src, dst = undirected([(0, k) for k in range(1, n)])
    o, S = oracle.gin(n, src, dst, np.ones((n, 2)), eps)
    assert np.allclose(o[0], 1 + eps + n - 1) and np.allclose(o[1:], 1 + eps + 1) and np.allclose(S, o)
    n, e, F = 30, 200, 4
    src, dst = rand_graph(n, e)
    X, R = RNG.standard_normal((n, F)), RNG.standard_normal((n, F))
    o, _ = oracle.gin(n, src, dst, X, eps)
    assert np.allclose(o, (dense_adj(n, src, dst).T + (1 + eps) * np.eye(n)) @ X, atol=1e-12)
    bw = oracle.gin_backward(n, src, dst, X, eps, R)
    ids = RNG.choice(X.size, 50, replace=False)
    assert np.allclose(fd(lambda: (oracle.gin(n, src, dst, X, eps)[0] * R).sum(), X, ids), bw["dX"].reshape(-1)[ids], rtol=1e-6, atol=1e-8)
    h = 1e-6
    num = ((oracle.gin(n, src, dst, X, eps + h)[0] * R).sum() - (oracle.gin(n, src, dst, X, eps - h)[0] * R).sum()) / (2 * h)
    assert abs(num - bw["deps"]) < 1e-6 * max(1.0, abs(num))


def test_hetero_sum_equals_one_propagate_over_the_merged_graph():
    """Three relations from three source node sets into one target set: the sum over relations equals one
    propagate over the union graph whose sources index the stacked feature matrix (mean as 1/deg weights)."""
    nd, F = 12, 3
    sizes = [7, 12, 20]
    rels, off, ms, md, mw, Xs = [], 0, [], [], [], []
    for t, ns in enumerate(sizes):
        e = 30 + 10 * t
        s = RNG.integers(0, ns, e).astype(np.int32)
        d = RNG.integers(0, nd, e).astype(np.int32)
        X = RNG.standard_normal((ns, F))
        op = "mean" if t == 1 else "sum"
        w = RNG.random(e).astype(np.float32) if t == 2 else None
        rels.append(dict(src=s, dst=d, X=X, w=w, op=op))
        deg = np.bincount(d, minlength=nd)
        ms.append(s + off); md.append(d); Xs.append(X)
        mw.append(1.0 / deg[d] if op == "mean" else (w.astype(np.float64) if w is not None else np.ones(e)))
        off += ns
    o, S = oracle.hetero_propagate(nd, rels)
    A = np.zeros((off, nd))
    np.add.at(A, (np.concatenate(ms), np.concatenate(md)), np.concatenate(mw))
    assert np.allclose(o, A.T @ np.concatenate(Xs), atol=1e-12) and (np.abs(o) <= S + 1e-15).all()


def test_epilogue_bias_relu_and_its_backward():
    Z = RNG.standard_normal((9, 5))
    b = RNG.standard_normal(5)
    R = RNG.standard_normal((9, 5))
    Y = oracle.epilogue(Z, b, "relu")
    assert (Y >= 0).all() and np.array_equal(Y[Y > 0], (Z + b)[Y > 0]) and np.array_equal(oracle.epilogue(Z, None, None), Z)
    dZ, db, _ = oracle.epilogue_backward(Y, R, "relu")
    ids = RNG.choice(Z.size, 30, replace=False)
    assert np.allclose(fd(lambda: (oracle.epilogue(Z, b, "relu") * R).sum(), Z, ids, h=1e-7), dZ.reshape(-1)[ids], atol=1e-6)
    assert np.allclose(fd(lambda: (oracle.epilogue(Z, b, "relu") * R).sum(), b, np.arange(5), h=1e-7), db, atol=1e-6)


def test_gatv2_logits_brute_force_linear_case_and_gradient():
    """GATv2-style logits: brute force by Python loops on a tiny graph; with slope 1 the nonlinearity vanishes and
    the logit is <a_h, xl_j + xr_i>; gradients against fp64 finite differences."""
    n, e, H, Cw = 9, 40, 2, 3
    F = H * Cw
    src, dst = rand_graph(n, e)
    Xl, Xr, a = RNG.standard_normal((n, F)), RNG.standard_normal((n, F)), RNG.standard_normal((H, Cw))
    s, S, _ = oracle.gatv2_logits(src, dst, Xl, Xr, a, H, slope=0.2)
    ref = np.zeros((e, H))
    for k in range(e):
        for h in range(H):
            for c in range(Cw):
                z = Xl[src[k], h * Cw + c] + Xr[dst[k], h * Cw + c]
                ref[k, h] += a[h, c] * (z if z > 0 else 0.2 * z)
    assert np.allclose(s, ref, atol=1e-13) and (np.abs(s) <= S + 1e-15).all()
    lin = oracle.gatv2_logits(src, dst, Xl, Xr, a, H, slope=1.0)[0]
    dense = np.einsum("khc,hc->kh", (Xl[src] + Xr[dst]).reshape(e, H, Cw), a)
    assert np.allclose(lin, dense, atol=1e-13)
    ds = RNG.standard_normal((e, H))
    loss = lambda: (oracle.gatv2_logits(src, dst, Xl, Xr, a, H, slope=0.2)[0] * ds).sum()
    bw = oracle.gatv2_logits_backward(n, src, dst, Xl, Xr, a, H, ds, slope=0.2)
    ids = RNG.choice(Xl.size, 30, replace=False)
    assert np.allclose(fd(loss, Xl, ids), bw["dXl"].reshape(-1)[ids], rtol=1e-6, atol=1e-8)
    assert np.allclose(fd(loss, Xr, ids), bw["dXr"].reshape(-1)[ids], rtol=1e-6, atol=1e-8)
    assert np.allclose(fd(loss, a, np.arange(a.size)), bw["da"].reshape(-1), rtol=1e-6, atol=1e-8)
