"""GPU parity of the merged sparse form for heterogeneous graphs (several relations into one target node set,
summed in relation order) and for temporal snapshot batches (same nodes, changing edges), against the CPU
checker: the relations / snapshots are looped over on the CPU and run as one launch on the device."""
import numpy as np
import pytest

import oracle
from paper_2412_06354_b200 import synth
from test_gpu_propagate import feats
from util import assert_close, bits, to_dev, to_host64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gnn():
    import torch
    from paper_2412_06354_b200 import gnn as g
    g.load()
    assert torch.cuda.is_available()
    return g


def merged_graph(gnn, segments, n_rows, n_cols, seg_is_mean, weights):
    """segments: [(src, dst, src_offset, dst_offset)] host arrays -> (graph, coef_csr, coef_csrT, host eid)."""
    import torch
    dev_segs = [(to_dev(s), to_dev(d), so, do) for s, d, so, do in segments]
    src, dst, seg = gnn.merge_edge_lists(dev_segs)
    g = gnn.coo_to_csr(max(n_rows, n_cols), src, dst)
    eid = g.eid[:g.E]
    seg_csr = gnn.permute_edge_data(eid, seg)
    w_csr = None
    if weights is not None:
        w_csr = gnn.permute_edge_data(eid, to_dev(np.concatenate(weights).astype(np.float32)))
    coef, coefT = gnn.segment_coef(g, seg_csr, torch.tensor(seg_is_mean, dtype=torch.int32, device="cuda"), w_csr)
    # inside every row the segments ascend: the sum over relations runs in relation order
    rp = g.rowptr.cpu().numpy()
    sc = seg_csr.cpu().numpy()
    inner = np.ones(g.E, bool)
    inner[rp[rp < g.E]] = False
    assert (np.diff(sc)[inner[1:]] >= 0).all()
    return g, coef, coefT


@pytest.mark.parametrize("dtype,F", [("f32", 64), ("bf16", 128), ("bf16", 512)])
def test_three_relations_into_one_target_type(gnn, dtype, F):
    rng = np.random.default_rng(F)
    n_dst = 600
    n_src = [500, 800, 300]  # three source node types; relation r sends from type r
    ne = [9000, 20000, 2500]
    ops = ["sum", "mean", "mean"]
    offs = np.concatenate([[0], np.cumsum(n_src)])
    rels, segments, weights = [], [], []
    for r in range(3):
        src = rng.integers(0, n_src[r], ne[r]).astype(np.int32)
        dst = rng.integers(0, n_dst - 40, ne[r]).astype(np.int32)  # the last targets receive nothing
        if r == 1:
            dst[:3000] = 5  # a hub target inside one relation
        w = synth.uniform_f32((ne[r],), 0.0, 1.0, 20 + r) if r != 2 else np.ones(ne[r], np.float32)
        X = feats((n_src[r], F), dtype, 30 + r + F)
        rels.append(dict(src=src, dst=dst, X=X, w=None if r == 2 else w, op=ops[r]))
        segments.append((src, dst, int(offs[r]), 0))
        weights.append(w)
    Xs = np.concatenate([r["X"] for r in rels])
    g, coef, coefT = merged_graph(gnn, segments, n_dst, int(offs[-1]), [int(o == "mean") for o in ops], weights)
    out = gnn.propagate_fused(g, to_dev(Xs), coef, "sum")
    o, S = oracle.hetero_propagate(n_dst, rels)
    assert_close(to_host64(out)[:n_dst], o, S, dtype, "sum over three relations")
    assert not to_host64(out)[n_dst:].any(), "rows beyond the target type must stay empty"
    assert np.array_equal(bits(out), bits(gnn.propagate_fused(g, to_dev(Xs), coef, "sum"))), "not bit-reproducible"
    # backward: every source type receives the gradient of its own relation
    R = feats((g.N, F), dtype, 40 + F, stream=1)
    if g.N > n_dst:
        R[n_dst:] = 0
    dX, _ = gnn.propagate_fused_backward(g, to_dev(R), "sum", w_csrT=coefT)
    got = to_host64(dX)
    for r, rel in enumerate(rels):
        n = max(n_dst, n_src[r])
        Rp = R[:n] if n <= R.shape[0] else np.concatenate([R, np.zeros((n - R.shape[0], F), R.dtype)])
        bw = oracle.propagate_backward(rel["op"], n, rel["src"], rel["dst"], None, rel["w"], Rp)
        a, b = int(offs[r]), int(offs[r + 1])
        assert_close(got[a:b], bw["dX"][:n_src[r]], bw["SdX"][:n_src[r]], dtype, f"dX of source type {r}")


@pytest.mark.parametrize("static_features", [True, False])
@pytest.mark.parametrize("dtype,F", [("f32", 32), ("bf16", 256)])
def test_temporal_snapshots_as_one_launch(gnn, dtype, F, static_features):
    rng = np.random.default_rng(7 + F)
    n, T = 700, 5
    snaps, segments = [], []
    for t in range(T):
        e = 3000 + 1500 * t
        src = rng.integers(0, n, e).astype(np.int32)
        dst = rng.integers(0, n, e).astype(np.int32)
        snaps.append((src, dst))
        segments.append((src, dst, 0 if static_features else t * n, t * n))
    X = feats((n if static_features else T * n, F), dtype, 50 + F)
    g, coef, coefT = merged_graph(gnn, segments, T * n, X.shape[0], [1] * T, None)
    out = to_host64(gnn.propagate_fused(g, to_dev(X), coef, "sum"))
    R = feats((T * n, F), dtype, 51 + F, stream=1)
    dX = to_host64(gnn.propagate_fused_backward(g, to_dev(R), "sum", w_csrT=coefT)[0])
    acc, accS = 0.0, 0.0
    for t, (src, dst) in enumerate(snaps):
        Xt = X if static_features else X[t * n:(t + 1) * n]
        o, S, _ = oracle.propagate("mean", n, src, dst, Xt)
        assert_close(out[t * n:(t + 1) * n], o, S, dtype, f"snapshot {t}")
        bw = oracle.propagate_backward("mean", n, src, dst, None, None, R[t * n:(t + 1) * n])
        if static_features:  # one feature matrix serves every snapshot: its gradient is the sum over time
            acc, accS = acc + bw["dX"], accS + bw["SdX"]
        else:
            assert_close(dX[t * n:(t + 1) * n], bw["dX"], bw["SdX"], dtype, f"dX of snapshot {t}")
    if static_features:
        assert_close(dX[:n], acc, accS, dtype, "dX summed over the snapshots")


def test_merge_rejects_bad_segments(gnn):
    import torch
    s = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(gnn.GnnError) as err:
        gnn.merge_edge_lists([(s, s, -1, 0)])
    assert err.value.status == 1
    src, dst, seg = gnn.merge_edge_lists([(s, s, 3, 2), (s[:0], s[:0], 0, 0), (s, s + 1, 0, 7)])
    assert src.cpu().tolist() == [3] * 4 + [0] * 4 and dst.cpu().tolist() == [2] * 4 + [8] * 4
    assert seg.cpu().tolist() == [0] * 4 + [2] * 4
