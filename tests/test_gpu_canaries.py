"""Guard bands around every buffer the binding allocates (outputs, saved tensors, workspaces, the graph's own
arrays): 4 KB of a known pattern directly before and directly after each buffer, checked after every call.
A kernel that writes one element outside what it was given fails here.  This stands in for a memory checker.
Values are checked elsewhere; here only the bands are."""
import numpy as np
import pytest

from paper_2412_06354_b200 import synth
from util import to_dev

pytestmark = pytest.mark.gpu

PAD = 4096
PATTERN = 0xA5


class GuardedTorch:
    """Stands in for the `torch` module inside the binding: empty() / empty_like() return exact-size views into
    larger buffers whose first and last 4 KB hold a pattern; everything else is the real torch."""

    def __init__(self, torch):
        self._torch = torch
        self.bufs = []

    def __getattr__(self, name):
        return getattr(self._torch, name)

    def empty(self, *size, dtype=None, device=None, **kw):
        torch = self._torch
        shape = tuple(size[0]) if len(size) == 1 and isinstance(size[0], (tuple, list, torch.Size)) else tuple(int(x) for x in size)
        dtype = dtype or torch.float32
        nbytes = int(np.prod(shape, dtype=np.int64)) * torch.empty(0, dtype=dtype).element_size()
        buf = torch.full((PAD + nbytes + PAD,), PATTERN, dtype=torch.uint8, device=device)
        self.bufs.append((buf, nbytes))
        return buf[PAD:PAD + nbytes].view(dtype).view(shape)

    def empty_like(self, t):
        return self.empty(tuple(t.shape), dtype=t.dtype, device=t.device)

    def check(self, what):
        torch = self._torch
        torch.cuda.synchronize()
        for k, (buf, nbytes) in enumerate(self.bufs):
            assert bool((buf[:PAD] == PATTERN).all()), f"{what}: write before buffer {k} ({nbytes} bytes)"
            assert bool((buf[PAD + nbytes:] == PATTERN).all()), f"{what}: write past buffer {k} ({nbytes} bytes)"
        self.bufs.clear()


@pytest.fixture()
def guarded(monkeypatch):
    import torch
    from paper_2412_06354_b200 import gnn
    gnn.load()
    gt = GuardedTorch(torch)
    monkeypatch.setattr(gnn, "torch", gt)
    return gnn, gt


def graph(n, e, seed, hub=0):
    rng = np.random.default_rng(seed)
    src = rng.integers(0, n, e).astype(np.int32)
    dst = rng.integers(0, max(n - n // 10, 1), e).astype(np.int32)  # the last tenth of the nodes receives nothing
    if hub:
        dst[:hub] = n // 3
    p = rng.permutation(e)
    return src[p].copy(), dst[p].copy()


@pytest.mark.parametrize("n,e,hub", [(1500, 30_000, 6000), (333, 777, 0), (5000, 200_001, 20_000), (9000, 600_013, 50_000)])
def test_graph_setup_and_propagate_stay_inside_their_buffers(guarded, n, e, hub):
    gnn, gt = guarded
    src, dst = graph(n, e, n + e, hub)
    g = gnn.coo_to_csr(n, to_dev(src), to_dev(dst))
    gt.check("coo_to_csr")
    gnn.degree(g); gnn.degree(g, transposed=True)
    gt.check("degree")
    w = to_dev(synth.uniform_f32((e,), 0.1, 1.0, 3))
    w_csr = gnn.permute_edge_data(g.eid[:g.E], w)
    gt.check("permute_edge_data")
    for dtype, F in [("f32", 4), ("f32", 100), ("f32", 128), ("f32", 260), ("f32", 512), ("bf16", 8), ("bf16", 200), ("bf16", 256), ("bf16", 520), ("bf16", 1024)]:
        X = to_dev(synth.normal((n, F), dtype, 5))
        for op in ("sum", "mean", "max", "min"):
            r = gnn.propagate_fused(g, X, w_csr if op == "sum" else None, op)
            gt.check(f"propagate {op} F={F} {dtype}")
            arg = r[1] if op in ("max", "min") else None
            gnn.propagate_fused_backward(g, X, op, X=X, w_csrT=w_csr if op == "sum" else None, argmax=arg, want_dW=op in ("sum", "mean"))
            gt.check(f"propagate backward {op} F={F} {dtype}")
    X = to_dev(synth.normal_f32((n, 64), 6))
    gnn.propagate_fused_static(g, X, None, "sum") if gnn.propagate_fused_workspace(g.E, 64, "sum") <= (8 << 20) else None
    gt.check("propagate static")


def test_row_walking_kernel_with_narrow_rows_stays_inside_its_buffers(guarded):
    """8.4 M edges: narrow rows on the row-walking kernel (1024 positions per warp)."""
    gnn, gt = guarded
    n, e = 50_000, 8_400_000
    src, dst = graph(n, e, 1, hub=400_000)
    g = gnn.coo_to_csr(n, to_dev(src), to_dev(dst))
    gt.check("coo_to_csr")
    for dtype, F in [("f32", 8), ("bf16", 32), ("bf16", 72), ("f32", 128)]:
        X = to_dev(synth.normal((n, F), dtype, 7))
        for op in ("sum", "max"):
            r = gnn.propagate_fused(g, X, None, op)
            gt.check(f"propagate {op} F={F} {dtype}")
            gnn.propagate_fused_backward(g, X, op, X=X, argmax=r[1] if op == "max" else None, want_dW=op == "sum")
            gt.check(f"backward {op} F={F} {dtype}")


def test_unfused_softmax_pooling_attention_and_dense_stay_inside_their_buffers(guarded):
    import torch
    gnn, gt = guarded
    n, e = 1500, 30_000
    src, dst = graph(n, e, 11, hub=5000)
    g = gnn.coo_to_csr(n, to_dev(src), to_dev(dst))
    for dtype, F in [("f32", 20), ("bf16", 64), ("f32", 256)]:
        X = to_dev(synth.normal((n, F), dtype, 12))
        m = gnn.gather(g.col[:g.E], X)
        gt.check("gather")
        gnn.gather_backward(g, m); gnn.gather_backward(g, m, by_src=True)
        gt.check("gather_backward")
        ew = to_dev(synth.uniform_f32((e,), 0.0, 1.0, 13))
        m = gnn.apply_edges(g, gnn.E_MUL_XJ, X, e=ew)
        gt.check("apply_edges")
        for op in ("sum", "mean", "max"):
            r = gnn.aggregate(g, m[:g.E], op)
            gt.check(f"aggregate {op}")
            gnn.aggregate_backward(g, X, op, argmax=r[1] if op == "max" else None)
            gt.check(f"aggregate_backward {op}")
    for H in (1, 3, 8):
        s = to_dev(synth.normal_f32((e, H), 14))
        a = gnn.edge_softmax(g, s, want_stats=True)[0]
        gt.check("edge_softmax")
        gnn.edge_softmax_backward(g, a, s)
        gt.check("edge_softmax_backward")
    # pooling: 40 graphs of uneven sizes, one of them empty
    sizes = np.array([0, 1, 37] + [int(x) for x in np.random.default_rng(2).integers(5, 60, 37)])
    gptr = to_dev(np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64))
    nn = int(sizes.sum())
    for dtype, F in [("f32", 128), ("bf16", 40)]:
        X = to_dev(synth.normal((nn, F), dtype, 15))
        for op in ("sum", "mean", "max"):
            r = gnn.reduce_nodes(gptr, X, op)
            gt.check(f"reduce_nodes {op}")
            out, arg = r if op == "max" else (r, None)
            gnn.reduce_nodes_backward(gptr, out, nn, op, argmax=arg)
            gt.check(f"reduce_nodes_backward {op}")
    ids = to_dev(np.repeat(np.arange(len(sizes)), sizes).astype(np.int32))
    gnn.graph_ptr_from_ids(ids, len(sizes))
    gt.check("graph_ptr_from_ids")
    # attention
    for dtype, H, C in [("bf16", 8, 32), ("f32", 4, 16), ("f32", 1, 64), ("bf16", 32, 8)]:
        Wx = to_dev(synth.normal((n, H * C), dtype, 16))
        a_s, a_d = to_dev(synth.normal_f32((H, C), 17)), to_dev(synth.normal_f32((H, C), 18))
        fwd = gnn.gat_fused(g, Wx, a_s, a_d, H)
        gt.check(f"gat_fused H={H} C={C} {dtype}")
        gnn.gat_fused_backward(g, Wx, a_s, a_d, fwd, Wx, H)
        gt.check(f"gat_fused_backward H={H} C={C} {dtype}")
    # dense transform: tensor-core shapes, ragged row counts, the FFMA fallback shapes
    for dt, N, K, M in [(torch.bfloat16, 1000, 128, 128), (torch.bfloat16, 4097, 256, 256), (torch.float32, 777, 128, 128),
                        (torch.float32, 2000, 64, 64), (torch.float32, 130, 20, 36), (torch.bfloat16, 515, 64, 256), (torch.float32, 300, 512, 128)]:
        X = torch.randn(N, K, device="cuda").to(dt)
        W = torch.randn(K, M, device="cuda").to(dt)
        dY = torch.randn(N, M, device="cuda").to(dt)
        gnn.linear(X, W)
        gt.check(f"linear {N}x{K}x{M}")
        gnn.linear_backward(X, W, dY)
        gt.check(f"linear_backward {N}x{K}x{M}")
    gnn.axpby(0.5, X, 2.0, X)
    gt.check("axpby")


def test_new_messages_merged_graphs_and_fused_transform_stay_inside_their_buffers(guarded):
    import torch
    gnn, gt = guarded
    n, e = 1500, 30_000
    src, dst = graph(n, e, 21, hub=5000)
    g = gnn.coo_to_csr(n, to_dev(src), to_dev(dst))
    gt.check("coo_to_csr")
    for dtype, F, H in [("f32", 64, 4), ("bf16", 128, 8), ("bf16", 1024, 4), ("f32", 260, 1)]:
        X = to_dev(synth.normal((n, F), dtype, 22))
        R = to_dev(synth.normal((n, F), dtype, 23))
        bias = to_dev(synth.uniform_f32((F,), -1.0, 1.0, 24))
        for op in ("sum", "mean", "max", "min"):
            r = gnn.propagate_msg(g, gnn.XI_SUB_XJ, X, Xi=R, op=op, epi=dict(bias=bias, relu=True))
            gt.check(f"x_i - x_j {op} F={F} {dtype}")
            arg = r[1] if op in ("max", "min") else None
            gnn.propagate_msg_backward(g, gnn.XI_SUB_XJ, R, op=op, argmax=arg, want_dXi=True,
                                       self_grad=dict(Xself=R, self_coef=1.0, self_mode=gnn.SELF_IF_NONEMPTY))
            gt.check(f"x_i - x_j backward {op} F={F} {dtype}")
        widths = [F] if H == 1 else [H, F]
        for ew in widths:
            ef = to_dev(synth.uniform_f32((e, ew), -1.0, 1.0, 25))
            gnn.propagate_msg(g, gnn.E_MUL_XJ, X, e_csr=ef, op="mean")
            gt.check(f"edge factors width {ew}")
            gnn.propagate_msg_backward(g, gnn.E_MUL_XJ, R, op="mean", Xj=X, e_csrT=ef, want_de=True)
            gt.check(f"edge factors backward width {ew}")
        Y = gnn.gin(g, X, 0.5)
        gt.check("gin")
        gnn.gin_backward(g, R, 0.5, X=X, want_deps=True)
        gt.check("gin_backward")
        gnn.row_epilogue_backward(Y, R, relu=True)
        gt.check("row_epilogue_backward")
        if F <= 512:
            s = gnn.edge_dot(g, X, R, H)
            gt.check("edge_dot")
            gnn.edge_dot_backward(g, X, R, s, H)
            gt.check("edge_dot_backward")
    # merged multi-relation graph
    a = (to_dev(src[:9000] % 500), to_dev(dst[:9000] % 600), 0, 0)
    b = (to_dev(src[9000:] % 800), to_dev(dst[9000:] % 600), 500, 0)
    ms, md, seg = gnn.merge_edge_lists([a, b])
    gt.check("merge_edge_lists")
    gm = gnn.coo_to_csr(1300, ms, md)
    seg_csr = gnn.permute_edge_data(gm.eid[:gm.E], seg)
    coef, coefT = gnn.segment_coef(gm, seg_csr, torch.tensor([1, 0], dtype=torch.int32, device="cuda"))
    gt.check("segment_coef")
    # aggregate -> transform fusion and the dense transform with its tail
    for dt, K, M in [(torch.bfloat16, 128, 128), (torch.bfloat16, 256, 256), (torch.float32, 64, 64), (torch.float32, 128, 128),
                     (torch.float32, 256, 64), (torch.bfloat16, 48, 80)]:
        X = torch.randn(n, K, device="cuda").to(dt)
        W = torch.randn(K, M, device="cuda").to(dt)
        dY = torch.randn(n, M, device="cuda").to(dt)
        bias = torch.randn(M, device="cuda")
        gnn.propagate_linear(g, X, W, op="mean", bias=bias, relu=True)
        gt.check(f"propagate_linear {K}x{M}")
        gnn.propagate_linear_backward(g, dY, X, W, op="mean", want_dW=False)
        gt.check(f"propagate_linear_backward dX {K}x{M}")
        gnn.propagate_linear_backward(g, dY, X, W, op="mean")
        gt.check(f"propagate_linear_backward dX+dW {K}x{M}")
        gnn.linear_bias_act(X, W, bias, relu=True)
        gt.check(f"linear_bias_act {K}x{M}")
