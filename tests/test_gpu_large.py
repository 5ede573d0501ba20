"""Full-size parity on the large power-law graph (N = 2.4 M, E = 123 M), in the launch configuration the
benchmark times: CSR conversion bit for bit, and fused propagate forward/backward on sampled output rows
(a seeded 2000-row sample plus the 50 longest rows, which span hundreds of chunks) that the CPU checker
computes one by one."""
import os

import numpy as np
import pytest

import oracle
from paper_2412_06354_b200 import synth
from util import assert_close, to_dev, to_host64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def big():
    import torch
    from paper_2412_06354_b200 import gnn
    gnn.load()
    wl = synth.workload_large_graph()
    g = gnn.coo_to_csr(wl["N"], torch.from_numpy(wl["src"]).cuda(), torch.from_numpy(wl["dst"]).cuda())
    oracle.set_threads(len(os.sched_getaffinity(0)))
    yield gnn, wl, g
    oracle.set_threads(1)


def sample_rows(deg, seed, k=2000, top=50):
    rng = np.random.default_rng(seed)
    rows = np.union1d(rng.choice(len(deg), k, replace=False), np.argsort(deg)[-top:])
    return rows.astype(np.int64)


def test_csr_bit_exact_full_size(big):
    gnn, wl, g = big
    n, src, dst = wl["N"], wl["src"], wl["dst"]
    rowptr, col, eid = oracle.coo_to_csr(n, dst, src)
    assert np.array_equal(g.rowptr.cpu().numpy(), rowptr)
    assert np.array_equal(g.col.cpu().numpy(), col) and np.array_equal(g.eid.cpu().numpy(), eid)
    rowptrT, colT, eidT = oracle.coo_to_csr(n, src, dst)
    assert np.array_equal(g.rowptrT.cpu().numpy(), rowptrT)
    assert np.array_equal(g.colT.cpu().numpy(), colT) and np.array_equal(g.eidT.cpu().numpy(), eidT)
    assert np.array_equal(g.t2f.cpu().numpy(), oracle.t2f(eid, eidT))


@pytest.mark.parametrize("dtype,F", [("bf16", 128), ("f32", 32), ("f32", 512), ("bf16", 512), ("f32", 256), ("bf16", 64), ("bf16", 256)])
def test_propagate_sampled_rows_full_size(big, dtype, F):
    """Every launch shape the benchmark times at this size: narrow and 512-byte rows on the row-walking kernel,
    and the column-slab passes (two for 1024-byte rows: bf16 F=512, f32 F=256; four for f32 F=512)."""
    import torch
    gnn, wl, g = big
    n, src, dst, w, seed = wl["N"], wl["src"], wl["dst"], wl["w"], wl["seed"]
    X32 = synth.normal_f32((n, F), seed, 20)
    R32 = synth.normal_f32((n, F), seed, 21)
    if dtype == "bf16":
        Xd, Rd = torch.from_numpy(X32).cuda().to(torch.bfloat16), torch.from_numpy(R32).cuda().to(torch.bfloat16)
        X = Xd.view(torch.int16).cpu().numpy().view(np.uint16)   # the bits the device holds (RNE of the fp32 draw)
        R = Rd.view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(X[:1000], synth.normal_bf16((n, F), seed, 20)[:1000])
    else:
        Xd, Rd, X, R = torch.from_numpy(X32).cuda(), torch.from_numpy(R32).cuda(), X32, R32
    w_csr = gnn.permute_edge_data(g.eid, torch.from_numpy(w).cuda())
    w_csrT = gnn.permute_edge_data(g.t2f, w_csr)
    deg_in = np.bincount(dst, minlength=n)
    rows = sample_rows(deg_in, 7)
    out = gnn.propagate_fused(g, Xd, w_csr, "sum")
    o, S, _ = oracle.propagate("sum", n, src, dst, X, w, rows=rows)
    assert_close(to_host64(out[torch.from_numpy(rows).cuda()]), o, S, dtype, f"forward F={F} {dtype}")
    out_c = gnn.propagate_fused(g, Xd, None, "sum")
    o, S, _ = oracle.propagate("sum", n, src, dst, X, None, rows=rows)
    assert_close(to_host64(out_c[torch.from_numpy(rows).cuda()]), o, S, dtype, f"forward copy_xj F={F} {dtype}")
    dX, _ = gnn.propagate_fused_backward(g, Rd, "sum", w_csrT=w_csrT)
    rows_s = sample_rows(np.bincount(src, minlength=n), 8)
    bw = oracle.propagate_backward("sum", n, src, dst, None, w, R, rows=rows_s)
    assert_close(to_host64(dX[torch.from_numpy(rows_s).cuda()]), bw["dX"], bw["SdX"], dtype, f"backward F={F} {dtype}")
    # properties that hold at any size: isolated targets get exact zeros; column sums match a direct sum
    iso = torch.from_numpy(np.nonzero(deg_in == 0)[0][:5000]).cuda()
    assert torch.count_nonzero(out[iso]) == 0


def test_mean_max_and_backward_of_max_full_size(big):
    """The row-walking kernel's other modes at a size where it (not the position-first kernel) runs:
    mean on sampled rows, max with winner positions on every row (bit-exact), routing backward on sampled rows."""
    import torch
    from util import bits, f64_to_dtype_bits
    gnn, wl, g = big
    n, src, dst, seed = wl["N"], wl["src"], wl["dst"], wl["seed"]
    F = 32
    X = synth.normal_f32((n, F), seed, 22)
    R = synth.normal_f32((n, F), seed, 23)
    Xd, Rd = torch.from_numpy(X).cuda(), torch.from_numpy(R).cuda()
    rows = sample_rows(np.bincount(dst, minlength=n), 9)
    out = gnn.propagate_fused(g, Xd, None, "mean")
    o, S, _ = oracle.propagate("mean", n, src, dst, X, None, rows=rows)
    assert_close(to_host64(out[torch.from_numpy(rows).cuda()]), o, S, "f32", "mean")
    out, arg = gnn.propagate_fused(g, Xd, None, "max")
    o, _, a = oracle.propagate("max", n, src, dst, X)
    assert np.array_equal(bits(out), f64_to_dtype_bits(o, "f32"))
    del o
    eid = g.eid.cpu().numpy()
    ga = arg.cpu().numpy()
    assert np.array_equal(np.where(ga >= 0, eid[np.maximum(ga, 0)], -1), a)
    del eid, ga
    dX, _ = gnn.propagate_fused_backward(g, Rd, "max", argmax=arg)
    rows_s = sample_rows(np.bincount(src, minlength=n), 10)
    bw = oracle.propagate_backward("max", n, src, dst, X, None, R, arg=a, rows=rows_s)
    assert_close(to_host64(dX[torch.from_numpy(rows_s).cuda()]), bw["dX"], bw["SdX"], "f32", "backward of max")


def test_edge_weight_gradient_full_size(big):
    """One dot product per edge on all 123 M edges (F = 32, fp32), against the CPU checker."""
    import torch
    gnn, wl, g = big
    n, src, dst, seed = wl["N"], wl["src"], wl["dst"], wl["seed"]
    F = 32
    X = synth.normal_f32((n, F), seed, 24)
    R = synth.normal_f32((n, F), seed, 25)
    _, dW = gnn.propagate_fused_backward(g, torch.from_numpy(R).cuda(), "sum", X=torch.from_numpy(X).cuda(), want_dX=False, want_dW=True)
    bw = oracle.propagate_backward("sum", n, src, dst, X, np.ones(len(src), np.float32), R, want_dX=False, want_dw=True)
    eid = g.eid.cpu().numpy()
    assert_close(to_host64(dW), bw["dw"][eid], bw["Sdw"][eid], "f32", "edge-weight gradient, all edges")
