"""GPU parity: fused GAT core, forward and backward, against the CPU checker."""
import numpy as np
import pytest

import oracle
from paper_2412_06354_b200 import synth
from util import assert_close, to_dev, to_host64
from test_gpu_propagate import build_graph, ragged_graph

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gnn():
    from paper_2412_06354_b200 import gnn as g
    g.load()
    return g


def run_case(gnn, n, src, dst, Wx, a_s, a_d, H, C, dtype, what):
    F = H * C
    g = build_graph(gnn, n, src, dst)
    eid = g.eid[:g.E].cpu().numpy() if g.E else np.zeros(0, np.int64)
    fwd = gnn.gat_fused(g, to_dev(Wx), to_dev(a_s), to_dev(a_d), H)
    ref = oracle.gat(n, src, dst, Wx, a_s, a_d, H, C)
    x64 = synth.to_f64(Wx).reshape(n, H, C)
    Sal = np.einsum("nhc,hc->nh", np.abs(x64), np.abs(a_s.astype(np.float64)))
    Sar = np.einsum("nhc,hc->nh", np.abs(x64), np.abs(a_d.astype(np.float64)))
    assert_close(to_host64(fwd["al"]), ref["al"], Sal, "f32", what + " al")
    assert_close(to_host64(fwd["ar"]), ref["ar"], Sar, "f32", what + " ar")
    if g.E:
        # a coefficient moves by about (error of its logit) * alpha; the logit is a two-dot-product sum
        scale = ref["alpha"][eid] * np.maximum(1.0, Sal[src[eid]] + Sar[dst[eid]])
        assert_close(to_host64(fwd["alpha"]), ref["alpha"][eid], scale, "f32", what + " alpha")
    assert_close(to_host64(fwd["out"]), ref["out"], ref["S"], dtype, what + " out")

    R = synth.normal((n, F), dtype, 4242, 3)
    bw = gnn.gat_fused_backward(g, to_dev(Wx), to_dev(a_s), to_dev(a_d), fwd, to_dev(R), H)
    rb = oracle.gat_backward(n, src, dst, Wx, a_s, a_d, H, C, ref, R)
    # LeakyReLU'(z) is decided by the sign of z.  Where |z| is below the fp32 resolution of its terms the
    # two precisions may decide differently: such an edge moves dz[k,h] by at most |ds[k,h]|*(1-slope), which
    # reaches dal[src], dar[dst] and, through them, three outputs.  The allowance is accumulated from the
    # checker's own intermediates and added to the bound of exactly the elements it can reach.
    slope = 0.2
    z = ref["al"][src] + ref["ar"][dst]
    risky = np.abs(z) < 2e-6 * (Sal[src] + Sar[dst])
    assert risky.mean() < 0.01, risky.mean()
    r64 = synth.to_f64(R).reshape(n, H, C)
    dalpha = np.empty((len(src), H))
    for h in range(H):
        dalpha[:, h] = (r64[dst, h, :] * x64[src, h, :]).sum(axis=1)
    ds, _ = oracle.edge_softmax_backward(n, dst, ref["alpha"], dalpha) if len(src) else (np.zeros((0, H)), None)
    slack = np.where(risky, np.abs(ds) * (1.0 - slope), 0.0)
    sl_al, sl_ar = np.zeros((n, H)), np.zeros((n, H))
    for h in range(H):
        sl_al[:, h] = np.bincount(src, weights=slack[:, h], minlength=n)
        sl_ar[:, h] = np.bincount(dst, weights=slack[:, h], minlength=n)
    as64, ad64 = np.abs(a_s.astype(np.float64)), np.abs(a_d.astype(np.float64))
    extra_dWx = (sl_al[:, :, None] * as64[None] + sl_ar[:, :, None] * ad64[None]).reshape(n, F)
    extra_src = np.einsum("nh,nhc->hc", sl_al, np.abs(x64))
    extra_dst = np.einsum("nh,nhc->hc", sl_ar, np.abs(x64))
    assert_close(to_host64(bw["dWx"]), rb["dWx"], rb["SdWx"], dtype, what + " dWx", extra=extra_dWx)
    assert_close(to_host64(bw["da_src"]), rb["da_src"], rb["Sda_src"], "f32", what + " da_src", extra=extra_src)
    assert_close(to_host64(bw["da_dst"]), rb["da_dst"], rb["Sda_dst"], "f32", what + " da_dst", extra=extra_dst)
    return g, fwd


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("H,C", [(4, 16), (8, 32), (1, 64), (2, 8), (16, 8), (32, 8), (8, 64)])
def test_gat_ragged(gnn, dtype, H, C):
    n, src, dst = ragged_graph(90 + H)
    Wx = synth.normal((n, H * C), dtype, 900 + H, 1)
    a = (6.0 / (C + 1)) ** 0.5
    a_s = synth.uniform_f32((H, C), -a, a, 901, 1)
    a_d = synth.uniform_f32((H, C), -a, a, 902, 1)
    run_case(gnn, n, src, dst, Wx, a_s, a_d, H, C, dtype, f"gat H={H} C={C} {dtype}")


@pytest.mark.parametrize("H,C", [(1, 64), (2, 16)])
def test_gat_one_and_two_heads_with_source_hubs(gnn, H, C):
    """Sources with 5000 and 1025 outgoing edges: the per-source sum of the logit gradients takes the
    block-per-row path (one and two heads do not go through the chunked reduction)."""
    n, src, dst = ragged_graph(97 + H)
    src = src.copy()
    src[100:5100] = 11
    src[6000:7025] = 1499
    Wx = synth.normal((n, H * C), "f32", 960 + H, 1)
    a = (6.0 / (C + 1)) ** 0.5
    a_s = synth.uniform_f32((H, C), -a, a, 961, 1)
    a_d = synth.uniform_f32((H, C), -a, a, 962, 1)
    run_case(gnn, n, src, dst, Wx, a_s, a_d, H, C, "f32", f"gat source hubs H={H}")


def test_gat_zero_attention_is_mean_aggregation(gnn):
    n, src, dst = ragged_graph(95)
    H, C = 4, 16
    Wx = synth.normal_f32((n, H * C), 950)
    zero = np.zeros((H, C), np.float32)
    g = build_graph(gnn, n, src, dst)
    fwd = gnn.gat_fused(g, to_dev(Wx), to_dev(zero), to_dev(zero), H)
    o, S, _ = oracle.propagate("mean", n, src, dst, Wx)
    assert_close(to_host64(fwd["out"]), o, S, "f32", "alpha = 1/deg")


def test_gat_degenerate(gnn):
    import torch
    H, C = 2, 8
    a_s = to_dev(synth.normal_f32((H, C), 1))
    g = build_graph(gnn, 4, np.zeros(0, np.int32), np.zeros(0, np.int32))
    Wx = to_dev(synth.normal_f32((4, H * C), 2))
    fwd = gnn.gat_fused(g, Wx, a_s, a_s, H)
    assert torch.count_nonzero(fwd["out"]) == 0
    bw = gnn.gat_fused_backward(g, Wx, a_s, a_s, fwd, Wx, H)
    assert torch.count_nonzero(bw["dWx"]) == 0 and torch.count_nonzero(bw["da_src"]) == 0
    with pytest.raises(gnn.GnnError) as e:  # three heads
        gnn.gat_fused(g, to_dev(synth.normal_f32((4, 24), 3)), a_s, a_s, 3)
    assert e.value.status == 5
    # a head of 24 bf16 values (three 16-byte chunks) is refused by the forward and the backward call alike
    Wx3 = to_dev(synth.normal_bf16((4, 48), 4))
    a3 = to_dev(synth.normal_f32((2, 24), 5))
    with pytest.raises(gnn.GnnError) as e:
        gnn.gat_fused(g, Wx3, a3, a3, 2)
    assert e.value.status == 5


def test_gat_attention_workload_full_size(gnn):
    """R-MAT N=100000, 1.6M directed edges, 8 heads x 32 features bf16."""
    wl = synth.workload_attention()
    oracle.set_threads(8)
    try:
        run_case(gnn, wl["N"], wl["src"], wl["dst"], wl["Wx"], wl["a_src"], wl["a_dst"], wl["H"], wl["C"], "bf16", "attention workload")
    finally:
        oracle.set_threads(1)


@pytest.mark.parametrize("E", [8_400_000, 17_000_000])
def test_gat_more_than_8mi_edges_uses_the_row_walking_kernels(gnn, E):
    """8.4 M edges: above the size where the per-head gather, its transposed form (with the permuted
    coefficients) and the per-head dot products switch from the position-first kernels to the row-walking ones.
    17 M edges: more than 16384 chunks, so the hub rows (cut into more than 64 chunks) are finished by the
    block-per-row fix-up, here with the per-head multipliers and the rank-1 row epilogue of the backward pass."""
    n, H, C = 200_000, 4, 8
    src, dst = synth.rmat(18, n, E, 4321, symmetric=False)
    Wx = synth.normal_f32((n, H * C), 4322)
    a = (6.0 / (C + 1)) ** 0.5
    a_s = synth.uniform_f32((H, C), -a, a, 4323)
    a_d = synth.uniform_f32((H, C), -a, a, 4324)
    oracle.set_threads(8)
    try:
        g, _ = run_case(gnn, n, src, dst, Wx, a_s, a_d, H, C, "f32", "gat %.1fM edges" % (E / 1e6))
        if E > 16_000_000:
            assert int(np.diff(g.rowptr.cpu().numpy()).max()) > 65 * 1024 and int(np.diff(g.rowptrT.cpu().numpy()).max()) > 65 * 1024
    finally:
        oracle.set_threads(1)
