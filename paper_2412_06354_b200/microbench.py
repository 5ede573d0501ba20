"""Device times of single library calls on the four smaller synthetic workloads.

    python -m paper_2412_06354_b200.microbench [linear] [propagate] [gat] [large] [--plain]

Each call is captured 20 times into one CUDA graph; the reported time is the replay time divided by 20
(CUDA events on the capturing stream), so launch gaps of the Python binding are not in it.  With
--plain every call runs three times without graph capture (for a profiler) and nothing is timed.
The large-graph sweep is bench.py's job; `large` (not run by default) adds the edge-weight gradient on that graph.
"""
from __future__ import annotations

import sys

import numpy as np
import torch

from . import gnn, synth

REPS = 20


def to_dev(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:  # bf16 bit patterns
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def device_time_us(f, plain):
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for _ in range(3):
            f()
        torch.cuda.synchronize()
        if plain:
            return float("nan")
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=s):
            for _ in range(REPS):
                f()
        gr.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s)
        gr.replay()
        b.record(s)
        torch.cuda.synchronize()
    return a.elapsed_time(b) / REPS * 1e3


def row(name, us, nbytes=None):
    extra = f"  {nbytes / us / 1e3:7.0f} GB/s of algorithmic bytes" if nbytes and us == us else ""
    print(f"{name:<64s} {us:9.1f} us{extra}", flush=True)


def bench_linear(plain):
    lib = gnn.load()
    for n, K, M, dt in [(100_000, 256, 256, torch.bfloat16), (170_000, 128, 128, torch.bfloat16), (170_000, 128, 128, torch.float32),
                        (12_729, 128, 128, torch.float32), (2_000, 64, 64, torch.float32)]:
        g = torch.Generator(device="cuda").manual_seed(n + K)
        X = torch.randn(n, K, device="cuda", generator=g).to(dt)
        W = (torch.randn(K, M, device="cuda", generator=g) * (2.0 / (K + M)) ** 0.5).to(dt)
        dY = torch.randn(n, M, device="cuda", generator=g).to(dt)
        ws = torch.empty(lib.gnn_linear_workspace(n, K, M), dtype=torch.uint8, device="cuda")
        s = X.element_size()
        tag = f"linear {n}x{K}x{M} {'bf16' if dt == torch.bfloat16 else 'f32'}"
        row(tag + " Y = X*W", device_time_us(lambda: gnn.linear(X, W, ws=ws), plain), (n * K + K * M + n * M) * s)
        row(tag + " dX = dY*W^T", device_time_us(lambda: gnn.linear_backward(X, W, dY, want_dW=False, ws=ws), plain), (n * K + K * M + n * M) * s)
        row(tag + " dW = X^T*dY", device_time_us(lambda: gnn.linear_backward(X, W, dY, want_dX=False, ws=ws), plain), (n * K + n * M) * s + K * M * s)


def bench_propagate(plain):
    wl = synth.workload_gcn_small()
    src, dst = synth.with_self_loops(wl["N"], wl["src"], wl["dst"])
    g = gnn.coo_to_csr(wl["N"], to_dev(src), to_dev(dst))
    _, coef, _ = gnn.gcn_norm(g)
    X = to_dev(wl["X"])
    row("config 1 (N=2000, E=12000, F=64 f32) propagate e_mul_xj+sum", device_time_us(lambda: gnn.propagate_fused(g, X, coef, "sum"), plain))
    wl = synth.workload_batched()
    g = gnn.coo_to_csr(wl["N"], to_dev(wl["src"]), to_dev(wl["dst"]))
    X = to_dev(wl["X"])
    row(f"config 2 (512 graphs, N={wl['N']}, F=128 f32) propagate copy_xj+mean", device_time_us(lambda: gnn.propagate_fused(g, X, None, "mean"), plain))
    gptr = to_dev(wl["graph_ptr"].astype(np.int64))
    row("config 2 reduce_nodes mean", device_time_us(lambda: gnn.reduce_nodes(gptr, X, "mean"), plain))
    for dtype in ("bf16", "f32"):
        wl = synth.workload_powerlaw(dtype=dtype)
        g = gnn.coo_to_csr(wl["N"], to_dev(wl["src"]), to_dev(wl["dst"]))
        X = to_dev(wl["X"])
        dO = X.clone()
        tag = f"config 3 (N=170000, E={g.E}, F=128 {dtype}) propagate "
        row(tag + "copy_xj+mean", device_time_us(lambda: gnn.propagate_fused(g, X, None, "mean"), plain))
        out, arg = gnn.propagate_fused(g, X, None, "max")
        row(tag + "copy_xj+max (+argmax)", device_time_us(lambda: gnn.propagate_fused(g, X, None, "max", out=out, argmax=arg), plain))
        m = gnn.apply_edges(g, gnn.COPY_XJ, X)  # the E x F message tensor that the fused call never forms
        row(tag + "UNFUSED apply_edges(copy_xj) + aggregate(mean)",
            device_time_us(lambda: gnn.aggregate(g, gnn.apply_edges(g, gnn.COPY_XJ, X), "mean"), plain))
        del m
        row(tag + "backward of mean", device_time_us(lambda: gnn.propagate_fused_backward(g, dO, "mean"), plain))
        row(tag + "backward of max", device_time_us(lambda: gnn.propagate_fused_backward(g, dO, "max", argmax=arg), plain))


def bench_gat(plain):
    wl = synth.workload_attention()
    g = gnn.coo_to_csr(wl["N"], to_dev(wl["src"]), to_dev(wl["dst"]))
    Wx, a_s, a_d = to_dev(wl["Wx"]), to_dev(wl["a_src"]), to_dev(wl["a_dst"])
    H = wl["H"]
    fwd = gnn.gat_fused(g, Wx, a_s, a_d, H)
    row("config 4 (N=100000, E=1.6M, 8x32 bf16) gat_fused forward", device_time_us(lambda: gnn.gat_fused(g, Wx, a_s, a_d, H), plain))
    row("config 4 gat_fused backward", device_time_us(lambda: gnn.gat_fused_backward(g, Wx, a_s, a_d, fwd, Wx, H), plain))


def bench_large(plain):
    """Edge-weight gradient (one dot product per edge) on the large power-law graph, beside the dX pass."""
    wl = synth.workload_large_graph()
    g = gnn.coo_to_csr(wl["N"], to_dev(wl["src"]), to_dev(wl["dst"]))
    n, E = wl["N"], g.E
    del wl
    for F, dt in [(32, torch.bfloat16), (128, torch.bfloat16), (128, torch.float32), (512, torch.float32)]:
        gen = torch.Generator(device="cuda").manual_seed(F)
        X = torch.randn(n, F, device="cuda", generator=gen).to(dt)
        R = torch.randn(n, F, device="cuda", generator=gen).to(dt)
        dW = torch.empty(E, dtype=torch.float32, device="cuda")
        dX = torch.empty_like(X)
        ws = torch.empty(gnn.propagate_fused_workspace(E, F, "sum"), dtype=torch.uint8, device="cuda")
        tag = f"large graph (N={n}, E={E}) F={F} {'bf16' if dt == torch.bfloat16 else 'f32'} backward of sum: "
        row(tag + "dX", device_time_us(lambda: gnn.propagate_fused_backward(g, R, "sum", dX=dX, ws=ws), plain))
        row(tag + "edge-weight gradient", device_time_us(lambda: gnn.propagate_fused_backward(g, R, "sum", X=X, want_dX=False, want_dW=True, dW=dW, ws=ws), plain))
        del X, R, dW, dX, ws


def main(argv):
    plain = "--plain" in argv
    which = [a for a in argv if not a.startswith("--")] or ["linear", "propagate", "gat"]
    gnn.load()
    table = {"linear": bench_linear, "propagate": bench_propagate, "gat": bench_gat, "large": bench_large}
    for w in which:
        table[w](plain)


if __name__ == "__main__":
    main(sys.argv[1:])
