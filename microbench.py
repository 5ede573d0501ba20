"""Device times of single library calls on the four smaller synthetic workloads.

    python microbench.py [linear] [fused] [config1] [config2] [config3] [config4] [large] [--plain] [--flush]

Each call is captured 20 times into one CUDA graph; the reported time is the replay time divided by 20
(CUDA events on the capturing stream), so launch gaps of the Python binding are not in it and the inputs
are warm in L2.  With --flush a second column times every call alone (CUDA events around the call) after a
256 MB buffer has been overwritten, i.e. with its inputs coming from HBM; the median of 20 is reported.
With --plain every call runs three times without graph capture (for a profiler) and nothing is timed.
`bench.py --config K` prints the same measurements as one JSON line.
The large-graph sweep is bench.py's job; `large` (not run by default) adds the edge-weight gradient on that graph.
"""
from __future__ import annotations

import os
import statistics
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

from paper_2412_06354_b200 import gnn, synth

REPS = 20
FLUSH_BYTES = 256 << 20  # twice the L2


def to_dev(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:  # bf16 bit patterns
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def device_time_us(f, plain=False):
    """Warm time: 20 calls replayed as one CUDA graph."""
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


_flush_buf = None


def flushed_time_us(f):
    """Cold time: the call alone, after 256 MB have been written (L2 holds none of its inputs); median of 20.
    The call is queued while the flush still runs, so no launch gap of the binding falls inside the events."""
    global _flush_buf
    if _flush_buf is None:
        _flush_buf = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    s = torch.cuda.current_stream()
    ts = []
    for i in range(REPS + 3):
        _flush_buf.fill_(i & 0xFF)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(s)
        f()
        b.record(s)
        torch.cuda.synchronize()
        if i >= 3:
            ts.append(a.elapsed_time(b) * 1e3)
    return statistics.median(ts)


# ------------------------------------------------------------------ call lists: (name, callable, algorithmic bytes or None)
def linear_calls(shapes=None):
    lib = gnn.load()
    calls = []
    for n, K, M, dt in shapes or [(100_000, 256, 256, torch.bfloat16), (170_000, 128, 128, torch.bfloat16), (170_000, 128, 128, torch.float32),
                                  (12_729, 128, 128, torch.float32), (2_000, 64, 64, torch.float32)]:
        g = torch.Generator(device="cuda").manual_seed(n + K)
        X = torch.randn(n, K, device="cuda", generator=g).to(dt)
        W = (torch.randn(K, M, device="cuda", generator=g) * (2.0 / (K + M)) ** 0.5).to(dt)
        dY = torch.randn(n, M, device="cuda", generator=g).to(dt)
        ws = torch.empty(lib.gnn_linear_workspace(n, K, M), dtype=torch.uint8, device="cuda")
        s = X.element_size()
        tag = f"linear {n}x{K}x{M} {'bf16' if dt == torch.bfloat16 else 'f32'}"
        calls.append((tag + " Y = X*W", lambda X=X, W=W, ws=ws: gnn.linear(X, W, ws=ws), (n * K + K * M + n * M) * s))
        calls.append((tag + " dX = dY*W^T", lambda X=X, W=W, dY=dY, ws=ws: gnn.linear_backward(X, W, dY, want_dW=False, ws=ws), (n * K + K * M + n * M) * s))
        calls.append((tag + " dW = X^T*dY", lambda X=X, W=W, dY=dY, ws=ws: gnn.linear_backward(X, W, dY, want_dX=False, ws=ws), (n * K + n * M) * s + K * M * s))
    return calls


def config1_calls():
    wl = synth.workload_gcn_small()
    src, dst = synth.with_self_loops(wl["N"], wl["src"], wl["dst"])
    g = gnn.coo_to_csr(wl["N"], to_dev(src), to_dev(dst))
    _, coef, coefT = gnn.gcn_norm(g)
    X = to_dev(wl["X"])
    dO = X.clone()
    tag = f"config 1 (N={wl['N']}, E={g.E} with loops, F=64 f32) "
    calls = [(tag + "propagate e_mul_xj+sum (GCN coefficients)", lambda: gnn.propagate_fused(g, X, coef, "sum"), None),
             (tag + "backward dX", lambda: gnn.propagate_fused_backward(g, dO, "sum", w_csrT=coefT), None)]
    return calls + linear_calls([(wl["N"], 64, 64, torch.float32)])


def config2_calls():
    wl = synth.workload_batched()
    g = gnn.coo_to_csr(wl["N"], to_dev(wl["src"]), to_dev(wl["dst"]))
    X = to_dev(wl["X"])
    gptr = to_dev(wl["graph_ptr"].astype(np.int64))
    pooled = gnn.reduce_nodes(gptr, X, "mean")
    tag = f"config 2 (512 graphs, N={wl['N']}, E={g.E}, F=128 f32) "
    calls = [(tag + "propagate copy_xj+mean", lambda: gnn.propagate_fused(g, X, None, "mean"), None),
             (tag + "backward of mean", lambda: gnn.propagate_fused_backward(g, X, "mean"), None),
             (tag + "reduce_nodes mean", lambda: gnn.reduce_nodes(gptr, X, "mean"), None),
             (tag + "reduce_nodes mean backward", lambda: gnn.reduce_nodes_backward(gptr, pooled, wl["N"], "mean"), None)]
    return calls + linear_calls([(wl["N"], 128, 128, torch.float32)])


def config3_calls():
    calls = []
    for dtype in ("bf16", "f32"):
        wl = synth.workload_powerlaw(dtype=dtype)
        g = gnn.coo_to_csr(wl["N"], to_dev(wl["src"]), to_dev(wl["dst"]))
        X = to_dev(wl["X"])
        dO = X.clone()
        w = torch.rand(g.E, device="cuda")
        tag = f"config 3 (N=170000, E={g.E}, F=128 {dtype}) propagate "
        out, arg = gnn.propagate_fused(g, X, None, "max")
        calls += [
            (tag + "copy_xj+mean", lambda g=g, X=X: gnn.propagate_fused(g, X, None, "mean"), None),
            (tag + "copy_xj+max (+argmax)", lambda g=g, X=X, out=out, arg=arg: gnn.propagate_fused(g, X, None, "max", out=out, argmax=arg), None),
            (tag + "e_mul_xj+sum", lambda g=g, X=X, w=w: gnn.propagate_fused(g, X, w, "sum"), None),
            (tag + "UNFUSED apply_edges(copy_xj) + aggregate(mean)", lambda g=g, X=X: gnn.aggregate(g, gnn.apply_edges(g, gnn.COPY_XJ, X), "mean"), None),
            (tag + "backward of mean", lambda g=g, dO=dO: gnn.propagate_fused_backward(g, dO, "mean"), None),
            (tag + "backward of max", lambda g=g, dO=dO, arg=arg: gnn.propagate_fused_backward(g, dO, "max", argmax=arg), None),
            (tag + "backward of e_mul_xj+sum (dX)", lambda g=g, dO=dO, w=w: gnn.propagate_fused_backward(g, dO, "sum", w_csrT=w), None),
        ]
    return calls + linear_calls([(170_000, 128, 128, torch.bfloat16), (170_000, 128, 128, torch.float32)])


def config4_calls():
    wl = synth.workload_attention()
    g = gnn.coo_to_csr(wl["N"], to_dev(wl["src"]), to_dev(wl["dst"]))
    Wx, a_s, a_d = to_dev(wl["Wx"]), to_dev(wl["a_src"]), to_dev(wl["a_dst"])
    H = wl["H"]
    fwd = gnn.gat_fused(g, Wx, a_s, a_d, H)
    calls = [("config 4 (N=100000, E=1.6M, 8x32 bf16) gat_fused forward", lambda: gnn.gat_fused(g, Wx, a_s, a_d, H), None),
             ("config 4 gat_fused backward", lambda: gnn.gat_fused_backward(g, Wx, a_s, a_d, fwd, Wx, H), None)]
    return calls + linear_calls([(100_000, 256, 256, torch.bfloat16)])


def large_calls():
    """Edge-weight gradient (one dot product per edge) on the large power-law graph, beside the dX pass."""
    wl = synth.workload_large_graph()
    g = gnn.coo_to_csr(wl["N"], to_dev(wl["src"]), to_dev(wl["dst"]))
    n, E = wl["N"], g.E
    del wl
    calls = []
    for F, dt in [(32, torch.bfloat16), (128, torch.bfloat16), (128, torch.float32)]:
        gen = torch.Generator(device="cuda").manual_seed(F)
        X = torch.randn(n, F, device="cuda", generator=gen).to(dt)
        R = torch.randn(n, F, device="cuda", generator=gen).to(dt)
        dW = torch.empty(E, dtype=torch.float32, device="cuda")
        dX = torch.empty_like(X)
        ws = torch.empty(gnn.propagate_fused_workspace(E, F, "sum"), dtype=torch.uint8, device="cuda")
        tag = f"large graph (N={n}, E={E}) F={F} {'bf16' if dt == torch.bfloat16 else 'f32'} backward of sum: "
        calls.append((tag + "dX", lambda R=R, dX=dX, ws=ws: gnn.propagate_fused_backward(g, R, "sum", dX=dX, ws=ws), None))
        calls.append((tag + "edge-weight gradient", lambda R=R, X=X, dW=dW, ws=ws: gnn.propagate_fused_backward(g, R, "sum", X=X, want_dX=False, want_dW=True, dW=dW, ws=ws), None))
    return calls


def gatherloop_calls():
    """The bare gathers of one pass over the large graph (no rows, no output) per row width, beside the sum over
    fp32 rows of the same width."""
    wl = synth.workload_large_graph()
    g = gnn.coo_to_csr(wl["N"], to_dev(wl["src"]), to_dev(wl["dst"]))
    n, E = wl["N"], g.E
    del wl
    calls = []
    sink = torch.empty(gnn.load().gnn_probe_gather_sink_floats(E), dtype=torch.float32, device="cuda")
    for rb in (64, 128, 256, 512):
        gen = torch.Generator(device="cuda").manual_seed(rb)
        X = torch.randn(n, rb // 4, device="cuda", generator=gen)
        out = torch.empty_like(X)
        ws = torch.empty(gnn.propagate_fused_workspace(E, rb // 4, "sum"), dtype=torch.uint8, device="cuda")
        calls.append((f"large graph (N={n}, E={E}) {rb}-byte rows: bare gather loop", lambda X=X, rb=rb: gnn.probe_gather(g.col[:E], X, rb, sink=sink), E * rb))
        calls.append((f"large graph {rb}-byte fp32 rows: propagate copy_xj+sum", lambda X=X, out=out, ws=ws: gnn.propagate_fused(g, X, None, "sum", out=out, ws=ws), E * rb))
    return calls


def fused_calls():
    """Aggregate -> transform: the fused call beside the two calls it replaces (configs 1, 3 and 4 shapes)."""
    lib = gnn.load()
    calls = []
    cases = []
    wl = synth.workload_gcn_small()
    src, dst = synth.with_self_loops(wl["N"], wl["src"], wl["dst"])
    cases.append(("config 1 GCN 64x64 f32", wl["N"], src, dst, to_dev(wl["X"]), 64, True))
    for dtype in ("bf16", "f32"):
        wl = synth.workload_powerlaw(dtype=dtype)
        cases.append((f"config 3 128x128 {dtype}", wl["N"], wl["src"], wl["dst"], to_dev(wl["X"]), 128, False))
    wl = synth.workload_attention()
    cases.append(("config 4 graph 256x256 bf16", wl["N"], wl["src"], wl["dst"], to_dev(wl["Wx"]), 256, False))
    for tag, n, src, dst, X, M, gcn in cases:
        g = gnn.coo_to_csr(n, to_dev(src), to_dev(dst))
        K = X.shape[1]
        gen = torch.Generator(device="cuda").manual_seed(K + M)
        W = (torch.randn(K, M, device="cuda", generator=gen) * (2.0 / (K + M)) ** 0.5).to(X.dtype)
        w = gnn.gcn_norm(g)[1] if gcn else None
        op = "sum" if gcn else "mean"
        wsf = torch.empty(lib.gnn_propagate_linear_workspace(n, g.E, K, M), dtype=torch.uint8, device="cuda")
        wsp = torch.empty(gnn.propagate_fused_workspace(g.E, K, op), dtype=torch.uint8, device="cuda")
        wsl = torch.empty(lib.gnn_linear_workspace(n, K, M), dtype=torch.uint8, device="cuda")
        H = torch.empty_like(X)
        calls.append((f"{tag} (N={n}, E={g.E}) FUSED propagate+linear", lambda g=g, X=X, W=W, w=w, op=op, wsf=wsf: gnn.propagate_linear(g, X, W, w_csr=w, op=op, ws=wsf), None))
        calls.append((f"{tag} propagate, then linear (two calls)",
                      lambda g=g, X=X, W=W, w=w, op=op, H=H, wsp=wsp, wsl=wsl: gnn.linear(gnn.propagate_fused(g, X, w, op, out=H, ws=wsp), W, ws=wsl), None))
        dY = torch.randn(n, M, device="cuda", generator=gen).to(X.dtype)
        calls.append((f"{tag} FUSED backward dX", lambda g=g, X=X, W=W, w=w, op=op, dY=dY, wsf=wsf: gnn.propagate_linear_backward(g, dY, X, W, w_csrT=w, op=op, want_dW=False, ws=wsf), None))
        calls.append((f"{tag} backward dX + dW", lambda g=g, X=X, W=W, w=w, op=op, dY=dY, wsf=wsf: gnn.propagate_linear_backward(g, dY, X, W, w_csrT=w, op=op, ws=wsf), None))
    return calls


TABLE = {"linear": linear_calls, "fused": fused_calls, "config1": config1_calls, "config2": config2_calls, "config3": config3_calls,
         "config4": config4_calls, "large": large_calls, "gatherloop": gatherloop_calls,
         # older names: the propagate calls of configs 1-3 together, the attention calls of config 4
         "propagate": lambda: config1_calls() + config2_calls() + config3_calls(), "gat": config4_calls}


def measure(calls, plain=False, flush=False):
    """-> list of dicts (name, us_warm, us_flushed or None, algorithmic GB/s or None); prints a table row per call."""
    rows = []
    for name, f, nbytes in calls:
        us = device_time_us(f, plain)
        usf = flushed_time_us(f) if flush and not plain else None
        extra = f"  {nbytes / us / 1e3:7.0f} GB/s of algorithmic bytes" if nbytes and us == us else ""
        cold = f"  cold {usf:9.1f} us" if usf is not None else ""
        print(f"{name:<72s} {us:9.1f} us{cold}{extra}", flush=True, file=sys.stderr if measure.to_stderr else sys.stdout)
        rows.append({"call": name, "us_warm": None if us != us else round(us, 2), "us_flushed": None if usf is None else round(usf, 2),
                     "algorithmic_GBs_warm": round(nbytes / us / 1e3, 1) if nbytes and us == us else None})
    return rows


measure.to_stderr = False


def main(argv):
    plain = "--plain" in argv
    flush = "--flush" in argv
    which = [a for a in argv if not a.startswith("--")] or ["linear", "config1", "config2", "config3", "config4"]
    gnn.load()
    for w in which:
        measure(TABLE[w](), plain, flush)


if __name__ == "__main__":
    main(sys.argv[1:])
