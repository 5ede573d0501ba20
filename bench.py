#!/usr/bin/env python
"""Benchmark: fused propagate forward + backward on the large power-law graph.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--cases 128:bf16,...] [--impl reference]

One step = the whole aggregation sweep on a seeded R-MAT graph (N = 2.4 M nodes, E = 123 M
directed edges, randomly relabelled, sorted by target): for every feature width F in
{32, 64, 128, 256, 512} x {bf16, f32} and for both fused messages (copy_xj+sum, e_mul_xj+sum),
one gnn_propagate_fused and one gnn_propagate_fused_backward (dX).  The metric is
edges*features per second: sum over the cases of E*F, divided by the time of the step.

Prints ONE JSON line (rank 0).  `value` is measured with every input resident in HBM; `e2e`
repeats the step through the *_host entry points with pinned host buffers, copying the features
and the incoming gradient to the device and the two results back inside the timed region.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "propagate fwd+bwd edges*feat/s"
UNIT = "edges*feat/s"
ALL_CASES = [(F, dt) for dt in ("bf16", "f32") for F in (32, 64, 128, 256, 512)]
FMAX = 512

# DRAM bytes (read + write, GB) of one gnn_propagate_fused / _backward call (all its propagate_chunk_kernel and
# fix-up launches: wide rows run as 512-byte column slabs), taken with the hardware counters
# dram__bytes_read.sum + dram__bytes_write.sum on a REDUCED graph of the same generator (--graph-scale 20:
# N = 600,000, E = 30,750,000, a quarter of the workload) so that the capture stays small.  The line reports
# these numbers times TRAFFIC_SCALE (the ratio of the edges*features processed).  That is a LOWER bound of the
# full-size traffic: the reduced feature matrix is four times smaller against the same L2, so a larger share of
# its gathers hits (a full-size capture of an earlier build of the same loop gave 79.6 GB where this gives 32.8).
# The numbers belong to the kernel sources whose digest is TRAFFIC_KERNEL_SHA256; with other sources the line
# reports traffic = null.
TRAFFIC_SOURCE = ("ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --clock-control none -k regex:propagate_ over one step of "
                  "`bench.py --graph-scale 20` (N=600000, E=30.75M), scaled by 4.0 = ratio of edges*features; lower bound of the "
                  "full-size traffic (better L2 reuse on the reduced matrix); summary under profiles/")
TRAFFIC_SCALE = 4.0
TRAFFIC_KERNEL_FILES = ("propagate.cu", "propagate.cuh", "common.cuh")
TRAFFIC_KERNEL_SHA256 = "62facf4d2c659f955d3468cd3144d3ed4b685ffbeb12d73cf41affba107fcf9c"
TRAFFIC_GB_REDUCED = {
    "32:bf16:copy_xj:fwd": 0.192,
    "32:bf16:copy_xj:bwd": 0.19,
    "32:bf16:e_mul_xj:fwd": 0.315,
    "32:bf16:e_mul_xj:bwd": 0.315,
    "64:bf16:copy_xj:fwd": 0.269,
    "64:bf16:copy_xj:bwd": 0.27,
    "64:bf16:e_mul_xj:fwd": 0.395,
    "64:bf16:e_mul_xj:bwd": 0.395,
    "128:bf16:copy_xj:fwd": 0.61,
    "128:bf16:copy_xj:bwd": 0.61,
    "128:bf16:e_mul_xj:fwd": 0.737,
    "128:bf16:e_mul_xj:bwd": 0.737,
    "256:bf16:copy_xj:fwd": 2.004,
    "256:bf16:copy_xj:bwd": 2.004,
    "256:bf16:e_mul_xj:fwd": 2.133,
    "256:bf16:e_mul_xj:bwd": 2.133,
    "512:bf16:copy_xj:fwd": 4.018,
    "512:bf16:copy_xj:bwd": 4.021,
    "512:bf16:e_mul_xj:fwd": 4.277,
    "512:bf16:e_mul_xj:bwd": 4.281,
    "32:f32:copy_xj:fwd": 0.257,
    "32:f32:copy_xj:bwd": 0.258,
    "32:f32:e_mul_xj:fwd": 0.381,
    "32:f32:e_mul_xj:bwd": 0.382,
    "64:f32:copy_xj:fwd": 0.579,
    "64:f32:copy_xj:bwd": 0.58,
    "64:f32:e_mul_xj:fwd": 0.706,
    "64:f32:e_mul_xj:bwd": 0.706,
    "128:f32:copy_xj:fwd": 1.918,
    "128:f32:copy_xj:bwd": 1.917,
    "128:f32:e_mul_xj:fwd": 2.047,
    "128:f32:e_mul_xj:bwd": 2.044,
    "256:f32:copy_xj:fwd": 3.848,
    "256:f32:copy_xj:bwd": 3.843,
    "256:f32:e_mul_xj:fwd": 4.107,
    "256:f32:e_mul_xj:bwd": 4.103,
    "512:f32:copy_xj:fwd": 7.685,
    "512:f32:copy_xj:bwd": 7.68,
    "512:f32:e_mul_xj:fwd": 8.199,
    "512:f32:e_mul_xj:bwd": 8.198,
}
TRAFFIC_GB = {k: v * TRAFFIC_SCALE for k, v in TRAFFIC_GB_REDUCED.items()}


def parse_cases(s):
    if not s or s == "sweep":
        return ALL_CASES
    out = []
    for tok in s.split(","):
        f, dt = tok.split(":")
        out.append((int(f), dt))
    return out


def kernel_sources_digest():
    """sha256 over the sources of the propagate kernels, in the order of TRAFFIC_KERNEL_FILES."""
    import hashlib
    h = hashlib.sha256()
    for f in TRAFFIC_KERNEL_FILES:
        with open(os.path.join(ROOT, "paper_2412_06354_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (earlier pool measurement, MEASURED_PEAKS.json absent)"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.t.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def compulsory_bytes(N, E, F, s, weighted):
    """Every array touched once: index (+weight) stream, row pointers, X read once, out written once."""
    return 4 * E + (4 * E if weighted else 0) + 8 * N + 2 * N * F * s


def gather_bytes(N, E, F, s, weighted):
    """No reuse at all: every edge fetches its source row."""
    return 4 * E + (4 * E if weighted else 0) + 8 * N + (E + N) * F * s


# ----------------------------------------------------------------------------- reference arm
def run_reference(args, rank):
    """The CPU checker, as it stands, on a bounded sample of the same workload."""
    if rank != 0:
        return
    import oracle
    from paper_2412_06354_b200 import synth
    cores = len(os.sched_getaffinity(0))
    oracle.set_threads(cores)
    sample = cpu_sample(synth)
    times = []
    for i in range(args.warmup + args.steps):
        t = cpu_step(oracle, sample)
        if i >= args.warmup:
            times.append(t)
    ms = 1e3 * sum(times) / len(times)
    val = sample["E"] * sample["F"] / (ms * 1e-3)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": "bounded sample for the CPU checker: " + sample["desc"], "N": sample["N"], "E": sample["E"], "cases": ["%d:bf16" % sample["F"]],
                       "sample_of": WORKLOAD_NAME},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample["desc"]},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


WORKLOAD_NAME = "large sparse aggregation sweep: R-MAT N=2.4M E=123M (a=.57 b=.19 c=.19, symmetrised, relabelled, sorted by dst), F in {32,64,128,256,512} x {bf16,f32}, copy_xj+sum and e_mul_xj+sum, fwd + bwd dX"


def cpu_sample(synth, pairs=16_000_000, F=128, scale=20):
    """A smaller graph of the same family for the CPU checker: R-MAT with the same parameters and
    the same mean degree (N=624,390, 32,000,000 directed edges), bf16 features of width 128: a few
    seconds of work per forward + backward pair on 16 cores."""
    n = 2_400_000 * (2 * pairs) // 123_000_000
    src, dst = synth.rmat(scale, n, pairs, synth.BASE_SEED + 5, symmetric=True, relabel=True, sort_by_dst=True)
    return dict(N=n, E=len(src), F=F, src=src, dst=dst, X=synth.normal_bf16((n, F), synth.BASE_SEED + 5, 20),
                R=synth.normal_bf16((n, F), synth.BASE_SEED + 5, 21), w=synth.uniform_f32((len(src),), 0, 1, synth.BASE_SEED + 5, 13),
                desc=f"same generator at N={n}, E={2 * pairs} (same mean degree), F={F} bf16, e_mul_xj+sum fwd + bwd dX, fp64")


def cpu_step(oracle, s):
    t0 = time.perf_counter()
    oracle.propagate("sum", s["N"], s["src"], s["dst"], s["X"], s["w"])
    oracle.propagate_backward("sum", s["N"], s["src"], s["dst"], s["X"], s["w"], s["R"])
    return time.perf_counter() - t0


def all_max(x, device, world):
    """Max over ranks of a host float (identity when single-process)."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(work_per_rank, ms_per_step_max, world):
    """Replicas only: every rank does the same work; the job's rate is all ranks' work over the slowest rank's time."""
    return world * work_per_rank / (ms_per_step_max * 1e-3)


# ----------------------------------------------------------------------------- smaller workloads
SMALL_WORKLOADS = {
    1: "GCN layer: Erdos-Renyi N=2000, 10000 directed edges + self-loops, F=64 f32, normalised sum",
    2: "batched small graphs: 512 graphs of 10-40 nodes, F=128 f32, mean aggregation + per-graph mean pooling",
    3: "power-law graph: preferential attachment N=170000, m=4, F=128 f32 and bf16, mean / max / normalised sum",
    4: "attention: R-MAT N=100000, 1.6M directed edges, 8 heads x 32 features bf16, fused GAT core",
}


def run_small_config(args, rank, local):
    """Layer-level calls of one of the smaller workloads: per call the warm device time (20 calls replayed as one
    CUDA graph) and the time after an L2 flush (256 MB written before every call, CUDA events, median of 20)."""
    if rank != 0:
        return
    import torch
    import microbench
    from paper_2412_06354_b200 import build, gnn
    build.build()
    gnn.load()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    microbench.measure.to_stderr = True
    sampler = ClockSampler(local)
    sampler.start()
    rows = microbench.measure(microbench.TABLE["config%d" % args.config](), flush=True)
    clocks = sampler.stop()
    line = {"metric": "device time per call", "unit": "us", "value": sum(r["us_warm"] for r in rows), "n_gpus": 1, "higher_is_better": False,
            "data": "synthetic", "config": {"workload": SMALL_WORKLOADS[args.config], "l2": "us_warm: inputs resident in L2 (graph replay); us_flushed: 256 MB written before every call"},
            "value_note": "sum of the warm per-call times", "clocks": clocks, "calls": rows}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- GPU arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200")
    ap.add_argument("--cases", default="sweep")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-lanes", type=int, default=3, help="streams per direction of the end-to-end leg (forward calls alternate over this many, backward calls likewise)")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-dw", action="store_true", help="skip the separate timing of the edge-weight gradient")
    ap.add_argument("--no-probe", action="store_true", help="skip the bare gather loop (the measured L2 -> SM ceiling)")
    ap.add_argument("--config", type=int, default=5, choices=[1, 2, 3, 4, 5],
                    help="5 (default): the large sweep.  1-4: device times of the layer-level calls of the smaller workloads, warm and after an L2 flush")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--natural-ids", action="store_true",
                    help="keep the generator's vertex ids (hubs at low ids) instead of the random relabelling of the headline workload")
    ap.add_argument("--graph-scale", type=int, default=22,
                    help="R-MAT scale; 22 is the full workload, smaller values shrink N and E by powers of two (profiling captures)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        return run_reference(args, rank)
    if args.config != 5:
        return run_small_config(args, rank, local)
    assert args.warmup >= 3 or os.environ.get("GNN_BENCH_ALLOW_SHORT"), "use at least 3 warm-up steps"

    import torch
    from paper_2412_06354_b200 import build, gnn, synth
    build.build()
    gnn.load()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    cases = parse_cases(args.cases)
    fmax = max(F for F, _ in cases)
    # ---- inputs (host, seeded) -> device
    shrink = 22 - args.graph_scale
    assert 0 <= shrink <= 10
    wl = synth.workload_large_graph(n=2_400_000 >> shrink, scale=args.graph_scale, pairs=61_500_000 >> shrink, relabel=not args.natural_ids)
    N, E, seed = wl["N"], len(wl["src"]), wl["seed"]
    src_d, dst_d = torch.from_numpy(wl["src"]).to(dev), torch.from_numpy(wl["dst"]).to(dev)
    g = gnn.coo_to_csr(N, src_d, dst_d)
    del src_d, dst_d
    w_csr = gnn.permute_edge_data(g.eid, torch.from_numpy(wl["w"]).to(dev))
    w_csrT = gnn.permute_edge_data(g.t2f, w_csr)
    # features and incoming gradients are drawn straight into pinned host memory (reused by the end-to-end leg)
    want_e2e = not args.no_e2e
    hX = torch.empty(N * fmax, dtype=torch.float32, pin_memory=want_e2e)
    hR = torch.empty(N * fmax, dtype=torch.float32, pin_memory=want_e2e)
    synth.normal_f32_into(hX.numpy(), seed, 20)
    synth.normal_f32_into(hR.numpy(), seed, 21)
    X32, R32 = hX.to(dev), hR.to(dev)
    wl["src"] = wl["dst"] = None  # host copies of the topology are no longer needed
    Xb, Rb = X32.to(torch.bfloat16), R32.to(torch.bfloat16)  # RNE, same bits as the host bf16 generator
    out32 = torch.empty(N * fmax, dtype=torch.float32, device=dev)
    dX32 = torch.empty(N * fmax, dtype=torch.float32, device=dev)
    # the reduction's scratch is asked for every width that runs (its size is not monotone in F)
    ws = torch.empty(max(gnn.propagate_fused_workspace(E, F, "sum") for F, _ in cases), dtype=torch.uint8, device=dev)
    torch.cuda.empty_cache()

    def views(F, dt):
        n = N * F
        if dt == "f32":
            return X32[:n].view(N, F), R32[:n].view(N, F), out32[:n].view(N, F), dX32[:n].view(N, F)
        return (Xb[:n].view(N, F), Rb[:n].view(N, F), out32.view(torch.bfloat16)[:n].view(N, F),
                dX32.view(torch.bfloat16)[:n].view(N, F))

    plan = []  # (F, dt, weighted, tensors)
    for F, dt in cases:
        for weighted in (False, True):
            plan.append((F, dt, weighted, views(F, dt)))
    stream = torch.cuda.current_stream()

    def step(events=None):
        for i, (F, dt, weighted, (X, R, out, dX)) in enumerate(plan):
            if events is not None:
                events[i][0].record(stream)
            gnn.propagate_fused(g, X, w_csr if weighted else None, "sum", out=out, ws=ws)
            if events is not None:
                events[i][1].record(stream)
            gnn.propagate_fused_backward(g, R, "sum", w_csrT=w_csrT if weighted else None, dX=dX, ws=ws)
            if events is not None:
                events[i][2].record(stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in plan] for _ in range(args.steps)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    t0.record(stream)
    for k in range(args.steps):
        step(ev[k])
    t1.record(stream)
    barrier()
    clocks = sampler.stop()
    total_ms = t0.elapsed_time(t1)
    total_ms = all_max(total_ms, dev, world)
    ms_per_step = total_ms / args.steps
    work = sum(E * F for F, _, _, _ in plan)  # edges*features per step (each fwd+bwd pair counted once)
    value = whole_job_value(work, ms_per_step, world)

    # ---- edge-weight gradient of the e_mul_xj cases (one dot product per edge), timed after the step and
    # reported per case beside the dX time; it is not part of `value`
    dw_ms = {}
    if not args.no_dw:
        dWbuf = torch.empty(E, dtype=torch.float32, device=dev)
        for F, dt, weighted, (X, R, out, dX) in plan:
            if not weighted:
                continue
            for _ in range(2):
                gnn.propagate_fused_backward(g, R, "sum", X=X, want_dX=False, want_dW=True, dW=dWbuf, ws=ws)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(3):
                gnn.propagate_fused_backward(g, R, "sum", X=X, want_dX=False, want_dW=True, dW=dWbuf, ws=ws)
            b.record(stream)
            torch.cuda.synchronize()
            dw_ms[(F, dt)] = a.elapsed_time(b) / 3
        del dWbuf

    # ---- the bare gathers of one pass (no rows, no multipliers, no output) per row width: the ceiling that the
    # L2 -> SM return path sets for the reduction kernels on this index stream, measured here on this machine
    gather_loop = {}
    if not args.no_probe:
        sink = torch.empty(gnn.load().gnn_probe_gather_sink_floats(E), dtype=torch.float32, device=dev)
        for rb in (64, 128, 256, 512):
            Xv = X32[:N * (rb // 4)].view(N, rb // 4)
            for _ in range(3):
                gnn.probe_gather(g.col[:E], Xv, rb, sink=sink)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(8):
                gnn.probe_gather(g.col[:E], Xv, rb, sink=sink)
            b.record(stream)
            torch.cuda.synchronize()
            gather_loop[rb] = E * rb / (a.elapsed_time(b) / 8) / 1e6  # GB/s
        del sink

    # ---- per-case breakdown and the roofline of the chunked propagate kernel
    peak, peak_src = measured_peak()
    per_case, tot_ms, tot_comp, tot_gath = [], 0.0, 0.0, 0.0
    for i, (F, dt, weighted, _) in enumerate(plan):
        s = 2 if dt == "bf16" else 4
        f_ms = statistics.mean(ev[k][i][0].elapsed_time(ev[k][i][1]) for k in range(args.steps))
        b_ms = statistics.mean(ev[k][i][1].elapsed_time(ev[k][i][2]) for k in range(args.steps))
        comp, gath = compulsory_bytes(N, E, F, s, weighted), gather_bytes(N, E, F, s, weighted)
        tot_ms += f_ms + b_ms
        tot_comp += 2 * comp
        tot_gath += 2 * gath
        per_case.append({"F": F, "dtype": dt, "msg": "e_mul_xj" if weighted else "copy_xj", "fwd_ms": round(f_ms, 4), "bwd_ms": round(b_ms, 4),
                         "edges_feat_per_s": E * F / ((f_ms + b_ms) * 1e-3), "compulsory_GBs_fwd": comp / f_ms / 1e6,
                         "l2_side_model_GBs_fwd": gath / f_ms / 1e6, "compulsory_frac_fwd": comp / f_ms / 1e6 / peak})
        if weighted and (F, dt) in dw_ms:
            per_case[-1]["bwd_dW_ms"] = round(dw_ms[(F, dt)], 4)
        if gather_loop:  # rows wider than 512 bytes run as 512-byte column slabs
            per_case[-1]["frac_of_gather_loop_fwd"] = E * F * s / f_ms / 1e6 / gather_loop[min(F * s, 512)]
    # dominant kernel instance = the case with the largest share of the step
    dom = max(per_case, key=lambda c: c["fwd_ms"] + c["bwd_ms"])
    sdom = 2 if dom["dtype"] == "bf16" else 4
    wdom = dom["msg"] == "e_mul_xj"
    comp = compulsory_bytes(N, E, dom["F"], sdom, wdom)
    tkey = "%d:%s:%s:fwd" % (dom["F"], dom["dtype"], dom["msg"])
    traffic_valid = shrink == 0 and not args.natural_ids and kernel_sources_digest() == TRAFFIC_KERNEL_SHA256
    traffic = TRAFFIC_GB.get(tkey) if traffic_valid else None
    achieved = comp / dom["fwd_ms"] / 1e6
    nslab = max(1, dom["F"] * sdom // 512)
    roofline = {"bound": "hbm", "kernel": "propagate_chunk_kernel, forward call of F=%d %s %s = %d column-slab launch(es) + fix-up (largest share of the step: %.1f %%); bytes, time and traffic are per call"
                % (dom["F"], dom["dtype"], dom["msg"], nslab, 100 * (dom["fwd_ms"] + dom["bwd_ms"]) / tot_ms),
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": None if traffic is None else traffic * 1e9,
                "traffic_scaled_from_reduced_graph": traffic is not None,
                "traffic_source": (TRAFFIC_SOURCE + "; kernel sources sha256 " + TRAFFIC_KERNEL_SHA256[:16]) if traffic is not None else
                                  "null: the kernel sources differ from the ones the counters were taken with, or this is not the full-size relabelled workload",
                "peak_source": peak_src, "bytes_model": "compulsory bytes per call: 4E(+4E weights)+8N+2*N*F*s = %d" % comp,
                "ms_per_call": dom["fwd_ms"], "launches_per_call": launches_per_pass(E) * nslab,
                "dram_traffic_GBs": None if traffic is None else traffic * 1e3 / dom["fwd_ms"],
                "dram_traffic_frac_of_peak": None if traffic is None else traffic * 1e3 / dom["fwd_ms"] / peak,
                "l2_side_model_GBs": gather_bytes(N, E, dom["F"], sdom, wdom) / dom["fwd_ms"] / 1e6,
                "gather_loop_GBs": {str(k): v for k, v in gather_loop.items()} or None,
                "gather_loop_note": "E * row bytes / time of gnn_probe_gather (the gathers of one pass and nothing else) per row width, measured in this run after the timed steps: the L2 -> SM ceiling of this index stream; per_case.frac_of_gather_loop_fwd = gathered bytes of the forward call / time / that ceiling",
                "l2_side_model_note": "bytes if every edge fetched its row with no reuse, over time: a rate on the L2 -> SM side (it can exceed any HBM peak), not DRAM bandwidth",
                "all_launches": {"compulsory_GBs": tot_comp / tot_ms / 1e6, "frac": tot_comp / tot_ms / 1e6 / peak,
                                 "l2_side_model_GBs": tot_gath / tot_ms / 1e6,
                                 "dram_traffic_GBs": (sum(TRAFFIC_GB["%d:%s:%s:%s" % (c["F"], c["dtype"], c["msg"], d)] for c in per_case for d in ("fwd", "bwd")) * 1e3 / tot_ms
                                                      if traffic_valid and all(TRAFFIC_GB.get("%d:%s:%s:fwd" % (c["F"], c["dtype"], c["msg"])) for c in per_case) else None)}}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32 accumulate (bf16 and f32 storage)", "data": "synthetic",
            "config": {"workload": ("VARIANT with the generator's natural vertex ids of: " if args.natural_ids else "") + WORKLOAD_NAME if shrink == 0 else f"REDUCED graph (R-MAT scale {args.graph_scale}) of: " + WORKLOAD_NAME, "N": N, "E": E, "cases": [f"{F}:{dt}" for F, dt in cases],
                       "l2": "inputs larger than L2: every launch streams >= 0.5 GB of indices and a feature matrix of 154 MB to 4.9 GB",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks, "gpu_launches": args.steps * sum(2 * launches_per_pass(E) * max(1, F * (2 if dt == "bf16" else 4) // 512) for F, dt, _, _ in plan), "roofline": roofline, "per_case": per_case}

    # ---- end to end through the host-buffer entry points
    if not args.no_e2e and hasattr(gnn, "propagate_fused_host"):
        line["e2e"] = run_e2e(args, torch, gnn, g, plan, hX, hR, w_csr, w_csrT, ws, N, E, fmax, dev, world, barrier)
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        cores = len(os.sched_getaffinity(0))
        oracle.set_threads(cores)
        sample = cpu_sample(synth)
        cpu_step(oracle, sample)
        t = min(cpu_step(oracle, sample) for _ in range(2))
        line["cpu_baseline"] = {"value": sample["E"] * sample["F"] / t, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample["desc"]}
        del sample
        oracle.set_threads(1)  # the same checker on one thread, on a sample an eighth of the size
        small = cpu_sample(synth, pairs=2_000_000, scale=17)
        t1 = min(cpu_step(oracle, small) for _ in range(2))
        line["cpu_baseline"].update({"value_1thread": small["E"] * small["F"] / t1, "sample_1thread": small["desc"]})
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def launches_per_pass(E):
    """Kernels one column-slab pass of a sum launches: the chunk kernel, the fix-up of cut rows and, on graphs of
    16384 chunks and more, the fix-up of hub rows (chunks are 1024 positions from 8 Mi edges on, 256 below)."""
    chunk = 1024 if E >= 8 * 1024 * 1024 else 256
    return 3 if -(-E // chunk) >= 16384 else 2


def run_e2e(args, torch, gnn, g, plan, hX, hR, w_csr, w_csrT, ws, N, E, fmax, dev, world, barrier):
    """Same step, but features and incoming gradients start in pinned host memory and both results
    end in pinned host memory, every case, inside the timed region.  The graph and the edge
    weights stay resident (they do not change from step to step in full-graph training)."""
    pin = dict(pin_memory=True)
    hXp, hRp = hX, hR  # already pinned
    hXb, hRb = hX.to(torch.bfloat16).pin_memory(), hR.to(torch.bfloat16).pin_memory()
    # forward calls and backward calls each alternate between `lanes` streams; every stream has its own pinned
    # result buffer, device staging buffers and workspace, so that independent calls overlap: the host->device
    # copy of one call runs beside the device->host copy of another (the link is full duplex) and beside the
    # kernels of a third
    lanes = max(1, args.e2e_lanes)
    nl = 2 * lanes
    hres = [torch.empty(N * fmax, dtype=torch.float32, **pin) for _ in range(nl)]
    stage = [torch.empty(N * fmax, dtype=torch.float32, device=dev) for _ in range(2 * nl)]
    wss = [ws] + [torch.empty_like(ws) for _ in range(nl - 1)]
    s_main = torch.cuda.current_stream()
    streams = [s_main] + [torch.cuda.Stream() for _ in range(nl - 1)]
    h2d = d2h = 0
    calls = []
    for i, (F, dt, weighted, _) in enumerate(plan):
        n = N * F
        lf, lb = 2 * (i % lanes), 2 * (i % lanes) + 1  # lanes of this case's forward and backward call

        def view(t):
            return (t if dt == "f32" else t.view(torch.bfloat16))[:n].view(N, F)
        hx, hr = (hXp, hRp) if dt == "f32" else (hXb, hRb)
        hx, hr = hx[:n].view(N, F), hr[:n].view(N, F)
        calls.append((hx, hr, view(hres[lf]), view(hres[lb]), [view(stage[2 * lf]), view(stage[2 * lf + 1]), view(stage[2 * lb]), view(stage[2 * lb + 1])],
                      weighted, lf, lb))
        h2d += 2 * hx.numel() * hx.element_size()
        d2h += 2 * hx.numel() * hx.element_size()

    def step():
        for hx, hr, ho, hd, st, weighted, lf, lb in calls:
            with torch.cuda.stream(streams[lf]):
                gnn.propagate_fused_host(g, hx, w_csr if weighted else None, "sum", ho, st[0], st[1], wss[lf])
            with torch.cuda.stream(streams[lb]):
                gnn.propagate_fused_backward_host(g, hr, "sum", w_csrT if weighted else None, hd, st[2], st[3], wss[lb])

    def join():  # the main stream waits for everything queued on the others
        for s_ in streams[1:]:
            s_main.wait_stream(s_)

    for s_ in streams[1:]:
        s_.wait_stream(s_main)
    step()
    join()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0.record(s_main)
    for s_ in streams[1:]:
        s_.wait_event(t0)
    for _ in range(args.e2e_steps):
        step()
    join()
    t1.record(s_main)
    barrier()
    ms = t0.elapsed_time(t1) / args.e2e_steps
    ms = all_max(ms, dev, world)
    work = sum(E * F for F, _, _, _ in plan)
    return {"value": whole_job_value(work, ms, world), "unit": UNIT, "ms_per_step": ms, "steps": args.e2e_steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "streams": nl,
            "note": "features and gradients copied from pinned host memory, results copied back, per case; forward and backward calls alternate over %d streams (copies in both directions and kernels of independent calls overlap); graph and edge weights resident" % nl}


if __name__ == "__main__":
    main()
