"""Seeded synthetic graphs and tensors (inputs only; no message-passing arithmetic).

Thin ctypes wrapper over ``synth.c``.  Every generator is a pure function of its
seed, so the CPU checker and the GPU library can be fed byte-identical arrays.
bf16 tensors are returned as ``uint16`` numpy arrays holding the raw bit patterns.

Workload recipes (``workload_*``) mirror the shapes the library is meant for:
a small Erdos-Renyi graph with self-loops (GCN), a block-diagonal batch of small
graphs (pooling), a preferential-attachment graph (SAGE), and R-MAT graphs
(attention; the large aggregation sweep).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libgnn_synth.so")
_lib = None

BASE_SEED = 2412063540


def build(force: bool = False) -> str:
    src = os.path.join(_HERE, "synth.c")
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", src, "-o", _LIB_PATH, "-lm"])
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB_PATH)
        i32p, u16p, f32p = C.POINTER(C.c_int32), C.POINTER(C.c_uint16), C.POINTER(C.c_float)
        L.synth_u64.restype = C.c_uint64
        L.synth_u64.argtypes = [C.c_uint64] * 3
        L.synth_fill_normal_f32.argtypes = [f32p, C.c_int64, C.c_uint64, C.c_uint64]
        L.synth_fill_normal_bf16.argtypes = [u16p, C.c_int64, C.c_uint64, C.c_uint64]
        L.synth_fill_uniform_f32.argtypes = [f32p, C.c_int64, C.c_double, C.c_double, C.c_uint64, C.c_uint64]
        L.synth_gnm.restype = C.c_int64
        L.synth_gnm.argtypes = [C.c_int32, C.c_int64, C.c_uint64, i32p, i32p]
        L.synth_batched_er.restype = C.c_int64
        L.synth_batched_er.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_double, C.c_uint64, i32p, i32p, i32p, C.c_int64]
        L.synth_barabasi_albert.restype = C.c_int64
        L.synth_barabasi_albert.argtypes = [C.c_int32, C.c_int32, C.c_uint64, i32p, i32p]
        L.synth_rmat.argtypes = [C.c_int32, C.c_int32, C.c_int64, C.c_double, C.c_double, C.c_double, C.c_int32, C.c_uint64, i32p, i32p]
        L.synth_relabel.argtypes = [C.c_int32, C.c_int64, C.c_uint64, i32p, i32p]
        L.synth_sort_by_dst.argtypes = [C.c_int32, C.c_int64, i32p, i32p]
        _lib = L
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t))


# ------------------------------------------------------------------ tensors
def normal_f32(shape, seed, stream=0):
    out = np.empty(shape, dtype=np.float32)
    _load().synth_fill_normal_f32(_p(out, C.c_float), out.size, seed, stream)
    return out


def normal_f32_into(out, seed, stream=0):
    """Fill an existing contiguous float32 array (e.g. a view of pinned memory) with the same draws as normal_f32."""
    assert out.dtype == np.float32 and out.flags["C_CONTIGUOUS"]
    _load().synth_fill_normal_f32(_p(out, C.c_float), out.size, seed, stream)
    return out


def normal_bf16(shape, seed, stream=0):
    out = np.empty(shape, dtype=np.uint16)
    _load().synth_fill_normal_bf16(_p(out, C.c_uint16), out.size, seed, stream)
    return out


def uniform_f32(shape, lo, hi, seed, stream=0):
    out = np.empty(shape, dtype=np.float32)
    _load().synth_fill_uniform_f32(_p(out, C.c_float), out.size, float(lo), float(hi), seed, stream)
    return out


def glorot_f32(fan_in, fan_out, seed, stream=0):
    a = (6.0 / (fan_in + fan_out)) ** 0.5
    return uniform_f32((fan_in, fan_out), -a, a, seed, stream)


def normal(shape, dtype, seed, stream=0):
    """dtype 'f32' -> float32 array, 'bf16' -> uint16 bit patterns."""
    return normal_f32(shape, seed, stream) if dtype == "f32" else normal_bf16(shape, seed, stream)


def bf16_to_f32(u16):
    return (u16.astype(np.uint32) << 16).view(np.float32)


def to_f64(a):
    """Exact widening of an f32 array or a bf16 bit-pattern array."""
    if a.dtype == np.uint16:
        return bf16_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


# ------------------------------------------------------------------ graphs
def gnm(n, pairs, seed):
    src = np.empty(2 * pairs, np.int32)
    dst = np.empty(2 * pairs, np.int32)
    e = _load().synth_gnm(n, pairs, seed, _p(src, C.c_int32), _p(dst, C.c_int32))
    return src[:e].copy(), dst[:e].copy()


def batched_er(G, nmin, nmax, p, seed):
    cap = G * nmax * (nmax - 1)
    src = np.empty(cap, np.int32)
    dst = np.empty(cap, np.int32)
    gptr = np.empty(G + 1, np.int32)
    e = _load().synth_batched_er(G, nmin, nmax, p, seed, _p(gptr, C.c_int32), _p(src, C.c_int32), _p(dst, C.c_int32), cap)
    assert e >= 0
    return src[:e].copy(), dst[:e].copy(), gptr


def barabasi_albert(n, m, seed, relabel=True):
    m0 = m + 1
    E = 2 * (m0 * (m0 - 1) // 2 + m * (n - m0))
    src = np.empty(E, np.int32)
    dst = np.empty(E, np.int32)
    e = _load().synth_barabasi_albert(n, m, seed, _p(src, C.c_int32), _p(dst, C.c_int32))
    assert e == E
    if relabel:
        _load().synth_relabel(n, E, seed, _p(src, C.c_int32), _p(dst, C.c_int32))
    return src, dst


def rmat(scale, n, pairs, seed, symmetric, relabel=True, sort_by_dst=False, a=0.57, b=0.19, c=0.19):
    E = pairs * (2 if symmetric else 1)
    src = np.empty(E, np.int32)
    dst = np.empty(E, np.int32)
    L = _load()
    L.synth_rmat(scale, n, pairs, a, b, c, int(symmetric), seed, _p(src, C.c_int32), _p(dst, C.c_int32))
    if relabel:
        L.synth_relabel(n, E, seed, _p(src, C.c_int32), _p(dst, C.c_int32))
    if sort_by_dst:
        L.synth_sort_by_dst(n, E, _p(src, C.c_int32), _p(dst, C.c_int32))
    return src, dst


def with_self_loops(n, src, dst):
    """Append one loop per node, in node order, after the original edges (input for tests
    that want the looped COO directly on the host)."""
    loops = np.arange(n, dtype=np.int32)
    return np.concatenate([src, loops]), np.concatenate([dst, loops])


# ------------------------------------------------------------------ workloads
def workload_gcn_small(seed=BASE_SEED + 1):
    """N=2000, 5000 symmetric pairs (10000 directed edges), X 2000x64 f32, W 64x64 Glorot."""
    n, F = 2000, 64
    src, dst = gnm(n, 5000, seed)
    return dict(N=n, src=src, dst=dst, X=normal_f32((n, F), seed, 10), W=glorot_f32(F, F, seed, 11), F=F)


def workload_batched(seed=BASE_SEED + 2, G=512, F=128):
    src, dst, gptr = batched_er(G, 10, 40, 0.2, seed)
    n = int(gptr[-1])
    return dict(N=n, G=G, src=src, dst=dst, graph_ptr=gptr, F=F, X=normal_f32((n, F), seed, 10),
                W1=glorot_f32(F, F, seed, 11), W2=glorot_f32(F, F, seed, 12))


def workload_powerlaw(seed=BASE_SEED + 3, n=170_000, m=4, F=128, dtype="f32"):
    src, dst = barabasi_albert(n, m, seed)
    return dict(N=n, src=src, dst=dst, F=F, X=normal((n, F), dtype, seed, 10),
                W_self=glorot_f32(F, F, seed, 11), W_neigh=glorot_f32(F, F, seed, 12))


def workload_attention(seed=BASE_SEED + 4, n=100_000, scale=17, E=1_600_000, H=8, Cw=32):
    src, dst = rmat(scale, n, E, seed, symmetric=False)
    a = (6.0 / (Cw + 1)) ** 0.5
    return dict(N=n, src=src, dst=dst, H=H, C=Cw, Wx=normal_bf16((n, H * Cw), seed, 10),
                a_src=uniform_f32((H, Cw), -a, a, seed, 11), a_dst=uniform_f32((H, Cw), -a, a, seed, 12))


def workload_large_graph(seed=BASE_SEED + 5, n=2_400_000, scale=22, pairs=61_500_000, relabel=True):
    """Topology and edge weights of the large sweep; features are drawn per (F, dtype)."""
    src, dst = rmat(scale, n, pairs, seed, symmetric=True, relabel=relabel, sort_by_dst=True)
    w = uniform_f32((src.shape[0],), 0.0, 1.0, seed, 13)
    return dict(N=n, src=src, dst=dst, w=w, seed=seed)
