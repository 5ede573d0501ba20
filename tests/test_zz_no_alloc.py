"""gnn_propagate_fused_static: the fused propagate for embedders that are not allowed to allocate device
memory (a host application that owns the whole GPU memory plan, or a latency-bound loop that cannot pay
for cudaMalloc).  Its scratch is an 8 MiB array inside the library, shared by all calls.

The check: through the C ABI, the static variant must give what gnn_propagate_fused gives with a
caller-provided workspace, on two calls in a row (the second call finds the first call's leftovers in the
shared scratch), and it must refuse problems whose scratch would not fit.  This file sorts last on
purpose, so a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest

from paper_2412_06354_b200 import synth
from util import assert_close, bits, to_dev, to_host64

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_workspace_variant_twice():
    import torch
    from paper_2412_06354_b200 import gnn
    gnn.load()
    n, F = 3000, 128
    src, dst = synth.rmat(12, n, 60_000, 77, symmetric=True)       # power-law rows, some cut by chunk boundaries
    g = gnn.coo_to_csr(n, to_dev(src), to_dev(dst))
    eid = g.eid[:g.E].cpu().numpy()
    w = to_dev(synth.uniform_f32((len(src),), 0.0, 1.0, 78)[eid])
    assert gnn.propagate_fused_workspace(g.E, F, "max") <= gnn.load().gnn_propagate_fused_static_max_bytes()
    for call, (dtype, op, weighted) in enumerate([("bf16", "sum", True), ("f32", "max", False)]):
        X = to_dev(synth.normal((n, F), dtype, 79 + call))
        ref = gnn.propagate_fused(g, X, w if weighted else None, op)
        out = torch.full((n, F), float("nan"), dtype=X.dtype, device="cuda")          # caller-owned output
        arg = torch.full((n, F), -7, dtype=torch.int32, device="cuda") if op == "max" else None
        got = gnn.propagate_fused_static(g, X, w if weighted else None, op, out=out, argmax=arg)
        torch.cuda.synchronize()
        if op == "max":
            (ref, ref_arg), (got, got_arg) = ref, got
            assert torch.equal(ref_arg, got_arg)
        r64 = to_host64(ref)
        # same kernels, same order of additions: the tolerance of the other tests is met with room to spare
        assert_close(to_host64(got), r64, np.abs(r64), dtype, f"static scratch, call {call + 1}")
        assert np.array_equal(bits(got), bits(ref))


def test_static_scratch_rejects_oversized_problems():
    from paper_2412_06354_b200 import gnn
    lib = gnn.load()
    cap = lib.gnn_propagate_fused_static_max_bytes()
    assert cap == 8 << 20
    n, F = 2000, 512
    src, dst = synth.rmat(11, n, 300_000, 80, symmetric=True)
    g = gnn.coo_to_csr(n, to_dev(src), to_dev(dst))
    assert gnn.propagate_fused_workspace(g.E, F, "sum") > cap
    with pytest.raises(gnn.GnnError) as e:
        gnn.propagate_fused_static(g, to_dev(synth.normal_f32((n, F), 81)))
    assert e.value.status == 4 and "built-in scratch" in str(e.value)
