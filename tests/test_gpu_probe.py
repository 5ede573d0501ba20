"""The bare gather loop (a measurement aid): it runs on every supported row width, touches only its sink, and
refuses other widths."""
import numpy as np
import pytest

from test_gpu_propagate import ragged_graph
from util import to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gnn():
    import torch
    from paper_2412_06354_b200 import gnn as g
    g.load()
    assert torch.cuda.is_available()
    return g


def test_probe_gather_runs_inside_its_sink(gnn):
    import torch
    n, src, dst = ragged_graph(5)
    g = gnn.coo_to_csr(n, to_dev(src), to_dev(dst))
    need = gnn.load().gnn_probe_gather_sink_floats(g.E)
    for rb in (64, 128, 256, 512):
        X = torch.ones(n, rb // 4, device="cuda")
        buf = torch.full((need + 2048,), -7.0, device="cuda")
        sink = buf[1024:1024 + need]
        gnn.probe_gather(g.col[:g.E], X, rb, sink=sink)
        torch.cuda.synchronize()
        assert bool((buf[:1024] == -7.0).all()) and bool((buf[1024 + need:] == -7.0).all()), "wrote outside the sink"
        got = sink.cpu().numpy()
        assert np.isfinite(got).all()
        # every position is gathered at least once and X is all ones: four ones per 16-byte chunk
        lanes = rb // 16
        assert got.sum() >= 4.0 * g.E * lanes
    with pytest.raises(gnn.GnnError) as err:
        gnn.probe_gather(g.col[:g.E], torch.ones(n, 24, device="cuda"), 96)
    assert err.value.status == 5  # UNSUPPORTED
