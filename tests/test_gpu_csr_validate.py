"""The check of a caller-built sparse form: graphs from the library's own conversion pass, and each kind of
damage (planted on the device copies; the check only reads) is reported under its own name."""
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


def fresh(gnn, seed=3):
    n, src, dst = ragged_graph(seed)
    return n, gnn.coo_to_csr(n, to_dev(src), to_dev(dst))


def test_library_graphs_pass(gnn):
    import torch
    for seed in (3, 4):
        n, g = fresh(gnn, seed)
        gnn.csr_validate(g)
    # no edges at all, and a single node
    z = torch.zeros(0, dtype=torch.int32, device="cuda")
    gnn.csr_validate(gnn.coo_to_csr(5, z, z))
    one = torch.zeros(3, dtype=torch.int32, device="cuda")
    gnn.csr_validate(gnn.coo_to_csr(1, one, one))


def expect(gnn, g, words):
    with pytest.raises(gnn.GnnError) as err:
        gnn.csr_validate(g)
    assert err.value.status == 1, err.value  # INVALID_ARG
    for w in words:
        assert w in str(err.value), (w, str(err.value))


def test_each_kind_of_damage_is_named(gnn):
    import torch
    n, g = fresh(gnn)
    g.rowptr[7] += 1  # rows 6 and 7 trade a position: still monotone, but the edges no longer sit in their rows
    expect(gnn, g, ["different edges"])

    n, g = fresh(gnn)
    g.rowptr[10] = g.rowptr[12] + 1
    expect(gnn, g, ["row pointers"])
    n, g = fresh(gnn)
    g.rowptrT[n] -= 1
    expect(gnn, g, ["row pointers"])

    n, g = fresh(gnn)
    g.col[17] = n
    expect(gnn, g, ["node index"])
    n, g = fresh(gnn)
    g.colT[0] = -1
    expect(gnn, g, ["node index"])

    n, g = fresh(gnn)
    g.eid[5] = g.E
    expect(gnn, g, ["edge index"])
    n, g = fresh(gnn)
    g.t2f[9] = -7
    expect(gnn, g, ["edge index"])

    n, g = fresh(gnn)
    g.eidT[100] = g.eidT[101]
    expect(gnn, g, ["permutation"])

    # two positions of one row trade places: everything stays a permutation, the order inside the row breaks
    n, g = fresh(gnn)
    rp = g.rowptr.cpu().numpy()
    r = int(np.argmax(np.diff(rp) >= 2))
    p = int(rp[r])
    e0, e1 = int(g.eid[p]), int(g.eid[p + 1])
    c0, c1 = int(g.col[p]), int(g.col[p + 1])
    g.eid[p], g.eid[p + 1] = e1, e0
    g.col[p], g.col[p + 1] = c1, c0
    expect(gnn, g, ["ascending"])

    # a source swapped for another node: both forms are sound alone but no longer the same edge list
    n, g = fresh(gnn)
    g.col[33] = (int(g.col[33]) + 1) % n
    expect(gnn, g, ["different edges"])

    # a too small workspace is refused before anything runs
    n, g = fresh(gnn)
    with pytest.raises(gnn.GnnError) as err:
        gnn.csr_validate(g, ws=torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert err.value.status == 4


def test_damage_far_into_a_large_graph_is_found(gnn):
    """More rows and positions than one wave of threads covers: the check reaches every one of them."""
    import torch
    n, e = 1_500_000, 2_600_000
    gen = torch.Generator(device="cuda").manual_seed(5)
    src = torch.randint(0, n, (e,), device="cuda", generator=gen, dtype=torch.int32)
    dst = torch.randint(0, n, (e,), device="cuda", generator=gen, dtype=torch.int32)
    g = gnn.coo_to_csr(n, src, dst)
    gnn.csr_validate(g)
    g.col[e - 3] = n + 5
    expect(gnn, g, ["node index"])
    g = gnn.coo_to_csr(n, src, dst)
    g.rowptrT[n - 1] = g.rowptrT[n] + 1
    expect(gnn, g, ["row pointers"])
