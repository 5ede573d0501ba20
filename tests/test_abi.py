"""The C-ABI library loads without a GPU and exports every symbol that include/gnn.h declares."""
import ctypes
import os
import re

import pytest

from paper_2412_06354_b200 import build, gnn

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gnn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gnn_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    build.build()
    lib = ctypes.CDLL(gnn.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in gnn.h but not exported"
    # and the binding knows every one of them
    assert set(names) == set(gnn.SIGNATURES), set(names) ^ set(gnn.SIGNATURES)


def test_host_only_calls():
    lib = gnn.load()
    assert lib.gnn_version() >= 100
    assert lib.gnn_status_string(0) == b"ok"
    assert lib.gnn_status_string(2) == b"index out of range"
    assert lib.gnn_coo_to_csr_workspace(10, 1000) >= 4 * 1000 * 4
    assert lib.gnn_propagate_fused_workspace(1000, 64, gnn.SUM) >= 4 * 2 * 64 * 4
    assert lib.gnn_propagate_fused_workspace(1000, 64, gnn.MAX) > lib.gnn_propagate_fused_workspace(1000, 64, gnn.SUM)


def test_argument_errors_are_reported_before_any_launch():
    lib = gnn.load()
    # null pointers / bad sizes never reach the device
    assert lib.gnn_coo_to_csr(-1, 0, None, None, None, None, 0, None) == 1
    assert b"negative" in lib.gnn_last_error_string()
    assert lib.gnn_add_self_loops(3, 2, None, None, None, None, None) == 1
    assert lib.gnn_permute_edge_data(None, 5, 1, 3, None, None, None) == 1
    assert lib.gnn_degree(None, 0, None, None, None) == 1


def test_binding_rejects_wrong_index_dtype():
    """The C ABI takes raw pointers, so the binding checks the element type of index tensors."""
    import torch
    from paper_2412_06354_b200 import gnn
    with pytest.raises(TypeError):
        gnn._pi(torch.zeros(3, dtype=torch.int32), torch.int64, "graph_ptr")
    with pytest.raises(TypeError):
        gnn._pf32(torch.zeros(3, dtype=torch.float64), "w_csr")
    assert gnn._pi(None, torch.int32, "argmax") is None
    assert gnn._pi(torch.zeros(3, dtype=torch.int32), torch.int32, "src") is not None
