"""GPU parity: dense node-wise transform Y = X*W, dX = dY*W^T, dW = X^T*dY against the CPU checker's
triple loop.  bf16 shapes with K, M multiples of 16 take the tensor-core path."""
import numpy as np
import pytest

import oracle
from paper_2412_06354_b200 import synth
from util import assert_close, bits, to_dev, to_host64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gnn():
    from paper_2412_06354_b200 import gnn as g
    g.load()
    return g


def status_word(ws):
    import torch
    torch.cuda.synchronize()
    return int(ws[:4].view(torch.int32).item())


CASES = [("f32", 2000, 64, 64), ("f32", 1000, 100, 36), ("f32", 333, 128, 128), ("f32", 1000, 256, 64), ("f32", 700, 128, 48), ("f32", 5000, 16, 256), ("bf16", 2000, 64, 64),
         ("bf16", 1000, 128, 128), ("bf16", 777, 256, 256), ("bf16", 129, 16, 32), ("bf16", 5, 256, 16),
         ("bf16", 300, 48, 112), ("bf16", 257, 40, 24),
         # one row; exactly one tile with K and M off the 64-element boxes; several tiles and slots per CTA
         ("bf16", 1, 64, 64), ("bf16", 128, 208, 240), ("bf16", 40000, 128, 64), ("bf16", 20001, 256, 144),
         # fp32 dW on the pipelined kernel (K and M multiples of 32 up to 128): one row, a ragged last slot of 32 rows, many slots per CTA
         ("f32", 1, 128, 32), ("f32", 31, 128, 96), ("f32", 33, 128, 64), ("f32", 30017, 128, 128),
         # ... and with fewer than the 128 feature rows of the MMA
         ("f32", 500, 32, 128), ("f32", 77, 96, 32), ("f32", 6001, 64, 96),
         # ... and up to 256 wide: 16-row slots, two accumulator halves, feature rows past K zero in the second half
         ("f32", 2049, 256, 256), ("f32", 900, 160, 224), ("f32", 300, 128, 256),
         # bf16 dW with K off the 128-row blocks of the MMA (boxes past column K arrive as zeros)
         ("bf16", 5000, 192, 192), ("bf16", 1234, 96, 80), ("bf16", 777, 224, 256), ("bf16", 40, 32, 16),
         # fp32 beyond 256: long contraction (16 slices per tile), many column blocks, four accumulator blocks in dW
         ("f32", 3000, 512, 64), ("f32", 3000, 64, 512), ("f32", 700, 384, 128), ("f32", 900, 512, 512),
         # bf16 dW with up to 512 features (four accumulator blocks)
         ("bf16", 3000, 512, 64), ("bf16", 2000, 384, 128), ("bf16", 1000, 320, 48),
         # bf16 forward / dX beyond 256: weight blocks of two boxes, several column blocks
         ("bf16", 3000, 64, 512), ("bf16", 900, 512, 512), ("bf16", 500, 288, 1024)]


@pytest.mark.parametrize("dtype,n,K,M", CASES)
def test_linear_forward_backward(gnn, dtype, n, K, M):
    oracle.set_threads(8)
    try:
        X = synth.normal((n, K), dtype, 1000 + K)
        a = (6.0 / (K + M)) ** 0.5
        W32 = synth.uniform_f32((K, M), -a, a, 1001 + M)
        W = W32
        if dtype == "bf16":
            import torch
            W = torch.from_numpy(W32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        dY = synth.normal((n, M), dtype, 1002 + M, 1)
        Y, ws = gnn.linear(to_dev(X), to_dev(W), return_ws=True)
        assert status_word(ws) == 0
        Yo, S = oracle.matmul(X, W)
        assert_close(to_host64(Y), Yo, S, dtype, f"Y {dtype} {n}x{K}x{M}")
        dX, dW, ws = gnn.linear_backward(to_dev(X), to_dev(W), to_dev(dY), return_ws=True)
        assert status_word(ws) == 0
        dXo, S = oracle.matmul(dY, W, tb=True)
        assert_close(to_host64(dX), dXo, S, dtype, "dX")
        dWo, S = oracle.matmul(X, dY, ta=True)
        assert_close(to_host64(dW), dWo, S, dtype, "dW")
        Y2 = gnn.linear(to_dev(X), to_dev(W))
        assert np.array_equal(bits(Y), bits(Y2)), "not bit-reproducible"
    finally:
        oracle.set_threads(1)


def test_linear_large_rows_tensor_core(gnn):
    """N = 100000 rows, 256 -> 256 bf16 (the attention workload's transform): many tiles per CTA."""
    import torch
    n, K, M = 100_000, 256, 256
    X = synth.normal_bf16((n, K), 1100)
    W = torch.from_numpy(synth.glorot_f32(K, M, 1101)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    Y, ws = gnn.linear(to_dev(X), to_dev(W), return_ws=True)
    assert status_word(ws) == 0
    rows = np.random.default_rng(3).choice(n, 3000, replace=False)
    rows = np.union1d(rows, [0, 127, 128, n - 1])
    Yo, S = oracle.matmul(X[rows], W)
    assert_close(to_host64(Y)[rows], Yo, S, "bf16", "sampled rows of Y")
    # linearity in exact arithmetic: rows of zeros give zeros
    Xz = X.copy()
    Xz[::2] = 0
    Yz = gnn.linear(to_dev(Xz), to_dev(W))
    assert torch.count_nonzero(Yz[::2]) == 0 and torch.equal(Yz[1::2], Y[1::2])


def test_linear_degenerate(gnn):
    import torch
    W = torch.zeros((64, 64), device="cuda")
    Y = gnn.linear(torch.zeros((0, 64), device="cuda"), W)
    assert Y.shape == (0, 64)
    dX, dW = gnn.linear_backward(torch.zeros((0, 64), device="cuda"), W, torch.zeros((0, 64), device="cuda"))
    assert torch.count_nonzero(dW) == 0
    with pytest.raises(gnn.GnnError) as e:
        gnn.linear(torch.zeros((8, 64), device="cuda"), W, ws=torch.empty(8, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_linear_back_to_back_launches_are_bitwise_identical(gnn, dtype):
    """Forty launches in a row with nothing in between (the pipelines' barrier phases and ring slots are
    reused at full speed): every result must equal the first one bit for bit, and no wait may expire."""
    import torch
    n, K, M = 170_000, 128, 128
    X = to_dev(synth.normal((n, K), dtype, 1200))
    W32 = synth.glorot_f32(K, M, 1201)
    W = to_dev(W32) if dtype == "f32" else torch.from_numpy(W32).to(torch.bfloat16).cuda()
    dY = to_dev(synth.normal((n, M), dtype, 1202))
    ws = torch.empty(gnn.load().gnn_linear_workspace(n, K, M), dtype=torch.uint8, device="cuda")
    Y0 = gnn.linear(X, W, ws=ws).clone()
    dX0, dW0 = (t.clone() for t in gnn.linear_backward(X, W, dY, ws=ws))
    for _ in range(40):
        Y = gnn.linear(X, W, ws=ws)
        dX, dW = gnn.linear_backward(X, W, dY, ws=ws)
    torch.cuda.synchronize()
    assert status_word(ws) == 0
    assert torch.equal(Y.view(torch.int16 if dtype == "bf16" else torch.int32), Y0.view(torch.int16 if dtype == "bf16" else torch.int32))
    assert torch.equal(dX.float(), dX0.float()) and torch.equal(dW.float(), dW0.float())
