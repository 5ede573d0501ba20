"""B200-native message-passing primitives (gather / apply_edges / aggregate / fused propagate,
edge softmax, batched-graph pooling and their backward passes) behind a C ABI.

``paper_2412_06354_b200.gnn``   ctypes binding of libgnn_b200.so (sm_100a CUDA kernels)
``paper_2412_06354_b200.synth`` seeded synthetic inputs (no message-passing arithmetic)

Nothing is imported eagerly: the CUDA library is loaded on first use of ``gnn`` and the
binding raises if it is missing (there is no CPU fallback).
"""
__version__ = "0.1.0"
