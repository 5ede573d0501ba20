"""Shared helpers of the GPU parity tests: host<->device conversion and the tolerance rule."""
import numpy as np

TOL = {"f32": 1e-5, "bf16": 2e-2}


def to_dev(a, device="cuda"):
    """numpy -> torch on the device; uint16 arrays are bf16 bit patterns."""
    import torch
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def to_host64(t):
    """torch (f32 / bf16 / int) -> numpy float64 (exact)."""
    import torch
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy().astype(np.float64)
    return t.cpu().numpy().astype(np.float64)


def bits(t):
    """Raw bit patterns of a device tensor as a numpy integer array (for bit-exact checks)."""
    import torch
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy()
    if t.dtype == torch.float32:
        return t.view(torch.int32).cpu().numpy()
    return t.cpu().numpy()


def host_bits(a):
    """Bit patterns a host input array would have when stored as its dtype on the device."""
    if a.dtype == np.uint16:
        return a.view(np.int16)
    if a.dtype == np.float32:
        return a.view(np.int32)
    return a


def f64_to_dtype_bits(x64, dtype):
    """Round float64 values that are exactly representable in dtype to their bit patterns."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x64))
    if dtype == "bf16":
        return t.to(torch.bfloat16).view(torch.int16).numpy()
    return t.to(torch.float32).view(torch.int32).numpy()


def assert_close(got, ref, S, dtype, what="", extra=None):
    """Element-wise: f32 |got-ref| <= 1e-5*S ; bf16 |got-ref| <= 2e-2*|ref| + 1e-5*S, where S is the
    sum of |terms| of the element (S >= |ref|).  Plus the norm-wise bound on the whole tensor.
    extra (optional, same shape): an absolute allowance per element that the caller derives for
    elements reached by a floating-point branch decision (zero elsewhere); it widens both bounds."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    S = np.asarray(S, np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref)
    bound = 1e-5 * S if dtype == "f32" else 2e-2 * np.abs(ref) + 1e-5 * S
    if extra is not None:
        extra = np.asarray(extra, np.float64)
        assert extra.shape == ref.shape and (extra >= 0).all()
        bound = bound + extra
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} elements out of tolerance; worst at {i}: "
                             f"got {got[i]!r} ref {ref[i]!r} S {S[i]!r} err {err[i]:.3e} bound {bound[i]:.3e}")
    den = np.abs(ref).max() if ref.size else 0.0
    if den > 0:
        nerr = err if extra is None else np.maximum(err - extra, 0.0)
        assert nerr.max() / den <= TOL[dtype], f"{what}: norm-wise error {nerr.max() / den:.3e}"
