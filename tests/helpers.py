"""Shared test helpers: tolerance for normed/rotated values, small utilities."""
import numpy as np


def bits_to_f32(b):
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def ulp_bf16(x):
    """Spacing of bf16 numbers at magnitude x (> 0): 2^(floor(log2 x) - 7)."""
    x = np.asarray(x, dtype=np.float64)
    return np.exp2(np.floor(np.log2(x)) - 7.0)


def norm_rope_tolerance(ref_bits, ref_f32):
    """Allowed |gpu - ref| per element: 2 bf16 ulp at max(|ref|, 2^-9 * rho),
    rho = magnitude of the rotated pair the element belongs to (from the
    oracle's unrounded fp32 values).  The floor matters only where a rotation
    cancels to almost zero."""
    ref = np.abs(bits_to_f32(ref_bits).astype(np.float64))
    f = ref_f32.astype(np.float64).reshape(-1, 2)
    rho = np.sqrt((f * f).sum(axis=1, keepdims=True)).repeat(2, axis=1).reshape(ref.shape)
    mag = np.maximum(ref, rho * 2.0 ** -9)
    mag = np.maximum(mag, 2.0 ** -126)
    return 2.0 * ulp_bf16(mag)


def assert_norm_rope_close(got_bits, ref_bits, ref_f32, what=""):
    got = bits_to_f32(got_bits).astype(np.float64)
    ref = bits_to_f32(ref_bits).astype(np.float64)
    tol = norm_rope_tolerance(ref_bits, ref_f32)
    err = np.abs(got - ref)
    bad = err > tol
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {bad.size} elements beyond 2 bf16 ulp; "
                           f"worst err/tol = {float((err / tol).max()):.3f}")
    # strict count (no cancellation floor), reported by callers that want it
    strict = err > 2.0 * ulp_bf16(np.maximum(np.abs(ref), 2.0 ** -126))
    return dict(max_err_over_tol=float((err / tol).max()), n_diff=int((got_bits != ref_bits).sum()),
                n_strict_fail=int(strict.sum()), n=int(bad.size))
