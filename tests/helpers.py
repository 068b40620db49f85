"""Shared test helpers: tolerance for normed/rotated values, small utilities."""
import warnings

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


def parity_stats(got_bits, ref_bits, ref_f32):
    """Distances between the kernel's and the oracle's normed / rotated values.

    Returns the worst error over the tolerance above, how many elements differ in
    their bits, how many lie beyond 2 bf16 ulp of their OWN magnitude (no floor:
    the strict reading) and a histogram of the distance in ulp of the reference's
    own magnitude: bins 0, 1, 2, 3-4, 5-8, 9-16, > 16."""
    got = bits_to_f32(got_bits).astype(np.float64)
    ref = bits_to_f32(ref_bits).astype(np.float64)
    tol = norm_rope_tolerance(ref_bits, ref_f32)
    err = np.abs(got - ref)
    own = ulp_bf16(np.maximum(np.abs(ref), 2.0 ** -126))
    d = np.rint(err / own).astype(np.int64)
    edges = [0, 1, 2, 4, 8, 16]
    hist = {"0": int((d == 0).sum()), "1": int((d == 1).sum()), "2": int((d == 2).sum())}
    for lo, hi in zip(edges[2:-1], edges[3:]):
        hist[f"{lo + 1}-{hi}"] = int(((d > lo) & (d <= hi)).sum())
    hist[">16"] = int((d > 16).sum())
    return dict(n=int(err.size), n_diff=int((np.asarray(got_bits) != np.asarray(ref_bits)).sum()),
                n_beyond_tolerance=int((err > tol).sum()), n_strict_fail=int((err > 2.0 * own).sum()),
                max_err_over_tol=float((err / tol).max()) if err.size else 0.0, ulp_hist=hist)


def assert_norm_rope_close(got_bits, ref_bits, ref_f32, what="", report=False):
    st = parity_stats(got_bits, ref_bits, ref_f32)
    assert st["n_beyond_tolerance"] == 0, (f"{what}: {st['n_beyond_tolerance']} of {st['n']} elements beyond 2 bf16 ulp; "
                                           f"worst err/tol = {st['max_err_over_tol']:.3f}")
    if report:
        note(f"{what}: {st}")
    return st


def note(text):
    """Keeps a measured figure visible in the run record: printed, and listed in
    pytest's warnings summary even in quiet mode."""
    print(text)
    warnings.warn(UserWarning("parity report: " + text), stacklevel=2)


def exact_norm_rope_rows(x_bits, w_bits, eps, pos_rows, theta):
    """The textbook formula in float64 for selected (token, head) rows.

    x_bits [R][D] bf16 bits, pos_rows [R][2]; returns float64 [R][D], unrounded.
    Written independently of the oracle: used to judge which of two fp32
    evaluations is closer to the truth."""
    x = bits_to_f32(x_bits).astype(np.float64)
    w = bits_to_f32(w_bits).astype(np.float64)
    R, D = x.shape
    y = x / np.sqrt((x * x).mean(axis=1, keepdims=True) + float(np.float32(eps))) * w[None, :]
    n = D // 4
    i = np.arange(D // 2) % n
    axis = np.arange(D // 2) // n
    freq = np.power(float(theta), -2.0 * i / (D // 2))
    phi = pos_rows[:, axis].astype(np.float64) * freq[None, :]
    c, s = np.cos(phi), np.sin(phi)
    a, b = y[:, 0::2], y[:, 1::2]
    out = np.empty_like(y)
    out[:, 0::2] = a * c - b * s
    out[:, 1::2] = a * s + b * c
    return out
