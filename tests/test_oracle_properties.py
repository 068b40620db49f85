"""Randomised property pins for the oracle (hypothesis): shapes and values are
drawn at random, the expected results come from definitions that do not share
code with the oracle (axis swap, sorted reference, fancy indexing)."""
import numpy as np
from hypothesis import given, settings, strategies as st

import oracle

_settings = dict(max_examples=40, deadline=None)


@st.composite
def shapes(draw):
    P = draw(st.integers(1, 6))
    S = P * draw(st.integers(1, 9))
    H = P * draw(st.integers(1, 4))
    D = 2 * draw(st.integers(1, 8))
    return P, S, H, D


@settings(**_settings)
@given(shapes(), st.integers(0, 2 ** 31))
def test_exchange_is_an_axis_swap_and_a_bijection(shape, seed):
    P, S, H, D = shape
    x = np.random.default_rng(seed).integers(0, 1 << 16, (S, H, D), dtype=np.uint16)
    y = oracle.ulysses_a2a(x, P)
    assert np.array_equal(y, x.transpose(1, 0, 2))
    assert np.array_equal(oracle.ulysses_a2a_inverse(y, P), x)
    if P % 2 == 0:
        assert np.array_equal(oracle.tapa_phase2(oracle.tapa_phase1(x, P), P), y)


@settings(**_settings)
@given(st.integers(1, 8), st.integers(1, 40), st.floats(0.0, 1.0), st.integers(1, 5), st.integers(0, 2 ** 31))
def test_selection_equals_sorting_by_metric_then_index(n_groups, g, r, spread, seed):
    n = n_groups * g
    metric = np.random.default_rng(seed).integers(0, spread * 3 + 1, n).astype(np.uint64)
    mask, idx, na = oracle.vmajor_select(metric, n_groups, r)
    want = np.ones(n, np.uint8)
    for grp in range(n_groups):
        order = sorted(range(grp * g, (grp + 1) * g), key=lambda i: (int(metric[i]), i))
        want[order[:int(np.floor(r * g))]] = 0
    assert np.array_equal(mask, want)
    assert np.array_equal(idx, np.flatnonzero(want)) and na == int(want.sum())
    # everything cached is no larger than everything active, group by group
    for grp in range(n_groups):
        m = metric[grp * g:(grp + 1) * g]
        k = mask[grp * g:(grp + 1) * g].astype(bool)
        if k.any() and (~k).any():
            assert m[~k].max() <= m[k].min()


@settings(**_settings)
@given(shapes(), st.integers(1, 4), st.integers(0, 2 ** 31))
def test_compaction_then_scatter_rebuilds_exactly_the_active_rows(shape, tdiv, seed):
    P, S, H, D = shape
    Sl = S // P
    T = max(1, Sl // tdiv)
    while Sl % T:
        T -= 1
    n = S // T
    rng = np.random.default_rng(seed)
    cur = rng.integers(0, 1 << 16, (S, H, D), dtype=np.uint16)
    old = rng.integers(0, 1 << 16, (H, S, D), dtype=np.uint16)
    idx = np.sort(rng.choice(n, rng.integers(0, n + 1), replace=False)).astype(np.int32)
    comp = oracle.pack_active(cur, idx, P, T)
    tok = (idx[:, None] * T + np.arange(T)[None, :]).reshape(-1)
    assert np.array_equal(comp, cur[tok].transpose(1, 0, 2))
    cache = oracle.unpack(comp, idx, old.copy(), P, T)
    want = old.copy()
    want[:, tok] = cur[tok].transpose(1, 0, 2)
    assert np.array_equal(cache, want)


@settings(**_settings)
@given(st.integers(1, 6), st.integers(1, 3), st.sampled_from([4, 8, 16]), st.integers(0, 2 ** 31))
def test_metric_is_additive_over_units_and_symmetric(n, H, D, seed):
    T = 2
    S = n * T
    rng = np.random.default_rng(seed)
    a = rng.integers(0, 0x7F80, (S, H, D), dtype=np.uint16)       # finite non-negative bf16
    b = rng.integers(0, 0x7F80, (S, H, D), dtype=np.uint16)
    m = oracle.vmajor_metric(a, b, 1, T)
    assert np.array_equal(m, oracle.vmajor_metric(b, a, 1, T))
    fine = oracle.vmajor_metric(a, b, 1, 1)                        # per-token metric
    assert np.array_equal(m, fine.reshape(n, T).sum(axis=1))
