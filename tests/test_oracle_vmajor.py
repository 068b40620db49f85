"""Pins for the oracle's V-Major metric, selection, compaction and unpack
(Section III-D of the paper): brute force on tiny inputs, special cases
(r = 0 is the full exchange, r = 1 sends nothing), a sort-based reference with
many ties, and the elementwise definition of compaction and scatter."""
import numpy as np
import pytest

import oracle
from paper_2604_14561_b200 import synth

from helpers import bits_to_f32


def _bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _randn_bits(shape, seed, std=1.0):
    return _bits(np.random.default_rng(seed).normal(0, std, size=shape))


# ------------------------------------------------------------------ metric --
def test_metric_zero_when_nothing_changed():
    v = _randn_bits((16, 2, 8), 0)
    assert np.all(oracle.vmajor_metric(v, v, 2, 4) == 0)


def test_metric_single_element_change():
    S, H, D, T = 16, 2, 8, 4
    prev = _bits(np.ones((S, H, D)))
    for delta, want in ((0.5, 32768), (2.0 ** -16, 1), (2.0 ** -17, 0), (3.0, 3 * 65536)):
        cur = bits_to_f32(prev).copy()
        cur[9, 1, 3] = 1.0 + delta if delta >= 2.0 ** -7 else 0.0    # keep it representable
        prev2 = bits_to_f32(prev).copy()
        if delta < 2.0 ** -7:                  # tiny deltas: compare delta against 0 instead
            prev2[9, 1, 3] = delta
            cur[9, 1, 3] = 0.0
        m = oracle.vmajor_metric(_bits(prev2), _bits(cur), 2, T)
        want_vec = np.zeros(S // T, np.uint64)
        want_vec[9 // T] = want
        assert np.array_equal(m, want_vec), delta


def test_metric_brute_force_and_symmetry():
    S, H, D, T, P = 12, 3, 4, 2, 3
    a, b = _randn_bits((S, H, D), 1), _randn_bits((S, H, D), 2)
    m = oracle.vmajor_metric(a, b, P, T)
    fa, fb = bits_to_f32(a), bits_to_f32(b)
    want = []
    for u in range(S // T):
        acc = 0
        for s in range(u * T, (u + 1) * T):
            for h in range(H):
                for j in range(D):
                    d = abs(np.float32(fb[s, h, j]) - np.float32(fa[s, h, j]))   # one fp32 subtraction
                    acc += min(int(float(d) * 65536.0), 2 ** 32 - 1)
        want.append(acc)
    assert m.tolist() == want
    assert np.array_equal(oracle.vmajor_metric(b, a, P, T), m)       # |x - y| = |y - x|
    # close to the real-valued L1 distance: truncation loses < 2^-16 per element
    l1 = np.abs(fb.astype(np.float64) - fa.astype(np.float64)).reshape(S // T, -1).sum(1)
    assert np.all(np.abs(m / 65536.0 - l1) < (T * H * D) * 2.0 ** -15)


def test_metric_saturates_and_counts_nan_as_largest():
    S, H, D = 2, 1, 8
    prev = _bits(np.zeros((S, H, D)))
    cur = np.zeros((S, H, D), np.float32)
    cur[0, 0, 0] = 1e30
    cb = _bits(cur)
    cb[1, 0, 0] = 0x7FC0                                   # NaN
    m = oracle.vmajor_metric(prev, cb, 1, 1)
    assert m.tolist() == [2 ** 32 - 1, 2 ** 32 - 1]


def test_metric_requires_units_inside_one_rank():
    v = _randn_bits((12, 2, 8), 3)
    with pytest.raises(ValueError):
        oracle.vmajor_metric(v, v, 3, 3)                   # S/P = 4, T = 3


# --------------------------------------------------------------- selection --
def _sorted_reference(metric, n_groups, r):
    n = len(metric)
    g = n // n_groups
    mask = np.ones(n, np.uint8)
    for grp in range(n_groups):
        members = sorted(range(grp * g, (grp + 1) * g), key=lambda i: (int(metric[i]), i))
        for i in members[:int(np.floor(r * g))]:
            mask[i] = 0
    return mask


@pytest.mark.parametrize("n,n_groups", [(144, 1), (144, 12), (60, 5), (7, 1), (64, 64)])
def test_selection_matches_sorted_reference_with_ties(n, n_groups):
    rng = np.random.default_rng(n * 31 + n_groups)
    for r in (0.0, 0.1, 0.5, 0.8, 0.999, 1.0):
        metric = rng.integers(0, 6, n).astype(np.uint64)         # many ties
        mask, idx, na = oracle.vmajor_select(metric, n_groups, r)
        want = _sorted_reference(metric, n_groups, r)
        assert np.array_equal(mask, want)
        assert np.array_equal(idx, np.flatnonzero(want)) and na == int(want.sum())
        g = n // n_groups
        assert na == n - n_groups * int(np.floor(r * g))


def test_selection_special_cases():
    metric = np.array([5, 1, 9, 1, 1, 7, 0, 3], np.uint64)
    mask, idx, na = oracle.vmajor_select(metric, 1, 0.0)     # r = 0: the full exchange
    assert mask.tolist() == [1] * 8 and idx.tolist() == list(range(8)) and na == 8
    mask, idx, na = oracle.vmajor_select(metric, 1, 1.0)     # r = 1: nothing is sent
    assert mask.tolist() == [0] * 8 and na == 0
    mask, idx, na = oracle.vmajor_select(metric, 1, 0.5)     # 4 smallest cached: 0,1,1,1
    assert mask.tolist() == [1, 0, 1, 0, 0, 1, 0, 1]
    mask, idx, na = oracle.vmajor_select(metric, 1, 0.375)   # 3 cached: the tie at 1 keeps lower indices
    assert mask.tolist() == [1, 0, 1, 0, 1, 1, 0, 1]
    same = np.full(6, 42, np.uint64)                         # all equal: lowest indices are cached
    mask, idx, na = oracle.vmajor_select(same, 2, 0.67)
    assert mask.tolist() == [0, 0, 1, 0, 0, 1]
    big = np.array([2 ** 63, 2 ** 63 + 1, 2 ** 40, 1], np.uint64)   # full 64-bit comparison
    mask, _, _ = oracle.vmajor_select(big, 1, 0.5)
    assert mask.tolist() == [1, 1, 0, 0]
    with pytest.raises(ValueError):
        oracle.vmajor_select(metric, 3, 0.5)
    with pytest.raises(ValueError):
        oracle.vmajor_select(metric, 1, 1.5)


def test_selection_finds_the_changed_tokens():
    """The most-changed (1 - r) of the units are the active ones."""
    S, H, D, T, P = 64, 2, 8, 4, 2
    rng = np.random.default_rng(5)
    prev = rng.normal(0, 1, (S, H, D)).astype(np.float32)
    cur = prev + rng.normal(0, 1e-3, prev.shape).astype(np.float32)
    changed = np.sort(rng.choice(S // T, 4, replace=False))
    for u in changed:
        cur[u * T:(u + 1) * T] += rng.normal(0, 0.5, (T, H, D)).astype(np.float32)
    m = oracle.vmajor_metric(_bits(prev), _bits(cur), P, T)
    mask, idx, na = oracle.vmajor_select(m, 1, 0.75)
    assert na == 4 and idx.tolist() == changed.tolist()


# ------------------------------------------------------ compaction, unpack --
@pytest.mark.parametrize("P,S,H,D,T", [(2, 16, 4, 8, 4), (3, 12, 3, 8, 1), (1, 8, 2, 8, 2), (4, 32, 4, 4, 8)])
def test_compaction_definition(P, S, H, D, T):
    x = _randn_bits((S, H, D), 6)
    n = S // T
    rng = np.random.default_rng(7)
    for k in (0, 1, n // 2, n):
        idx = np.sort(rng.choice(n, k, replace=False)).astype(np.int32)
        c = oracle.pack_active(x, idx, P, T)
        assert c.shape == (H, k * T, D)
        for h in range(H):
            for a in range(k):
                for j in range(T):
                    assert np.array_equal(c[h, a * T + j], x[idx[a] * T + j, h])


def test_compaction_with_all_units_is_the_full_exchange():
    P, S, H, D, T = 2, 16, 4, 8, 4
    x = _randn_bits((S, H, D), 8)
    c = oracle.pack_active(x, np.arange(S // T, dtype=np.int32), P, T)
    assert np.array_equal(c, oracle.ulysses_a2a(x, P))


def test_unpack_definition_and_idempotence():
    P, S, H, D, T = 2, 32, 4, 8, 4
    n = S // T
    cur = _randn_bits((S, H, D), 9)
    old = _randn_bits((H, S, D), 10)
    idx = np.array([1, 2, 6], np.int32)
    cache = old.copy()
    comp = oracle.pack_active(cur, idx, P, T)
    oracle.unpack(comp, idx, cache, P, T)
    active = np.zeros(n, bool)
    active[idx] = True
    for h in range(H):
        for s in range(S):
            want = cur[s, h] if active[s // T] else old[h, s]
            assert np.array_equal(cache[h, s], want)
    again = cache.copy()
    oracle.unpack(comp, idx, again, P, T)
    assert np.array_equal(again, cache)
    # r = 1: nothing active, every cached bit survives
    guard = old.copy()
    oracle.unpack(np.empty((H, 0, D), np.uint16), np.empty(0, np.int32), guard, P, T)
    assert np.array_equal(guard, old)
    # r = 0 over garbage equals the full exchange
    full = _randn_bits((H, S, D), 11)
    allidx = np.arange(n, dtype=np.int32)
    oracle.unpack(oracle.pack_active(cur, allidx, P, T), allidx, full, P, T)
    assert np.array_equal(full, oracle.ulysses_a2a(cur, P))


def test_prologue_is_the_composition():
    cfg = synth.config("tiny")
    L = synth.make_layer(cfg)
    cs = oracle.rope_table_2d(L["pos"], cfg["D"], cfg["theta"])
    qh, kh, vh = oracle.prologue(L["q"], L["k"], L["v"], L["wq"], L["wk"], cfg["eps"], cs, cfg["P"])
    assert np.array_equal(vh, L["v"].transpose(1, 0, 2))        # V is only moved
    assert np.array_equal(qh, oracle.norm_rope(L["q"], L["wq"], cfg["eps"], cs).transpose(1, 0, 2))
    assert np.array_equal(kh, oracle.norm_rope(L["k"], L["wk"], cfg["eps"], cs).transpose(1, 0, 2))
    assert not np.array_equal(qh, kh)


def test_two_readings_of_the_cached_v_give_the_same_masks():
    """What "the cached v" of the selection rule holds is not fixed by the paper.
    Reading A: V of the previous step, refreshed every step (V's Phase 1 is full-size).
    Reading B: the receivers' copy, refreshed only on the units that were sent.
    On data that follow the temporal law of the workload (small noise everywhere, a
    fifth of the tiles strongly perturbed, re-drawn every step) both readings select
    the same units at every step, and the cache differs from the exact tensor only
    on units that were never sent, by no more than the accumulated small noise."""
    cfg = synth.config("temporal")
    cfg.update(grid=(32, 24), P=4, H=4, D=64, T=16, steps=8)
    cfg["S"] = 32 * 24
    P, S, H, D, T, r = cfg["P"], cfg["S"], cfg["H"], cfg["D"], cfg["T"], cfg["r"]
    n = S // T
    seq = synth.TemporalSequence(cfg)
    v0 = seq.current()["v"]
    prev_a = v0.copy()
    prev_b = v0.copy()                              # SEQ-layout view of what the receivers hold
    cache = oracle.ulysses_a2a(v0, P)               # step 0: full exchange
    ever_sent = np.zeros(n, bool)
    for step in range(1, cfg["steps"]):
        hot = seq.advance()
        v = seq.current()["v"]
        mask_a, idx_a, _ = oracle.vmajor_select(oracle.vmajor_metric(prev_a, v, P, T), cfg["n_groups"], r)
        mask_b, idx_b, _ = oracle.vmajor_select(oracle.vmajor_metric(prev_b, v, P, T), cfg["n_groups"], r)
        assert np.array_equal(mask_a, mask_b), step
        assert np.array_equal(idx_a, hot)
        oracle.unpack(oracle.pack_active(v, idx_b, P, T), idx_b, cache, P, T)
        tok = (idx_b[:, None] * T + np.arange(T)[None, :]).reshape(-1)
        prev_b[tok] = v[tok]
        prev_a = v
        ever_sent[idx_b] = True
        assert np.array_equal(oracle.ulysses_a2a_inverse(cache, P), prev_b), "reading B is the receivers' copy"
        exact = oracle.ulysses_a2a(v, P)
        stale_tok = (cache != exact).any(axis=(0, 2))
        sent_now = np.zeros(S, bool)
        sent_now[tok] = True
        assert not (stale_tok & sent_now).any(), "a unit sent in this step is exact"
        c64, e64 = synth.bf16_bits_to_f32(cache).astype(np.float64), synth.bf16_bits_to_f32(exact).astype(np.float64)
        one_ulp = np.exp2(np.floor(np.log2(np.maximum(np.maximum(np.abs(c64), np.abs(e64)), 2.0 ** -100))) - 7.0)
        # the accumulated small noise, plus the one bf16 step by which it can move a rounding
        assert np.all(np.abs(c64 - e64) <= 6 * cfg["sigma_small"] * np.sqrt(step) + one_ulp), "only accumulated small noise"
    assert 0 < ever_sent.sum() < n
