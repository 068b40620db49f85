"""Pins for the oracle's QK RMSNorm and 2-D RoPE (Section II-B of the paper).

Properties and special cases that the mathematics fixes: unit RMS, power-of-two
scale invariance, a 3-4-5 hand case, identity at position 0, pair-norm
preservation, the relative-position property the paper states for RoPE, a
quarter turn, axis separation, the complex-multiplication form of 1-D RoPE,
and angles with closed-form frequencies (theta^(-1/4) = 0.1 ...).
"""
import numpy as np
import pytest

import oracle
from paper_2604_14561_b200 import synth

from helpers import bits_to_f32


def _bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _randn_bits(shape, seed, std=1.0):
    return _bits(np.random.default_rng(seed).normal(0, std, size=shape))


def _identity_cs(S, D):
    cs = np.zeros((S, D // 2, 2), np.float32)
    cs[..., 0] = 1.0
    return cs


# ----------------------------------------------------------------- RMSNorm --
def test_unit_rms_with_constant_weight():
    S, H, D = 7, 3, 64
    x = _randn_bits((S, H, D), 0, std=3.0)
    for c in (1.0, 0.5, 2.0):
        w = _bits(np.full(D, c))
        _, yf = oracle.norm_rope(x, w, 1e-6, None, want_f32=True)
        rms = np.sqrt((yf.astype(np.float64) ** 2).mean(axis=-1))
        assert np.allclose(rms, c, rtol=2e-6)
        y = bits_to_f32(oracle.norm_rope(x, w, 1e-6, None)).astype(np.float64)
        assert np.allclose(np.sqrt((y ** 2).mean(axis=-1)), c, rtol=2.0 ** -8)


def test_power_of_two_scale_invariance():
    S, H, D = 5, 2, 32
    x = _randn_bits((S, H, D), 1)
    w = _randn_bits((D,), 2) 
    base = oracle.norm_rope(x, w, 0.0, None)
    for a in (0.25, 2.0, 64.0):
        xa = _bits(bits_to_f32(x) * np.float32(a))       # exact in bf16
        assert np.array_equal(oracle.norm_rope(xa, w, 0.0, None), base)


def test_three_four_five_hand_case():
    D = 8
    x = np.zeros((1, 1, D), np.float32)
    x[0, 0, 0], x[0, 0, 1] = 3.0, 4.0              # mean square = 25/8
    w = _bits(np.array([1, 2, 1, 1, 1, 1, 1, 1], np.float32))
    _, yf = oracle.norm_rope(_bits(x), w, 0.0, None, want_f32=True)
    inv = 1.0 / np.sqrt(25.0 / 8.0)
    assert np.allclose(yf[0, 0, :3], [3 * inv, 2 * 4 * inv, 0.0], rtol=1e-6)
    # eps sits inside the square root: with x = 0 the output is 0, not NaN
    _, z = oracle.norm_rope(_bits(np.zeros((1, 1, D))), w, 1e-6, None, want_f32=True)
    assert np.all(z == 0.0)
    # and a large eps shrinks the result by sqrt(ms / (ms + eps))
    _, ye = oracle.norm_rope(_bits(x), w, 25.0 / 8.0, None, want_f32=True)
    assert np.allclose(ye[0, 0, 0], 3 * inv / np.sqrt(2.0), rtol=1e-6)


def test_against_fp64_textbook_rmsnorm():
    S, H, D = 9, 4, 128
    x = _randn_bits((S, H, D), 3)
    w = _bits(np.random.default_rng(4).normal(1, 0.1, D))
    _, yf = oracle.norm_rope(x, w, 1e-6, None, want_f32=True)
    xd = bits_to_f32(x).astype(np.float64)
    ref = xd / np.sqrt((xd ** 2).mean(-1, keepdims=True) + 1e-6) * bits_to_f32(w).astype(np.float64)
    assert np.allclose(yf, ref, rtol=4e-7, atol=1e-9)
    # rows are normalised one (token, head) at a time: changing one row leaves the others alone
    x2 = x.copy()
    x2[2, 1] = _randn_bits((D,), 5, std=10.0)
    y1, y2 = oracle.norm_rope(x, w, 1e-6, None), oracle.norm_rope(x2, w, 1e-6, None)
    same = np.ones((S, H), bool)
    same[2, 1] = False
    assert np.array_equal(y1[same], y2[same]) and not np.array_equal(y1[2, 1], y2[2, 1])


def test_v_is_untouched_without_weight_and_table():
    x = _randn_bits((4, 2, 16), 6)
    assert np.array_equal(oracle.norm_rope(x, None, 1e-6, None), x)


# -------------------------------------------------------------------- RoPE --
def test_table_closed_form_angles():
    """theta = 10000: frequency i of an axis is theta^(-2i/(D/2)), so for
    D = 64 (16 pairs per axis) i = 4 -> 0.1 and i = 8 -> 0.01; for D = 128,
    i = 8 -> 0.1, i = 16 -> 0.01, i = 24 -> 0.001."""
    pos = np.array([[10, 100], [0, 0], [1, 0], [0, 1]], np.int32)
    cs = oracle.rope_table_2d(pos, 64, 10000.0)
    one = (np.float32(np.cos(1.0)), np.float32(np.sin(1.0)))
    assert np.allclose(cs[0, 4], one, atol=1e-6)              # row 10 * 0.1
    assert np.allclose(cs[0, 16 + 8], one, atol=1e-6)         # col 100 * 0.01
    assert np.allclose(cs[0, 0], (np.cos(10.0), np.sin(10.0)), atol=1e-6)   # i = 0: freq 1, row axis
    assert np.allclose(cs[0, 16], (np.cos(100.0), np.sin(100.0)), atol=1e-6)  # i = 0, col axis
    assert np.all(cs[1, :, 0] == 1.0) and np.all(cs[1, :, 1] == 0.0)
    # row position drives pairs [0, D/4), column position pairs [D/4, D/2)
    assert np.all(cs[2, 16:, 1] == 0.0) and cs[2, 0, 1] == np.float32(np.sin(1.0))
    assert np.all(cs[3, :16, 1] == 0.0) and cs[3, 16, 1] == np.float32(np.sin(1.0))
    cs128 = oracle.rope_table_2d(np.array([[10, 1000]], np.int32), 128, 10000.0)
    assert np.allclose(cs128[0, 8], one, atol=1e-6)
    assert np.allclose(cs128[0, 32 + 24], one, atol=1e-6)
    assert np.allclose(cs128[0, 32 + 16], (np.cos(10.0), np.sin(10.0)), atol=2e-6)
    # frequencies fall monotonically inside an axis
    ang = np.arctan2(cs128[0, :32, 1].astype(np.float64), cs128[0, :32, 0])
    assert ang[31] > 0 and ang[31] < 0.02


def test_position_zero_is_identity():
    S, H, D = 3, 2, 64
    x = _randn_bits((S, H, D), 7)
    w = _randn_bits((D,), 8)
    cs = oracle.rope_table_2d(np.zeros((S, 2), np.int32), D, 10000.0)
    assert np.array_equal(oracle.norm_rope(x, w, 1e-6, cs), oracle.norm_rope(x, w, 1e-6, None))
    assert np.array_equal(oracle.norm_rope(x, w, 1e-6, _identity_cs(S, D)),
                          oracle.norm_rope(x, w, 1e-6, None))


def test_pair_norm_is_preserved():
    S, H, D = 6, 2, 64
    x = _randn_bits((S, H, D), 9)
    w = _randn_bits((D,), 10)
    pos = np.random.default_rng(11).integers(0, 150, (S, 2)).astype(np.int32)
    cs = oracle.rope_table_2d(pos, D, 10000.0)
    _, plain = oracle.norm_rope(x, w, 1e-6, None, want_f32=True)
    _, rot = oracle.norm_rope(x, w, 1e-6, cs, want_f32=True)
    n0 = (plain.astype(np.float64).reshape(S, H, D // 2, 2) ** 2).sum(-1)
    n1 = (rot.astype(np.float64).reshape(S, H, D // 2, 2) ** 2).sum(-1)
    assert np.allclose(n0, n1, rtol=1e-6, atol=1e-12)


def test_quarter_turn_and_half_turn():
    S, H, D = 1, 1, 8
    x = _bits(np.arange(1, D + 1, dtype=np.float32).reshape(S, H, D))
    cs = np.zeros((S, D // 2, 2), np.float32)
    cs[..., 1] = 1.0                                   # cos 0, sin 1: (a, b) -> (-b, a)
    got = bits_to_f32(oracle.norm_rope(x, None, 0.0, cs))
    assert got.reshape(-1).tolist() == [-2, 1, -4, 3, -6, 5, -8, 7]
    cs[..., 0], cs[..., 1] = -1.0, 0.0                 # half turn: (a, b) -> (-a, -b)
    got = bits_to_f32(oracle.norm_rope(x, None, 0.0, cs))
    assert got.reshape(-1).tolist() == [-1, -2, -3, -4, -5, -6, -7, -8]


def test_axes_are_separate():
    S, H, D = 4, 2, 64
    x = _randn_bits((S, H, D), 12)
    w = _randn_bits((D,), 13)
    plain = oracle.norm_rope(x, w, 1e-6, None)
    rows_only = np.stack([np.arange(1, S + 1), np.zeros(S)], 1).astype(np.int32)
    cols_only = rows_only[:, ::-1].copy()
    r = oracle.norm_rope(x, w, 1e-6, oracle.rope_table_2d(rows_only, D, 10000.0))
    c = oracle.norm_rope(x, w, 1e-6, oracle.rope_table_2d(cols_only, D, 10000.0))
    assert np.array_equal(r[..., D // 2:], plain[..., D // 2:]) and not np.array_equal(r[..., :D // 2], plain[..., :D // 2])
    assert np.array_equal(c[..., :D // 2], plain[..., :D // 2]) and not np.array_equal(c[..., D // 2:], plain[..., D // 2:])


def test_relative_position_property():
    """q_i . k_j depends on the positions only through their difference
    (the property the paper states): shifting every position by a constant
    leaves all dot products unchanged."""
    S, H, D = 8, 1, 64
    q, k = _randn_bits((S, H, D), 14), _randn_bits((S, H, D), 15)
    w = _bits(np.ones(D))
    pos = np.random.default_rng(16).integers(0, 40, (S, 2)).astype(np.int32)
    dots = []
    for shift in ((0, 0), (17, 0), (5, 29)):
        cs = oracle.rope_table_2d(pos + np.array(shift, np.int32), D, 10000.0)
        _, qf = oracle.norm_rope(q, w, 1e-6, cs, want_f32=True)
        _, kf = oracle.norm_rope(k, w, 1e-6, cs, want_f32=True)
        dots.append(qf[:, 0].astype(np.float64) @ kf[:, 0].astype(np.float64).T)
    assert np.allclose(dots[0], dots[1], rtol=0, atol=2e-4)
    assert np.allclose(dots[0], dots[2], rtol=0, atol=2e-4)
    # and they do depend on the difference
    cs = oracle.rope_table_2d(pos, D, 10000.0)
    _, qf = oracle.norm_rope(q, w, 1e-6, cs, want_f32=True)
    _, k0 = oracle.norm_rope(k, w, 1e-6, None, want_f32=True)
    assert not np.allclose(dots[0], qf[:, 0].astype(np.float64) @ k0[:, 0].astype(np.float64).T, atol=1e-2)


@pytest.mark.parametrize("D", [32, 64, 128])
def test_one_d_positions_match_complex_form(D):
    """Text tokens carry pos = (j, j): each half of the head is then a 1-D
    RoPE of dimension D/2, i.e. pair p of a half is multiplied, as the complex
    number a + ib, by exp(i * j * theta^(-2p/(D/2)))."""
    S, H = 12, 2
    x = _randn_bits((S, H, D), 17)
    j = np.arange(S, dtype=np.int32) * 3
    cs = oracle.rope_table_2d(np.stack([j, j], 1), D, 10000.0)
    _, got = oracle.norm_rope(x, None, 0.0, cs, want_f32=True)
    xd = bits_to_f32(x).astype(np.float64).reshape(S, H, 2, D // 4, 2)      # [.., half, pair, (re, im)]
    z = xd[..., 0] + 1j * xd[..., 1]
    freq = 10000.0 ** (-2.0 * np.arange(D // 4) / (D // 2))
    rot = z * np.exp(1j * j[:, None, None, None].astype(np.float64) * freq)
    ref = np.stack([rot.real, rot.imag], -1).reshape(S, H, D)
    assert np.allclose(got, ref, rtol=0, atol=2e-6)


def test_final_rounding_is_single_rne():
    """The bf16 result is the fp32 result rounded once, to nearest even."""
    S, H, D = 5, 3, 64
    x = _randn_bits((S, H, D), 18)
    w = _randn_bits((D,), 19)
    pos = np.random.default_rng(20).integers(0, 99, (S, 2)).astype(np.int32)
    cs = oracle.rope_table_2d(pos, D, 10000.0)
    y, yf = oracle.norm_rope(x, w, 1e-6, cs, want_f32=True)
    assert np.array_equal(y, synth.f32_to_bf16_bits(yf))
    for bits in (0x0000, 0x3F80, 0xBF81, 0x7F7F, 0x0001, 0x8000):
        assert oracle.f32_to_bf16(oracle.bf16_to_f32(bits)) == bits
    assert oracle.f32_to_bf16(1.00390625) == 0x3F80       # midpoint between 1.0 and 1.0078125 -> even
    assert oracle.f32_to_bf16(1.01171875) == 0x3F82       # midpoint above 0x3F81 -> even
