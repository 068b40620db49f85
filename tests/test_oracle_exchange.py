"""Pins for the oracle's Ulysses exchange (Section II-A of the paper).

None of these re-types the oracle's message loops: the closed form is a plain
axis swap, the index-fill test checks destination addresses arithmetically and
the size pins are numbers printed in the paper (tests/golden/paper_sizes.txt).
"""
import os

import numpy as np
import pytest

import oracle


def _rand_bits(shape, seed):
    return np.random.default_rng(seed).integers(0, 1 << 16, size=shape, dtype=np.uint16)


def _valid_P(S, H):
    return [p for p in range(1, H + 1) if S % p == 0 and H % p == 0]


@pytest.mark.parametrize("S,H,D", [(12, 6, 8), (8, 4, 16), (30, 6, 8), (24, 12, 4)])
def test_closed_form_for_every_P(S, H, D):
    """Each rank ends with all tokens of its H/P heads, tokens in global order:
    HEAD[h][s] = SEQ[s][h], whatever P is."""
    x = _rand_bits((S, H, D), 1)
    for P in _valid_P(S, H):
        got = oracle.ulysses_a2a(x, P)
        assert np.array_equal(got, x.transpose(1, 0, 2)), P


def test_rank_view_of_the_result():
    """Rank p's slice of the HEAD tensor is [H/P][S][D]: heads p*H/P.. of every
    token, and the slab received from source rank q holds q's tokens."""
    P, S, H, D = 3, 12, 6, 4
    x = _rand_bits((S, H, D), 2)
    head = oracle.ulysses_a2a(x, P).reshape(P, H // P, S, D)
    seq = x.reshape(P, S // P, H, D)
    for dst in range(P):
        for src in range(P):
            for hl in range(H // P):
                for sl in range(S // P):
                    assert np.array_equal(head[dst, hl, src * (S // P) + sl],
                                          seq[src, sl, dst * (H // P) + hl])


@pytest.mark.parametrize("P", [1, 2, 4])
def test_bijection_both_ways(P):
    S, H, D = 16, 8, 8
    x = _rand_bits((S, H, D), 3)
    assert np.array_equal(oracle.ulysses_a2a_inverse(oracle.ulysses_a2a(x, P), P), x)
    y = _rand_bits((H, S, D), 4)
    assert np.array_equal(oracle.ulysses_a2a(oracle.ulysses_a2a_inverse(y, P), P), y)


def test_p1_moves_no_data_between_ranks_and_h1_is_a_copy():
    x = _rand_bits((10, 1, 8), 5)
    assert np.array_equal(oracle.ulysses_a2a(x, 1).reshape(-1), x.reshape(-1))
    x = _rand_bits((10, 3, 8), 6)
    assert np.array_equal(oracle.ulysses_a2a(x, 1), x.transpose(1, 0, 2))


def test_index_fill_addresses():
    """Fill every D-vector with its own (token, head); check where each lands."""
    P, S, H, D = 4, 16, 8, 2
    x = np.zeros((S, H, D), dtype=np.uint16)
    x[:, :, 0] = np.arange(S, dtype=np.uint16)[:, None]
    x[:, :, 1] = np.arange(H, dtype=np.uint16)[None, :]
    flat = oracle.ulysses_a2a(x, P).reshape(-1, D)
    for row, (s, h) in enumerate(flat):
        rank, rem = divmod(row, (H // P) * S)
        hl, tok = divmod(rem, S)
        assert (s, h) == (tok, rank * (H // P) + hl)


def test_bad_shapes_rejected():
    x = _rand_bits((10, 4, 8), 7)
    with pytest.raises(ValueError):
        oracle.ulysses_a2a(x, 3)


def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_sizes.txt")
    rows = {}
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        name, shape, extra, expected, _cite = [f.strip() for f in line.split("|")]
        rows[name] = (shape, extra, float(expected))
    return rows


def test_sizes_printed_in_the_paper():
    g = _golden()
    P, S, H, D = map(int, g["cache_mib"][0].split())
    per_tensor = oracle.head_shard_elems(P, S, H, D) * 2
    mib = 4 * per_tensor * 60 * 4 / 2 ** 20
    assert mib == g["cache_mib"][2]
    assert round(100 * mib / 65536, 1) == g["cache_pct_of_64gib"][2]
    msg_mb = 3 * oracle.seq_shard_elems(P, S, H, D) * 2 / 1e6
    assert round(msg_mb) == g["phase1_message_mb"][2]
    from paper_2604_14561_b200 import synth
    assert synth.config("qwen768")["grid"][0] == g["grid_768"][2]
    assert synth.config("temporal")["grid"][0] == g["grid_1536"][2]
    assert synth.config("qwen2304")["grid"][0] == g["grid_2304"][2]


# ------------------------------------------------- TAPA (Section III-B) -----
@pytest.mark.parametrize("P,S,H,D", [(2, 8, 2, 4), (4, 16, 4, 8), (6, 24, 12, 4), (12, 48, 12, 8)])
def test_tapa_phase1_every_tile_holds_its_gpus_tokens(P, S, H, D):
    x = _rand_bits((S, H, D), 20)
    p1 = oracle.tapa_phase1(x, P).reshape(2, P // 2, 2 * S // P, H, D)
    Sg = 2 * S // P
    for t in range(2):
        for g in range(P // 2):
            assert np.array_equal(p1[t, g], x[g * Sg:(g + 1) * Sg])
    # so each ring's copies, taken together, are the whole sequence-parallel tensor again
    assert np.array_equal(oracle.tapa_phase1(x, P)[0], x) and np.array_equal(oracle.tapa_phase1(x, P)[1], x)


@pytest.mark.parametrize("P,S,H,D", [(2, 8, 2, 4), (4, 16, 4, 8), (6, 24, 12, 4), (12, 48, 24, 8)])
def test_tapa_phases_compose_to_the_flat_exchange(P, S, H, D):
    x = _rand_bits((S, H, D), 21)
    got = oracle.tapa_phase2(oracle.tapa_phase1(x, P), P)
    assert np.array_equal(got, x.transpose(1, 0, 2))
    assert np.array_equal(got, oracle.ulysses_a2a(x, P))


def test_tapa_rings_are_independent():
    """Phase 2 runs one all-to-all per ring with no traffic between them:
    ranks of ring 0 depend only on the copies held by ring 0."""
    P, S, H, D = 4, 16, 8, 4
    x = _rand_bits((S, H, D), 22)
    p1 = oracle.tapa_phase1(x, P)
    base = oracle.tapa_phase2(p1, P).reshape(P, H // P, S, D)
    p1b = p1.copy()
    p1b[1] ^= np.uint16(0xFFFF)                       # corrupt everything ring 1 holds
    got = oracle.tapa_phase2(p1b, P).reshape(P, H // P, S, D)
    for r in range(P):
        same = np.array_equal(got[r], base[r])
        assert same == (r % 2 == 0), r


def test_tapa_needs_an_even_rank_count_and_its_message_is_the_whole_shard():
    with pytest.raises(ValueError):
        oracle.tapa_phase1(_rand_bits((9, 3, 4), 23), 3)
    g = _golden()
    P, S, H, D = map(int, g["phase1_message_mb"][0].split())
    # a tile sends its S/P tokens with all heads, for Q, K and V: the 14 MB message size of Section III-B
    assert round(3 * (S // P) * H * D * 2 / 1e6) == g["phase1_message_mb"][2]
