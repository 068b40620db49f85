"""The seeded input generator: determinism, counter addressing, distributions."""
import numpy as np

from paper_2604_14561_b200 import synth


def test_streams_are_counter_based_and_independent():
    a = synth.normal_f32(0, "q", 1000)
    b = synth.normal_f32(0, "q", 5_000_000)[:1000]   # spans several chunks
    assert np.array_equal(a, b)
    assert not np.array_equal(a, synth.normal_f32(0, "k", 1000))
    assert not np.array_equal(a, synth.normal_f32(1, "q", 1000))


def test_normal_moments():
    x = synth.normal_f32(3, "v", 1_000_000).astype(np.float64)
    assert abs(x.mean()) < 5e-3 and abs(x.std() - 1.0) < 5e-3
    w = synth.bf16_bits_to_f32(synth.normal_bf16(3, "wq", 100_000, 1.0, 0.1)).astype(np.float64)
    assert abs(w.mean() - 1.0) < 2e-3 and abs(w.std() - 0.1) < 2e-3


def test_bf16_rounding_is_rne_and_roundtrips():
    bits = np.arange(0, 0x7F80, dtype=np.uint16)            # all finite non-negative bf16
    f = synth.bf16_bits_to_f32(bits)
    assert np.array_equal(synth.f32_to_bf16_bits(f), bits)
    # exact midpoints go to the even neighbour
    lo = synth.bf16_bits_to_f32(np.array([0x3F80, 0x3F81], dtype=np.uint16))   # 1.0, 1.0078125
    mid = np.float32((float(lo[0]) + float(lo[1])) / 2)
    assert synth.f32_to_bf16_bits(np.array([mid]))[0] == 0x3F80
    hi = synth.bf16_bits_to_f32(np.array([0x3F82], dtype=np.uint16))
    mid2 = np.float32((float(lo[1]) + float(hi[0])) / 2)
    assert synth.f32_to_bf16_bits(np.array([mid2]))[0] == 0x3F82


def test_positions_and_configs():
    pos = synth.positions(3, 4, 2)
    assert pos.tolist() == [[0, 0], [0, 1], [0, 2], [0, 3], [1, 0], [1, 1], [1, 2], [1, 3],
                            [2, 0], [2, 1], [2, 2], [2, 3], [0, 0], [1, 1]]
    want_S = dict(tiny=256, sd3=4352, qwen768=2560, qwen2304=21024, temporal=9216)
    for name, S in want_S.items():
        c = synth.config(name)
        assert c["S"] == S and c["S"] % c["P"] == 0 and c["H"] % c["P"] == 0
    t = synth.config("temporal")
    assert (t["S"] // t["P"]) % t["T"] == 0 and t["S"] // t["T"] == 144


def test_temporal_sequence_perturbs_the_drawn_tiles():
    cfg = dict(synth.config("temporal"), grid=(16, 16), P=2, H=2, D=32, T=16)
    cfg["S"] = 256
    seq = synth.TemporalSequence(cfg)
    before = {n: seq.master[n].copy() for n in "qkv"}
    large = seq.advance()
    n = cfg["S"] // cfg["T"]
    assert len(large) == int(np.ceil(0.2 * n)) and np.all(np.diff(large) > 0)
    again = synth.perturbed_tiles(cfg["seed"], 1, n, 0.2)
    assert np.array_equal(large, again)
    for name in "qkv":
        d = np.abs(seq.master[name] - before[name]).reshape(n, -1).mean(axis=1)
        big = np.zeros(n, bool)
        big[large] = True
        assert d[big].min() > 0.2 and d[~big].max() < 5e-3
    assert not np.array_equal(large, synth.perturbed_tiles(cfg["seed"], 2, n, 0.2))
