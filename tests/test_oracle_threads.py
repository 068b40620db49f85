"""The oracle built with OpenMP (the benchmark's all-cores CPU baseline) computes
exactly what the single-threaded build computes."""
import numpy as np

import oracle
from paper_2604_14561_b200 import synth


def test_all_cores_build_is_bit_identical():
    cfg = synth.config("tiny")
    L = synth.make_layer(cfg)
    cs = oracle.rope_table_2d(L["pos"], cfg["D"], cfg["theta"])
    rng = np.random.default_rng(0)
    other = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(L["v"]) + rng.normal(0, 0.1, L["v"].shape).astype(np.float32))
    one = oracle.prologue(L["q"], L["k"], L["v"], L["wq"], L["wk"], cfg["eps"], cs, cfg["P"])
    m_one = oracle.vmajor_metric(L["v"], other, cfg["P"], 4)
    try:
        oracle.use_all_cores(True)
        many = oracle.prologue(L["q"], L["k"], L["v"], L["wq"], L["wk"], cfg["eps"], cs, cfg["P"])
        m_many = oracle.vmajor_metric(L["v"], other, cfg["P"], 4)
    finally:
        oracle.use_all_cores(False)
    for a, b in zip(one, many):
        assert np.array_equal(a, b)
    assert np.array_equal(m_one, m_many) and m_one.any()
