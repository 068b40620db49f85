"""Pins for the oracle's time-varying cache schedule (Section III-D): the
paper's experimental setting (50 steps, 5 warm-up steps, full refresh every 10
steps) and the properties its text fixes."""
import pytest

import oracle


def test_paper_setting_50_steps_warmup_5_refresh_10():
    sched = [oracle.cache_schedule(t, 50, 5, 10) for t in range(50)]
    full = [t for t, (f, _) in enumerate(sched) if f]
    assert full == [0, 1, 2, 3, 4, 10, 20, 30, 40]        # warm-up, then every 10th step
    assert all(r == 0.0 for f, r in sched if f)            # a full step sends everything
    sel = [(t, r) for t, (f, r) in enumerate(sched) if not f]
    assert sel[0] == (5, 0.0)                              # r starts at 0 at the warm-up boundary
    assert sel[-1] == (49, 1.0)                            # and reaches 1 at the last step
    for (t0, r0), (t1, r1) in zip(sel, sel[1:]):
        assert r1 > r0                                      # caching grows with the step
        assert abs((r1 - r0) / (t1 - t0) - 1.0 / 44.0) < 1e-12   # linearly


def test_degenerate_settings():
    assert oracle.cache_schedule(0, 1, 0, 0) == (False, 0.0)
    assert [oracle.cache_schedule(t, 4, 0, 0) for t in range(4)] == [(False, 0.0), (False, 1 / 3), (False, 2 / 3), (False, 1.0)]
    assert all(oracle.cache_schedule(t, 6, 6, 0)[0] for t in range(6))      # warm-up covers everything
    assert all(oracle.cache_schedule(t, 6, 0, 1)[0] for t in range(6))      # refresh at every step
    with pytest.raises(ValueError):
        oracle.cache_schedule(7, 5, 1, 0)
    with pytest.raises(ValueError):
        oracle.cache_schedule(-1, 5, 1, 0)
