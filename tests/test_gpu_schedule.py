"""The time-varying cache schedule driven through the GPU path, step by step
against the oracle: warm-up, linearly growing cache ratio, periodic refresh.
Reports what the policy saves (elements crossing the exchange) and the drift of
the cached tensors from the exact ones, which a refresh step resets to zero."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle
from paper_2604_14561_b200 import binding, synth

from gpu_util import Guarded, dev, rope_table
from helpers import assert_norm_rope_close


def test_schedule_driver_against_oracle():
    cfg = synth.config("temporal")
    cfg.update(grid=(24, 16), P=4, H=4, D=64, T=16)
    cfg["S"] = 24 * 16
    P, S, H, D, T = cfg["P"], cfg["S"], cfg["H"], cfg["D"], cfg["T"]
    E, n = S * H * D, S // T
    total, warmup, interval, n_groups = 14, 2, 6, 2
    seq = synth.TemporalSequence(cfg)
    cs_ref, cs = oracle.rope_table_2d(seq.pos, D, cfg["theta"]), rope_table(seq.pos, D, cfg["theta"])
    wq, wk = dev(seq.wq), dev(seq.wk)
    cache = {x: Guarded(E) for x in "qkv"}
    comp = {x: Guarded(E) for x in "qkv"}
    cache_ref = {x: np.zeros((H, S, D), np.uint16) for x in "qkv"}
    metric = torch.zeros(n, dtype=torch.int64, device="cuda")
    mask = torch.zeros(n, dtype=torch.uint8, device="cuda")
    idx = torch.zeros(n, dtype=torch.int32, device="cuda")
    na = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws_bytes = binding.vmajor_workspace_bytes(P, S, H, D, T)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    sq, sv = torch.cuda.Stream(), torch.cuda.Stream()
    prev_v = None
    sent_total, drift = 0, []
    for step in range(total):
        if step:
            seq.advance()
        cur = seq.current()
        d = {x: dev(cur[x]) for x in "qkv"}
        full, r = binding.cache_schedule(step, total, warmup, interval)
        assert (full, r) == oracle.cache_schedule(step, total, warmup, interval)
        torch.cuda.synchronize()
        _, sent = binding.layer_step(step, total, warmup, interval, dev(prev_v) if prev_v is not None else d["v"],
                                     d["q"], d["k"], d["v"], wq, wk, cfg["eps"], cs, P, S, H, D, T, n_groups,
                                     metric, mask, idx, na, *([None] * 3 if step % 2 else [comp[x].t for x in "qkv"]),
                                     cache["q"].t, cache["k"].t, cache["v"].t, ws, ws_bytes,
                                     order=binding.V_FIRST, stream_qk=sq, stream_v=sv)     # odd steps: direct delivery
        sq.synchronize()
        exact = dict(zip("qkv", oracle.prologue(cur["q"], cur["k"], cur["v"], seq.wq, seq.wk, cfg["eps"], cs_ref, P)))
        if full:
            assert sent == 3 * E
            tok = np.arange(S)
            for x in "qkv":
                cache_ref[x] = exact[x].copy()
        else:
            m_ref = oracle.vmajor_metric(prev_v, cur["v"], P, T)
            mask_ref, idx_ref, na_ref = oracle.vmajor_select(m_ref, n_groups, r)
            assert sent == 3 * na_ref * T * H * D
            assert int(na.item()) == na_ref and np.array_equal(idx.cpu().numpy()[:na_ref], idx_ref)
            assert np.array_equal(mask.cpu().numpy(), mask_ref)
            tok = (idx_ref[:, None] * T + np.arange(T)[None, :]).reshape(-1)
            for x in "qkv":     # the oracle extracts from the exact tensors and scatters
                seq_layout = np.ascontiguousarray(exact[x].transpose(1, 0, 2))
                oracle.unpack(oracle.pack_active(seq_layout, idx_ref, P, T), idx_ref, cache_ref[x], P, T)
        sent_total += sent
        untouched = np.ones(S, bool)
        untouched[tok] = False
        for x in "qkv":
            got = cache[x].host((H, S, D))
            assert np.array_equal(got[:, untouched], cache_ref[x][:, untouched]), (x, step)
            if x == "v":
                assert np.array_equal(got, cache_ref[x]), step
            elif len(tok):
                _, f = oracle.norm_rope(cur[x], seq.wq if x == "q" else seq.wk, cfg["eps"], cs_ref, want_f32=True)
                assert_norm_rope_close(got[:, tok], cache_ref[x][:, tok], np.ascontiguousarray(f[tok].transpose(1, 0, 2)),
                                       f"{x} step {step}")
                cache[x].t.copy_(dev(cache_ref[x]).reshape(-1))      # keep both sides bit-aligned
            cache[x].assert_guards()
        stale = float((cache_ref["v"] != exact["v"]).any(axis=(0, 2)).mean())
        drift.append(stale)
        if full:
            assert stale == 0.0, "a full step resets the cache to the exact values"
        prev_v = cur["v"]
    assert drift[-1] > 0.5 and drift[warmup] == 0.0        # r -> 1: almost nothing is refreshed at the end
    assert sent_total < 0.75 * total * 3 * E                # the schedule saves traffic over always-full
