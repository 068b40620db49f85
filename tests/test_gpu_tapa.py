"""GPU parity of the two-phase (TAPA) exchange on virtual ranks against the
oracle: both phases bit-exact, their composition equal to the flat exchange,
rings independent, and the paper's per-GPU selection scope run on what a tile
holds after Phase 1 of V."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle
from paper_2604_14561_b200 import binding, synth

from gpu_util import Guarded, dev, u16


@pytest.mark.parametrize("P,S,H,D", [(2, 256, 4, 64), (4, 1000, 8, 128), (12, 1752, 24, 128), (6, 66, 6, 32), (8, 320, 16, 256),
                                      (2, 130, 4, 96), (4, 36, 4, 8), (2, 50, 2, 200),
                                      (24, 9216, 24, 128)])      # the size the benchmark times
def test_two_phases_match_oracle_and_flat_exchange(P, S, H, D):
    E = S * H * D
    x = {t: synth.normal_bf16(3, t, E).reshape(S, H, D) for t in "qkv"}
    d = {t: dev(x[t]) for t in "qkv"}
    p1 = {t: Guarded(2 * E) for t in "qkv"}
    head = {t: Guarded(E) for t in "qkv"}
    flat = {t: Guarded(E) for t in "qkv"}
    binding.tapa_phase1(d["q"], d["k"], d["v"], p1["q"].t, p1["k"].t, p1["v"].t, P, S, H, D)
    binding.tapa_phase2(p1["q"].t, p1["k"].t, p1["v"].t, head["q"].t, head["k"].t, head["v"].t, P, S, H, D)
    binding.ulysses_a2a(d["q"], d["k"], d["v"], flat["q"].t, flat["k"].t, flat["v"].t, P, S, H, D)
    torch.cuda.synchronize()
    for t in "qkv":
        ref_p1 = oracle.tapa_phase1(x[t], P)
        assert np.array_equal(p1[t].host((2, S, H, D)), ref_p1), t
        assert np.array_equal(head[t].host((H, S, D)), oracle.tapa_phase2(ref_p1, P)), t
        assert np.array_equal(head[t].host(), flat[t].host()), "two phases == flat exchange"
        for g in (p1[t], head[t], flat[t]):
            g.assert_guards(t)
    # only V, and ring independence: corrupting what ring 1 holds changes odd ranks only
    only = Guarded(E)
    bad = p1["v"].t.clone()
    bad[E:] = ~bad[E:]
    binding.tapa_phase2(None, None, bad, None, None, only.t, P, S, H, D)
    torch.cuda.synchronize()
    got = only.host((P, H // P, S, D))
    ref = head["v"].host((P, H // P, S, D))
    for r in range(P):
        assert np.array_equal(got[r], ref[r]) == (r % 2 == 0), r


def test_per_gpu_selection_on_phase1_holdings():
    """V-Major as the paper runs it: after Phase 1 of V one tile of every GPU
    compares all v it holds with the cached ones and selects inside its GPU."""
    P, S, H, D, T, r = 12, 1536, 12, 64, 16, 0.75
    E, n = S * H * D, S // T
    rng = np.random.default_rng(4)
    prev = rng.normal(0, 1, (S, H, D)).astype(np.float32)
    cur = prev + rng.normal(0, 1e-3, prev.shape).astype(np.float32)
    for u in rng.choice(n, n // 5, replace=False):
        cur[u * T:(u + 1) * T] += rng.normal(0, 0.5, (T, H, D)).astype(np.float32)
    prev_b, cur_b = synth.f32_to_bf16_bits(prev), synth.f32_to_bf16_bits(cur)
    p1_prev, p1_cur = torch.empty(2 * E, dtype=torch.int16, device="cuda"), torch.empty(2 * E, dtype=torch.int16, device="cuda")
    binding.tapa_phase1(None, None, dev(prev_b), None, None, p1_prev, P, S, H, D)
    binding.tapa_phase1(None, None, dev(cur_b), None, None, p1_cur, P, S, H, D)
    metric = torch.zeros(n, dtype=torch.int64, device="cuda")
    mask = torch.zeros(n, dtype=torch.uint8, device="cuda")
    idx = torch.zeros(n, dtype=torch.int32, device="cuda")
    na = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws_bytes = binding.vmajor_workspace_bytes(P, S, H, D, T)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    comp = Guarded(E)
    # tile 0 of every GPU: the first half of the p1 buffers, a [S][H][D] tensor; groups = GPUs
    binding.vmajor_select_compact(p1_prev[:E], p1_cur[:E], P, S, H, D, T, r, P // 2, metric, mask, idx, na, comp.t,
                                  ws, ws_bytes)
    torch.cuda.synchronize()
    ref_prev, ref_cur = oracle.tapa_phase1(prev_b, P)[0], oracle.tapa_phase1(cur_b, P)[0]
    m_ref = oracle.vmajor_metric(ref_prev, ref_cur, P, T)
    mask_ref, idx_ref, na_ref = oracle.vmajor_select(m_ref, P // 2, r)
    assert np.array_equal(metric.cpu().numpy().view(np.uint64), m_ref)
    assert int(na.item()) == na_ref and np.array_equal(mask.cpu().numpy(), mask_ref)
    assert np.array_equal(idx.cpu().numpy()[:na_ref], idx_ref)
    per_gpu = mask_ref.reshape(P // 2, -1).sum(axis=1)
    assert np.all(per_gpu == per_gpu[0]), "every GPU keeps the same number of active units"
    ref_c = oracle.pack_active(ref_cur, idx_ref, P, T)
    assert np.array_equal(comp.host()[:ref_c.size].reshape(ref_c.shape), ref_c)
