"""The allocation-free V-Major entry point.

Some callers of this library may not allocate device memory at all (a plug-in
living inside someone else's memory pool, a hook running in a no-allocation
phase of the host application), so they cannot provide the scratch workspace
that `vmajor_select_compact` asks for.  `vmajor_select_compact_static` keeps that
scratch inside the library instead.  This test drives it through the C ABI and
requires bit-identical results to the workspace-taking call, twice in a row on
different inputs - the second call sees whatever the first one left in the
shared scratch and must not be disturbed by it.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle
from paper_2604_14561_b200 import binding, synth


def _dev(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(a).cuda()


def _inputs(S, H, D, T, seed):
    rng = np.random.default_rng(seed)
    prev = rng.normal(0, 1, (S, H, D)).astype(np.float32)
    cur = prev + rng.normal(0, 1e-3, prev.shape).astype(np.float32)
    n = S // T
    for u in rng.choice(n, max(1, n // 4), replace=False):
        cur[u * T:(u + 1) * T] += rng.normal(0, 0.5, (T, H, D)).astype(np.float32)
    return _dev(synth.f32_to_bf16_bits(prev)), _dev(synth.f32_to_bf16_bits(cur))


class _Outputs:
    def __init__(self, S, H, D, T):
        n = S // T
        self.metric = torch.full((n,), -1, dtype=torch.int64, device="cuda")
        self.mask = torch.full((n,), 7, dtype=torch.uint8, device="cuda")
        self.idx = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        self.n_active = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        self.v_compact = torch.full((S * H * D,), 0x5A5A, dtype=torch.int16, device="cuda")

    def tensors(self):
        return self.metric, self.mask, self.idx, self.n_active, self.v_compact


def test_static_scratch_matches_workspace_call_twice_in_a_row():
    calls = [  # (P, S, H, D, T, r, n_groups, seed): the second call uses fewer, larger units than the first
        (4, 2048, 4, 64, 1, 0.6, 4, 1),
        (2, 1024, 8, 128, 16, 0.8, 1, 2),
    ]
    for P, S, H, D, T, r, n_groups, seed in calls:
        prev, cur = _inputs(S, H, D, T, seed)
        want, got = _Outputs(S, H, D, T), _Outputs(S, H, D, T)
        ws_bytes = binding.vmajor_workspace_bytes(P, S, H, D, T)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        binding.vmajor_select_compact(prev, cur, P, S, H, D, T, r, n_groups, *want.tensors(), ws, ws_bytes)
        binding.vmajor_select_compact_static(prev, cur, P, S, H, D, T, r, n_groups, *got.tensors())
        torch.cuda.synchronize()
        assert int(want.n_active.item()) == S // T - n_groups * int(np.floor(r * (S // T // n_groups)))
        for name, a, b in zip(("metric", "mask", "idx", "n_active", "v_compact"), want.tensors(), got.tensors()):
            assert torch.equal(a, b), f"{name} differs from the workspace-taking entry point"
        # and directly against the CPU oracle's rule
        m_ref = oracle.vmajor_metric(prev.cpu().numpy().view(np.uint16).reshape(S, H, D),
                                     cur.cpu().numpy().view(np.uint16).reshape(S, H, D), P, T)
        mask_ref, idx_ref, na_ref = oracle.vmajor_select(m_ref, n_groups, r)
        assert np.array_equal(got.metric.cpu().numpy().view(np.uint64), m_ref)
        assert int(got.n_active.item()) == na_ref and np.array_equal(got.mask.cpu().numpy(), mask_ref)
        assert np.array_equal(got.idx.cpu().numpy()[:na_ref], idx_ref)


def test_static_scratch_at_its_unit_limit():
    """Exactly STATIC_MAX_UNITS per-token units in one group: the largest call the
    entry point accepts, checked against the oracle."""
    P, S, H, D, T, r = 2, binding.STATIC_MAX_UNITS, 2, 32, 1, 0.8
    prev, cur = _inputs(S, H, D, T, 3)
    got = _Outputs(S, H, D, T)
    for _ in range(2):
        binding.vmajor_select_compact_static(prev, cur, P, S, H, D, T, r, 1, *got.tensors())
    torch.cuda.synchronize()
    m_ref = oracle.vmajor_metric(prev.cpu().numpy().view(np.uint16).reshape(S, H, D),
                                 cur.cpu().numpy().view(np.uint16).reshape(S, H, D), P, T)
    mask_ref, idx_ref, na_ref = oracle.vmajor_select(m_ref, 1, r)
    assert np.array_equal(got.metric.cpu().numpy().view(np.uint64), m_ref)
    assert int(got.n_active.item()) == na_ref and np.array_equal(got.mask.cpu().numpy(), mask_ref)
    assert np.array_equal(got.idx.cpu().numpy()[:na_ref], idx_ref)
    comp_ref = oracle.pack_active(cur.cpu().numpy().view(np.uint16).reshape(S, H, D), idx_ref, P, T)
    assert np.array_equal(got.v_compact.cpu().numpy().view(np.uint16)[:comp_ref.size], comp_ref.reshape(-1))


def test_static_scratch_refuses_more_units_than_it_holds():
    S, T = (binding.STATIC_MAX_UNITS + 1) * 2, 1            # one unit too many, P = 2 divides it
    fake = 1 << 20                                          # never dereferenced: the call is refused first
    rc = binding.vmajor_select_compact_static(fake, fake * 2, 2, S, 2, 64, T, 0.5, 1, fake * 3, fake * 4,
                                              fake * 5, fake * 6, None, check=False)
    assert rc == -4
    assert "workspace" in binding.status_string(rc)
