"""The C-ABI library: it loads without a GPU, exports every symbol the header
declares, and rejects bad arguments before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2604_14561_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "cocodiff.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cocodiff_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert len(names) >= 14
    handle = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(handle, n), n
    assert set(names) == set(binding.SIGNATURES), set(names) ^ set(binding.SIGNATURES)


def test_status_strings_and_version():
    assert binding.version() >= 100
    assert binding.status_string(0) == "ok"
    for code in range(-6, 0):
        assert binding.status_string(code) != "unknown status"


A = 1 << 20          # fake, 16-byte aligned "device addresses"; never dereferenced:
                     # every call below fails validation before any launch


def _addr(i):
    return A * (i + 1)


def test_shape_validation():
    q, k, v, qh, kh, vh = (_addr(i) * 64 for i in range(6))
    ok = dict(P=2, S=8, H=4, D=64)
    for bad, want in ((dict(P=3), -2), (dict(S=7), -2), (dict(H=3), -2), (dict(D=44), -2), (dict(D=4), -2), (dict(D=264), -2),
                      (dict(P=8, S=8, H=4), -2), (dict(P=0), -1), (dict(H=0), -1)):
        a = dict(ok, **bad)
        rc = binding.ulysses_a2a(q, k, v, qh, kh, vh, a["P"], a["S"], a["H"], a["D"], check=False)
        assert rc == want, (bad, rc)
    assert binding.ulysses_a2a(q, k, v, qh, kh, vh, 2, 8, 4, 64, order=7, check=False) == -1


def test_pointer_validation():
    q, k, v, qh, kh, vh = (_addr(i) * 64 for i in range(6))
    assert binding.ulysses_a2a(q + 2, k, v, qh, kh, vh, 2, 8, 4, 64, check=False) == -3
    assert binding.ulysses_a2a(q, None, v, qh, kh, vh, 2, 8, 4, 64, check=False) == -1      # half a pair
    assert binding.ulysses_a2a(q, k, v, q + 16, kh, vh, 2, 8, 4, 64, check=False) == -6     # in/out overlap
    assert binding.ulysses_a2a(q, k, v, qh, qh, vh, 2, 8, 4, 64, check=False) == -6         # out/out overlap
    w, cs = _addr(40), _addr(41)
    assert binding.prologue(q, k, v, qh, kh, vh, None, w, 1e-6, cs, 2, 8, 4, 64, check=False) == -1
    assert binding.prologue(q, k, v, qh, kh, vh, w, w, 1e-6, None, 2, 8, 4, 64, check=False) == -1
    assert binding.prologue(q, k, None, qh, kh, vh, w, w, 1e-6, cs, 2, 8, 4, 64, check=False) == -1
    assert binding.prologue(q, k, v, qh, kh, vh, w, w, -1.0, cs, 2, 8, 4, 64, check=False) == -1
    assert binding.prologue(q, k, v, qh, kh, vh, w, w, 1e-6, cs + 4, 2, 8, 4, 64, check=False) == -3
    # norm + rope in place is allowed to alias exactly, not partially
    assert binding.qk_norm_rope(q, None, q + 32, None, w, None, 1e-6, cs, 8, 4, 64, check=False) == -6
    assert binding.qk_norm_rope(q, None, None, None, w, None, 1e-6, cs, 8, 4, 64, check=False) == -1


def test_vmajor_validation():
    prev, cur, comp = (_addr(i) * 64 for i in range(3))
    m, mask, idx, na, ws = (_addr(10 + i) for i in range(5))
    need = binding.vmajor_workspace_bytes(2, 64, 4, 64, 8)
    assert need >= 8 * 8 + 4 and need % 256 == 0
    args = dict(P=2, S=64, H=4, D=64, T=8, r=0.5, n_groups=1)

    def call(ws_bytes=need, **kw):
        a = dict(args, **kw)
        return binding.vmajor_select_compact(prev, cur, a["P"], a["S"], a["H"], a["D"], a["T"], a["r"],
                                             a["n_groups"], m, mask, idx, na, comp, ws, ws_bytes, check=False)
    assert call(T=3) == -2              # T must divide S/P
    assert call(T=0) == -1
    assert call(r=1.5) == -1 and call(r=-0.1) == -1 and call(r=float("nan")) == -1
    assert call(n_groups=3) == -2 and call(n_groups=0) == -1
    assert call(ws_bytes=need - 1) == -4
    assert binding.vmajor_select(m, 10, 0.5, 3, mask, idx, na, check=False) == -2
    assert binding.vmajor_select(m, 10, 2.0, 1, mask, idx, na, check=False) == -1
    assert binding.pack_active(cur, None, 0.0, None, idx, na, cur, 2, 64, 4, 64, 8, check=False) == -6
    assert binding.unpack(comp, idx, na, comp + 16, 2, 64, 4, 64, 8, check=False) == -6
    assert binding.unpack(comp, None, na, cur, 2, 64, 4, 64, 8, check=False) == -1


def test_selective_prologue_validation_of_direct_delivery():
    """Compact buffers are all given or all NULL, and all NULL only with the caches."""
    prev, q, k, v = (_addr(i) * 64 for i in range(4))
    comp = [_addr(4 + i) * 64 for i in range(3)]
    cache = [_addr(8 + i) * 64 for i in range(3)]
    m, mask, idx, na, ws, w, cs = (_addr(100 + i) for i in range(7))
    need = binding.vmajor_workspace_bytes(2, 64, 4, 64, 8)

    def call(comp, cache):
        return binding.selective_prologue(prev, q, k, v, w, w, 1e-6, cs, 2, 64, 4, 64, 8, 0.5, 1, m, mask, idx, na,
                                          *comp, *cache, ws, need, check=False)
    none = [None] * 3
    assert call(none, none) == -1                              # nowhere to deliver to
    assert call([comp[0], None, comp[2]], cache) == -1         # half a set of compact buffers
    assert call([None, None, comp[2]], cache) == -1
    assert call(comp, [cache[0], None, None]) == -1            # half a set of caches
    assert call(none, [cache[0], cache[0], cache[2]]) == -6    # two caches on one buffer
    assert call(none, [q, cache[1], cache[2]]) == -6           # a cache over an input
    assert call(none, [prev, cache[1], cache[2]]) == -6
    assert call(none, [cache[0] + 2, cache[1], cache[2]]) == -3


def test_static_unit_limit_is_the_headers():
    text = open(os.path.join(ROOT, "include", "cocodiff.h")).read()
    m = re.search(r"#define\s+COCODIFF_STATIC_MAX_UNITS\s+(\d+)", text)
    assert m and int(m.group(1)) == binding.STATIC_MAX_UNITS


def test_workspace_size_follows_the_cut_of_the_units():
    # 144 units of 24576 vectors are cut into 4 pieces each; per-token units are not cut
    assert binding.vmajor_workspace_bytes(24, 9216, 24, 128, 64) == 144 * 4 * 8 + 256
    assert binding.vmajor_workspace_bytes(24, 9216, 24, 128, 1) == 9216 * 8 + 256
    assert binding.vmajor_workspace_bytes(24, 9216, 24, 44, 1) == 0      # unsupported head dimension


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", binding.LIB_PATH + ".absent")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.lib()


def test_cache_schedule_matches_oracle_everywhere():
    """Host-only entry point: compared with the oracle over a grid of settings."""
    import oracle
    for total, warmup, interval in ((50, 5, 10), (8, 1, 0), (20, 3, 5), (4, 0, 0), (6, 6, 0), (1, 0, 0), (30, 2, 7)):
        for t in range(total):
            assert binding.cache_schedule(t, total, warmup, interval) == oracle.cache_schedule(t, total, warmup, interval)
    with pytest.raises(binding.CocodiffError):
        binding.cache_schedule(5, 5, 0, 0)
