"""The bounds-checked build of the library (every global access of every kernel
checked against the extent of its buffer, violations counted and skipped) run
over ragged and degenerate shapes of every entry point: no access may fall
outside, and the results must equal the normal build's bit for bit.  This stands
in for a memory checker, which the GPU pool does not offer."""
import contextlib

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_2604_14561_b200 import binding, build, synth

from gpu_util import dev, rope_table


@contextlib.contextmanager
def library(path):
    old = (binding.LIB_PATH, binding._lib)
    binding.LIB_PATH, binding._lib = path, None
    try:
        yield
    finally:
        binding.LIB_PATH, binding._lib = old


def _run_everything(P, S, H, D, T, r, n_groups, seed):
    """Every kernel-launching entry point once; returns all outputs as one list of tensors."""
    E, n = S * H * D, S // T
    x = {t: dev(synth.normal_bf16(seed, t, E).reshape(S, H, D)) for t in "qkv"}
    prev = dev(synth.normal_bf16(seed, "prev", E).reshape(S, H, D))
    wq, wk = dev(synth.normal_bf16(seed, "wq", D, 1.0, 0.1)), dev(synth.normal_bf16(seed, "wk", D, 1.0, 0.1))
    pos = np.random.default_rng(seed).integers(0, 150, (S, 2)).astype(np.int32)
    cs = rope_table(pos, D, 10000.0)
    new = lambda k=1: torch.zeros(k * E, dtype=torch.int16, device="cuda")
    outs = []
    sq, sv = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    h = [new() for _ in range(3)]
    binding.prologue(x["q"], x["k"], x["v"], *h, wq, wk, 1e-6, cs, P, S, H, D, order=binding.V_FIRST, stream_qk=sq, stream_v=sv)
    h2 = [new() for _ in range(3)]
    binding.prologue(x["q"], x["k"], x["v"], *h2, wq, wk, 1e-6, cs, P, S, H, D, order=binding.LUMP, stream_qk=sq, stream_v=sq)
    back = [new() for _ in range(3)]
    binding.ulysses_a2a_inverse(*h, *back, P, S, H, D, stream=sq)
    nr = [new() for _ in range(2)]
    binding.qk_norm_rope(x["q"], x["k"], *nr, wq, wk, 1e-6, cs, S, H, D, stream=sq)
    outs += h + h2 + back + nr
    if P % 2 == 0:
        p1 = [new(2) for _ in range(3)]
        th = [new() for _ in range(3)]
        binding.tapa_phase1(x["q"], x["k"], x["v"], *p1, P, S, H, D, stream=sq)
        binding.tapa_phase2(*p1, *th, P, S, H, D, stream=sq)
        outs += p1 + th
    metric = torch.zeros(max(n, 1), dtype=torch.int64, device="cuda")
    mask = torch.zeros(max(n, 1), dtype=torch.uint8, device="cuda")
    idx = torch.zeros(max(n, 1), dtype=torch.int32, device="cuda")
    na = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws_bytes = binding.vmajor_workspace_bytes(P, S, H, D, T)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    comp = [new() for _ in range(3)]
    cache = [new() for _ in range(3)]
    for order, s_v in ((binding.LUMP, sq), (binding.V_FIRST, sv)):
        binding.selective_prologue(prev, x["q"], x["k"], x["v"], wq, wk, 1e-6, cs, P, S, H, D, T, r, n_groups,
                                   metric, mask, idx, na, *comp, *cache, ws, ws_bytes, order=order, stream_qk=sq, stream_v=s_v)
    direct = [new() for _ in range(3)]      # no compact buffers: straight to the caches
    for order, s_v in ((binding.LUMP, sq), (binding.V_FIRST, sv)):
        binding.selective_prologue(prev, x["q"], x["k"], x["v"], wq, wk, 1e-6, cs, P, S, H, D, T, r, n_groups,
                                   metric, mask, idx, na, None, None, None, *direct, ws, ws_bytes, order=order,
                                   stream_qk=sq, stream_v=s_v)
    outs += direct
    vc = new()
    binding.vmajor_select_compact(prev, x["v"], P, S, H, D, T, r, n_groups, metric, mask, idx, na, vc, ws, ws_bytes, stream=sq)
    vs = new()
    binding.vmajor_select_compact_static(prev, x["v"], P, S, H, D, T, r, n_groups, metric, mask, idx, na, vs, stream=sq)
    c2, k2 = [new() for _ in range(3)], [new() for _ in range(3)]
    binding.pack_active_qkv(x["q"], x["k"], x["v"], wq, wk, 1e-6, cs, idx, na, *c2, P, S, H, D, T, stream=sq)
    binding.unpack_qkv(*c2, idx, na, *k2, P, S, H, D, T, stream=sq)
    sel_only = [torch.zeros(max(n, 1), dtype=torch.uint8, device="cuda"), torch.zeros(max(n, 1), dtype=torch.int32, device="cuda")]
    binding.vmajor_select(metric, n, r, n_groups, sel_only[0], sel_only[1], na, stream=sq)
    torch.cuda.synchronize()
    outs += comp + cache + [vc, vs, metric, mask, idx, na] + c2 + k2 + sel_only
    return outs


SHAPES = [  # P, S, H, D, T, r, n_groups
    (2, 256, 4, 64, 16, 0.8, 1), (3, 99, 3, 32, 11, 0.5, 3), (1, 37, 1, 32, 1, 0.3, 1), (4, 1000, 8, 128, 1, 0.7, 4),
    (2, 130, 2, 256, 5, 0.0, 1), (6, 66, 6, 64, 11, 1.0, 2), (12, 1752, 24, 128, 2, 0.9, 1), (2, 2306, 6, 64, 1153, 0.5, 2),
    (2, 258, 4, 96, 3, 0.6, 2), (4, 2400, 4, 40, 1, 0.8, 1), (2, 4096, 8, 128, 1024, 0.5, 1), (1, 70, 3, 8, 7, 0.5, 1),
]


def _random_shapes(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(count):
        P = int(rng.choice([1, 2, 3, 4, 6]))
        H = P * int(rng.integers(1, 4))
        D = int(rng.choice([8, 24, 32, 56, 64, 104, 128, 192, 256]))
        T = int(rng.choice([1, 2, 3, 7, 16, 40]))
        S = P * T * int(rng.integers(1, 60 if T < 16 else 8))
        n = S // T
        groups = int(rng.choice([g for g in (1, 2, P, n) if n % g == 0]))
        out.append((P, S, H, D, T, float(rng.choice([0.0, 0.3, 0.8, 1.0])), groups))
    return out


SHAPES += _random_shapes(8, seed=5)


@pytest.mark.parametrize("shape", SHAPES, ids=[str(s[:5]) for s in SHAPES])
def test_no_access_leaves_its_buffer(shape):
    debug = build.build(debug_bounds=True)
    want = _run_everything(*shape, seed=31)
    assert binding.debug_bounds_violations() == -1          # the normal build carries no checks
    with library(debug):
        assert binding.debug_bounds_violations() == 0       # clears the counter
        got = _run_everything(*shape, seed=31)
        assert binding.debug_bounds_violations() == 0, "a kernel reached outside one of its buffers"
    assert len(got) == len(want)
    for i, (a, b) in enumerate(zip(got, want)):
        assert torch.equal(a, b), f"output {i} differs between the two builds"


def test_the_checker_catches_and_skips_what_it_should():
    debug = build.build(debug_bounds=True)
    S, H, D = 101, 3, 64
    x = dev(synth.normal_bf16(5, "x", S * H * D).reshape(S, H, D))
    y = torch.full((S * H * D,), 0x5A5A, dtype=torch.int16, device="cuda")
    assert binding.debug_bounds_selftest(x, y, S, H, D) == -1               # normal build: no checker
    with library(debug):
        caught = binding.debug_bounds_selftest(x, y, S, H, D)
    half = (S // 2) * H * D
    assert caught == 2 * (S - S // 2) * H * (D // 8)
    assert torch.equal(y[:half], x.reshape(-1)[:half]), "accesses inside the claimed extent are performed"
    assert torch.all(y[half:] == 0x5A5A), "accesses outside the claimed extent are skipped"
