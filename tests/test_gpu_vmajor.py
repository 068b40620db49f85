"""GPU parity of the V-Major path (metric, selection, compaction, unpack)
against the CPU oracle through the C ABI: everything here is bit-exact except
the normed and rotated values inside compacted Q/K (2 bf16 ulp)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle
from paper_2604_14561_b200 import binding, synth

from gpu_util import Guarded, dev, rope_table, u16
from helpers import assert_norm_rope_close


class Selector:
    """Device buffers of one V-Major call."""

    def __init__(self, P, S, H, D, T):
        self.shape = (P, S, H, D, T)
        n = S // T
        self.n = n
        self.metric = torch.zeros(max(n, 1), dtype=torch.int64, device="cuda")
        self.mask = torch.full((max(n, 1),), 77, dtype=torch.uint8, device="cuda")
        self.idx = torch.full((max(n, 1),), -1, dtype=torch.int32, device="cuda")
        self.n_active = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        self.ws_bytes = binding.vmajor_workspace_bytes(P, S, H, D, T)
        self.ws = torch.full((self.ws_bytes,), 0xAB, dtype=torch.uint8, device="cuda")   # dirty on purpose
        self.v_compact = Guarded(S * H * D)

    def run(self, prev_v, cur_v, r, n_groups, compact=True, stream=None):
        P, S, H, D, T = self.shape
        binding.vmajor_select_compact(prev_v, cur_v, P, S, H, D, T, r, n_groups, self.metric, self.mask,
                                      self.idx, self.n_active, self.v_compact.t if compact else None,
                                      self.ws, self.ws_bytes, stream=stream)
        torch.cuda.synchronize()
        na = int(self.n_active.item())
        return (self.metric.cpu().numpy().view(np.uint64)[:self.n], self.mask.cpu().numpy()[:self.n],
                self.idx.cpu().numpy()[:na], na)


def _pair(S, H, D, T, seed, frac=0.25):
    rng = np.random.default_rng(seed)
    prev = rng.normal(0, 1, (S, H, D)).astype(np.float32)
    cur = prev + rng.normal(0, 1e-3, prev.shape).astype(np.float32)
    n = S // T
    hot = np.sort(rng.choice(n, max(1, int(frac * n)), replace=False))
    for u in hot:
        cur[u * T:(u + 1) * T] += rng.normal(0, 0.5, (T, H, D)).astype(np.float32)
    return synth.f32_to_bf16_bits(prev), synth.f32_to_bf16_bits(cur), hot


@pytest.mark.parametrize("P,S,H,D,T,n_groups", [
    (2, 256, 4, 64, 16, 1), (2, 256, 4, 64, 16, 2), (4, 512, 4, 128, 1, 4), (4, 512, 4, 128, 1, 1),
    (3, 96, 3, 32, 8, 12), (1, 40, 2, 256, 5, 1), (8, 2560, 8, 128, 64, 4), (2, 1200, 2, 64, 1, 1),
    # units cut into pieces (few large units), one block per unit, and head dimensions off the powers of two
    (2, 1024, 8, 128, 256, 1), (4, 2048, 8, 96, 32, 2), (2, 640, 4, 40, 4, 1), (1, 520, 3, 8, 1, 1),
    (2, 16384, 2, 64, 8192, 1), (3, 3000, 3, 72, 1, 3)])
@pytest.mark.parametrize("r", [0.0, 0.3, 0.8, 1.0])
def test_metric_selection_and_v_compaction(P, S, H, D, T, n_groups, r):
    prev, cur, _ = _pair(S, H, D, T, seed=S + T)
    sel = Selector(P, S, H, D, T)
    metric, mask, idx, na = sel.run(dev(prev), dev(cur), r, n_groups)
    m_ref = oracle.vmajor_metric(prev, cur, P, T)
    assert np.array_equal(metric, m_ref)
    mask_ref, idx_ref, na_ref = oracle.vmajor_select(m_ref, n_groups, r)
    assert na == na_ref and np.array_equal(mask, mask_ref) and np.array_equal(idx, idx_ref)
    comp_ref = oracle.pack_active(cur, idx_ref, P, T)
    got = sel.v_compact.host()[:comp_ref.size].reshape(comp_ref.shape)
    assert np.array_equal(got, comp_ref)
    assert np.all(sel.v_compact.host()[comp_ref.size:] == 0x5A5A), "nothing beyond the compact extent is written"
    sel.v_compact.assert_guards()
    # a second call on the same (now used) workspace gives the same answer
    metric2, mask2, idx2, na2 = sel.run(dev(prev), dev(cur), r, n_groups, compact=False)
    assert np.array_equal(metric2, m_ref) and np.array_equal(mask2, mask_ref) and na2 == na_ref


def test_metric_special_values():
    S, H, D, T = 64, 2, 64, 4
    prev = synth.f32_to_bf16_bits(np.zeros((S, H, D), np.float32))
    cur = prev.copy()
    cur[3, 1, 5] = 0x7FC0            # NaN
    cur[20, 0, 0] = 0x7F7F           # largest finite bf16: saturates
    cur[40, 1, 63] = 0x3880          # 2^-14 -> 4
    cur[41, 1, 63] = 0x3700          # 2^-17 -> 0
    sel = Selector(1, S, H, D, T)
    metric, _, _, _ = sel.run(dev(prev), dev(cur), 0.5, 1, compact=False)
    assert np.array_equal(metric, oracle.vmajor_metric(prev, cur, 1, T))
    assert metric[0] == 2 ** 32 - 1 and metric[5] == 2 ** 32 - 1 and metric[10] == 4
    same, _, _, na = sel.run(dev(cur), dev(cur), 0.5, 1, compact=False)
    assert np.all(np.delete(same, 0) == 0)      # NaN - NaN is NaN: unit 0 stays saturated


@pytest.mark.parametrize("n,n_groups", [(144, 1), (1000, 1), (1000, 8), (5000, 1), (21024, 1), (4096, 2), (513, 1), (600, 600),
                                        (32768, 1), (30000, 1), (65535, 1), (70000, 1), (140000, 2), (512, 1), (1024, 2)])
def test_selection_alone_with_ties_and_wide_keys(n, n_groups):
    rng = np.random.default_rng(n + n_groups)
    for r, kind in ((0.8, "ties"), (0.5, "wide"), (0.999, "ties"), (0.0, "wide"), (1.0, "ties"), (0.25, "equal"),
                    (0.8, "sums"), (0.3, "sums"), (0.6, "narrow")):
        if kind == "ties":
            m = rng.integers(0, 7, n).astype(np.uint64)
        elif kind == "equal":
            m = np.full(n, 12345, np.uint64)
        elif kind == "sums":      # like per-token distances: a tight cluster and a far, wide one
            m = rng.normal(2.0e5, 3.0e3, n)
            hot = rng.random(n) < 0.2
            m[hot] = rng.normal(8.0e7, 2.0e6, int(hot.sum()))
            m = np.maximum(m, 0).astype(np.uint64)
        elif kind == "narrow":    # thousands of units inside one key of the coarse histogram
            m = (np.uint64(3 << 40) + rng.integers(0, 1 << 20, n).astype(np.uint64))
        else:
            m = rng.integers(0, 2 ** 63, n).astype(np.uint64) * np.uint64(2) + rng.integers(0, 2, n).astype(np.uint64)
            m[rng.integers(0, n, n // 4)] = m[0]
        mask = torch.full((n,), 9, dtype=torch.uint8, device="cuda")
        idx = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        na = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        binding.vmajor_select(dev(m), n, r, n_groups, mask, idx, na)
        torch.cuda.synchronize()
        mask_ref, idx_ref, na_ref = oracle.vmajor_select(m, n_groups, r)
        assert int(na.item()) == na_ref, (r, kind)
        assert np.array_equal(mask.cpu().numpy(), mask_ref), (r, kind)
        assert np.array_equal(idx.cpu().numpy()[:na_ref], idx_ref), (r, kind)
        assert np.all(idx.cpu().numpy()[na_ref:] == -1)


def test_selection_alone_random_shapes():
    """Seeded random draws of the group structure, the ratio and the shape of the metric
    distribution: every selection kernel and every branch inside them against the oracle."""
    rng = np.random.default_rng(2024)
    for case in range(60):
        g = int(rng.choice([1, 2, 31, 32, 33, 100, 255, 256, 257, 300, 512, 1000, 2047, 2048, 2049, 4097, 9000, 16385, 40000]))
        n_groups = int(rng.choice([1, 1, 2, 3, 7])) if g < 20000 else 1
        n = g * n_groups
        r = float(rng.choice([0.0, 1.0, rng.random(), rng.random(), 1.0 / g, 1.0 - 1.0 / g]))
        kind = rng.integers(0, 5)
        if kind == 0:
            m = rng.integers(0, 3, n).astype(np.uint64)                                   # almost all ties
        elif kind == 1:
            m = rng.integers(0, 2 ** 63, n).astype(np.uint64) * np.uint64(2)              # all 64 bits in use
        elif kind == 2:
            m = np.maximum(rng.normal(3.0e5, 4.0e3, n), 0).astype(np.uint64)               # one tight cluster
        elif kind == 3:
            m = (np.uint64(1) << rng.integers(0, 60, n).astype(np.uint64)) + rng.integers(0, 2, n).astype(np.uint64)
        else:
            m = np.full(n, int(rng.integers(0, 2 ** 40)), np.uint64)                      # all equal
            m[rng.integers(0, n, max(1, n // 10))] += np.uint64(1)
        mask = torch.full((n,), 9, dtype=torch.uint8, device="cuda")
        idx = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        na = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        binding.vmajor_select(dev(m), n, r, n_groups, mask, idx, na)
        torch.cuda.synchronize()
        mask_ref, idx_ref, na_ref = oracle.vmajor_select(m, n_groups, r)
        what = (case, g, n_groups, r, int(kind))
        assert int(na.item()) == na_ref, what
        assert np.array_equal(mask.cpu().numpy(), mask_ref), what
        assert np.array_equal(idx.cpu().numpy()[:na_ref], idx_ref), what


@pytest.mark.parametrize("P,S,H,D,T", [(2, 256, 4, 64, 16), (4, 512, 4, 128, 1), (3, 99, 3, 32, 11), (2, 384, 2, 256, 64)])
def test_pack_active_qk_and_unpack(P, S, H, D, T):
    rng = np.random.default_rng(S)
    n = S // T
    x = synth.normal_bf16(5, "x", S * H * D).reshape(S, H, D)
    w = synth.normal_bf16(5, "w", D, 1.0, 0.1)
    pos = rng.integers(0, 150, (S, 2)).astype(np.int32)
    cs_ref = oracle.rope_table_2d(pos, D, 10000.0)
    cs = rope_table(pos, D, 10000.0)
    normed, normed_f = oracle.norm_rope(x, w, 1e-6, cs_ref, want_f32=True)
    for k in (0, 1, n // 3, n):
        idx_np = np.sort(rng.choice(n, k, replace=False)).astype(np.int32)
        idx = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        idx[:k] = dev(idx_np)
        na = torch.tensor([k], dtype=torch.int32, device="cuda")
        comp = Guarded(S * H * D)
        binding.pack_active(dev(x), dev(w), 1e-6, cs, idx, na, comp.t, P, S, H, D, T)
        torch.cuda.synchronize()
        comp.assert_guards()
        ref = oracle.pack_active(normed, idx_np, P, T)
        tok = (idx_np[:, None] * T + np.arange(T)[None, :]).reshape(-1)
        ref_f32 = np.ascontiguousarray(normed_f[tok].transpose(1, 0, 2))
        got = comp.host()[:ref.size].reshape(ref.shape)
        if k:
            assert_norm_rope_close(got, ref, ref_f32, "compact q/k")
        assert np.all(comp.host()[ref.size:] == 0x5A5A)
        # plain move of the same units is bit-exact
        plain = Guarded(S * H * D)
        binding.pack_active(dev(x), None, 0.0, None, idx, na, plain.t, P, S, H, D, T)
        torch.cuda.synchronize()
        ref_plain = oracle.pack_active(x, idx_np, P, T)
        assert np.array_equal(plain.host()[:ref_plain.size].reshape(ref_plain.shape), ref_plain)
        # scatter over a cached tensor
        old = synth.normal_bf16(6, "old", S * H * D).reshape(H, S, D)
        cache = Guarded(S * H * D, fill=old)
        binding.unpack(plain.t, idx, na, cache.t, P, S, H, D, T)
        torch.cuda.synchronize()
        cache.assert_guards()
        want = oracle.unpack(ref_plain, idx_np, old.copy(), P, T)
        assert np.array_equal(cache.host((H, S, D)), want)
        binding.unpack(plain.t, idx, na, cache.t, P, S, H, D, T)          # idempotent
        torch.cuda.synchronize()
        assert np.array_equal(cache.host((H, S, D)), want)


def _temporal_cfg(small):
    cfg = synth.config("temporal")
    if small:
        cfg.update(grid=(32, 24), P=4, H=4, D=64, T=16, steps=4)
        cfg["S"] = 32 * 24
    return cfg


@pytest.mark.parametrize("small", [True, False], ids=["reduced", "full-size"])
def test_temporal_steps_select_compact_unpack(small):
    """Several denoising steps: step 0 runs the full prologue and fills the
    caches; every later step selects on V, compacts V, K, Q (norm + RoPE fused)
    and scatters them over the caches.  Compared with the oracle step by step;
    the active set must equal the generator's strongly perturbed tiles."""
    cfg = _temporal_cfg(small)
    P, S, H, D, T = cfg["P"], cfg["S"], cfg["H"], cfg["D"], cfg["T"]
    E, n = S * H * D, S // T
    seq = synth.TemporalSequence(cfg)
    cs_ref = oracle.rope_table_2d(seq.pos, D, cfg["theta"])
    cs = rope_table(seq.pos, D, cfg["theta"])
    wq, wk = dev(seq.wq), dev(seq.wk)
    cur = seq.current()
    # step 0: full exchange on both sides
    cache_ref = dict(zip("qkv", oracle.prologue(cur["q"], cur["k"], cur["v"], seq.wq, seq.wk, cfg["eps"], cs_ref, P)))
    cache = {x: Guarded(E) for x in "qkv"}
    d = {x: dev(cur[x]) for x in "qkv"}
    binding.prologue(d["q"], d["k"], d["v"], cache["q"].t, cache["k"].t, cache["v"].t, wq, wk, cfg["eps"], cs,
                     P, S, H, D, order=binding.V_FIRST, stream_qk=None, stream_v=torch.cuda.Stream())
    torch.cuda.synchronize()
    assert np.array_equal(cache["v"].host((H, S, D)), cache_ref["v"])
    # Q and K caches start from the oracle's bits on both sides so that later steps compare exactly
    for x in "qk":
        cache[x].t.copy_(dev(cache_ref[x]).reshape(-1))
    prev_v = cur["v"]
    sel = Selector(P, S, H, D, T)
    comp = {x: Guarded(E) for x in "qk"}
    for step in range(1, cfg["steps"]):
        hot = seq.advance()
        cur = seq.current()
        d = {x: dev(cur[x]) for x in "qkv"}
        metric, mask, idx, na = sel.run(dev(prev_v), d["v"], cfg["r"], cfg["n_groups"])
        m_ref = oracle.vmajor_metric(prev_v, cur["v"], P, T)
        mask_ref, idx_ref, na_ref = oracle.vmajor_select(m_ref, cfg["n_groups"], cfg["r"])
        assert np.array_equal(metric, m_ref) and np.array_equal(mask, mask_ref)
        assert na == na_ref and np.array_equal(idx, idx_ref)
        assert np.array_equal(idx, hot), "active set = the strongly perturbed tiles"
        if step % 2:      # one tensor per call
            for x, w, w_np in (("k", wk, seq.wk), ("q", wq, seq.wq)):
                binding.pack_active(d[x], w, cfg["eps"], cs, sel.idx, sel.n_active, comp[x].t, P, S, H, D, T)
            for x, src in (("v", sel.v_compact), ("k", comp["k"]), ("q", comp["q"])):
                binding.unpack(src.t, sel.idx, sel.n_active, cache[x].t, P, S, H, D, T)
        else:             # the batched calls
            binding.pack_active_qkv(d["q"], d["k"], None, wq, wk, cfg["eps"], cs, sel.idx, sel.n_active,
                                    comp["q"].t, comp["k"].t, None, P, S, H, D, T)
            binding.unpack_qkv(comp["q"].t, comp["k"].t, sel.v_compact.t, sel.idx, sel.n_active,
                               cache["q"].t, cache["k"].t, cache["v"].t, P, S, H, D, T)
        torch.cuda.synchronize()
        # oracle: norm + RoPE on all rows, extract the active ones, scatter
        oracle.unpack(oracle.pack_active(cur["v"], idx_ref, P, T), idx_ref, cache_ref["v"], P, T)
        assert np.array_equal(cache["v"].host((H, S, D)), cache_ref["v"]), f"V cache, step {step}"
        tok = (idx_ref[:, None] * T + np.arange(T)[None, :]).reshape(-1)
        for x, w_np in (("k", seq.wk), ("q", seq.wq)):
            ref, ref_f = oracle.norm_rope(cur[x], w_np, cfg["eps"], cs_ref, want_f32=True)
            oracle.unpack(oracle.pack_active(ref, idx_ref, P, T), idx_ref, cache_ref[x], P, T)
            got = cache[x].host((H, S, D))
            inactive = np.ones(S, bool)
            inactive[tok] = False
            assert np.array_equal(got[:, inactive], cache_ref[x][:, inactive]), f"{x}: cached rows must not move"
            assert_norm_rope_close(got[:, tok], cache_ref[x][:, tok],
                                   np.ascontiguousarray(ref_f[tok].transpose(1, 0, 2)), f"{x} cache, step {step}")
            cache[x].t.copy_(dev(cache_ref[x]).reshape(-1))     # re-align the two sides bit for bit
            cache[x].assert_guards()
        prev_v = cur["v"]


@pytest.mark.parametrize("order,two_streams", [(binding.LUMP, False), (binding.V_FIRST, True), (binding.V_FIRST, False)])
@pytest.mark.parametrize("P,S,H,D,T,r,n_groups", [(4, 768, 4, 64, 16, 0.8, 1), (2, 256, 6, 128, 1, 0.5, 2),
                                                   (3, 99, 3, 32, 11, 0.0, 1), (2, 384, 2, 256, 64, 1.0, 1)])
def test_selective_prologue_one_call(order, two_streams, P, S, H, D, T, r, n_groups):
    """The fused selective step equals the oracle's select -> extract -> scatter,
    and the batched pack / unpack entry points equal the single-tensor ones."""
    E, n = S * H * D, S // T
    rng = np.random.default_rng(S + T)
    prev, cur_v, _ = _pair(S, H, D, T, seed=S)
    x = {"q": synth.normal_bf16(8, "q", E).reshape(S, H, D), "k": synth.normal_bf16(8, "k", E).reshape(S, H, D),
         "v": cur_v}
    w = {"q": synth.normal_bf16(8, "wq", D, 1.0, 0.1), "k": synth.normal_bf16(8, "wk", D, 1.0, 0.1)}
    pos = rng.integers(0, 150, (S, 2)).astype(np.int32)
    cs_ref, cs = oracle.rope_table_2d(pos, D, 10000.0), rope_table(pos, D, 10000.0)
    old = {t: synth.normal_bf16(9, "old" + t, E).reshape(H, S, D) for t in "qkv"}
    comp = {t: Guarded(E) for t in "qkv"}
    cache = {t: Guarded(E, fill=old[t]) for t in "qkv"}
    sel = Selector(P, S, H, D, T)
    d = {t: dev(x[t]) for t in "qkv"}
    sq = torch.cuda.Stream()
    sv = torch.cuda.Stream() if two_streams else sq
    torch.cuda.synchronize()
    binding.selective_prologue(dev(prev), d["q"], d["k"], d["v"], dev(w["q"]), dev(w["k"]), 1e-6, cs, P, S, H, D, T,
                               r, n_groups, sel.metric, sel.mask, sel.idx, sel.n_active,
                               comp["q"].t, comp["k"].t, comp["v"].t, cache["q"].t, cache["k"].t, cache["v"].t,
                               sel.ws, sel.ws_bytes, order=order, stream_qk=sq, stream_v=sv)
    sq.synchronize()
    m_ref = oracle.vmajor_metric(prev, cur_v, P, T)
    mask_ref, idx_ref, na_ref = oracle.vmajor_select(m_ref, n_groups, r)
    assert np.array_equal(sel.metric.cpu().numpy().view(np.uint64)[:n], m_ref)
    assert int(sel.n_active.item()) == na_ref
    assert np.array_equal(sel.mask.cpu().numpy()[:n], mask_ref)
    assert np.array_equal(sel.idx.cpu().numpy()[:na_ref], idx_ref)
    tok = (idx_ref[:, None] * T + np.arange(T)[None, :]).reshape(-1).astype(np.int64)
    inactive = np.ones(S, bool)
    inactive[tok] = False
    for t in "qkv":
        if t == "v":
            ref, ref_f = x["v"], None
        else:
            ref, ref_f = oracle.norm_rope(x[t], w[t], 1e-6, cs_ref, want_f32=True)
        comp_ref = oracle.pack_active(ref, idx_ref, P, T)
        got_c = comp[t].host()[:comp_ref.size].reshape(comp_ref.shape)
        want_cache = oracle.unpack(comp_ref, idx_ref, old[t].copy(), P, T)
        got_cache = cache[t].host((H, S, D))
        assert np.array_equal(got_cache[:, inactive], want_cache[:, inactive])
        if t == "v":
            assert np.array_equal(got_c, comp_ref) and np.array_equal(got_cache, want_cache)
        elif na_ref:
            f = np.ascontiguousarray(ref_f[tok].transpose(1, 0, 2))
            assert_norm_rope_close(got_c, comp_ref, f, t + " compact")
            assert np.array_equal(got_cache[:, tok], got_c), "scatter moves the compact rows bit-exactly"
        assert np.all(comp[t].host()[comp_ref.size:] == 0x5A5A)
        comp[t].assert_guards()
        cache[t].assert_guards()
    # batched entry points against the fused call's own outputs
    comp2 = {t: Guarded(E) for t in "qkv"}
    cache2 = {t: Guarded(E, fill=old[t]) for t in "qkv"}
    binding.pack_active_qkv(d["q"], d["k"], d["v"], dev(w["q"]), dev(w["k"]), 1e-6, cs, sel.idx, sel.n_active,
                            comp2["q"].t, comp2["k"].t, comp2["v"].t, P, S, H, D, T)
    binding.unpack_qkv(comp2["q"].t, comp2["k"].t, comp2["v"].t, sel.idx, sel.n_active,
                       cache2["q"].t, cache2["k"].t, cache2["v"].t, P, S, H, D, T)
    torch.cuda.synchronize()
    for t in "qkv":
        assert np.array_equal(comp2[t].host(), comp[t].host())
        assert np.array_equal(cache2[t].host(), cache[t].host())


def test_selective_prologue_random_small_shapes():
    """Seeded random draws of (P, S, H, D, T, r, groups, order): the fused selective step
    against the oracle on shapes nobody picked by hand."""
    rng = np.random.default_rng(77)
    for case in range(36):
        P = int(rng.choice([1, 2, 3, 4, 6]))
        H = P * int(rng.integers(1, 4))
        D = int(rng.choice([8, 16, 24, 32, 48, 64, 96, 128, 160, 256]))
        T = int(rng.choice([1, 2, 3, 5, 8, 16, 64]))
        S = P * T * int(rng.integers(1, 40 if T < 16 else 6))
        n = S // T
        divisors = [g for g in (1, 2, 3, P, n) if g >= 1 and n % g == 0]
        n_groups = int(rng.choice(divisors))
        r = float(rng.choice([0.0, 1.0, 0.5, 0.8, rng.random()]))
        order, two = [(binding.LUMP, False), (binding.V_FIRST, True), (binding.V_FIRST, False)][case % 3]
        what = dict(case=case, P=P, S=S, H=H, D=D, T=T, r=r, n_groups=n_groups, order=order, two_streams=two)
        E = S * H * D
        prev, cur_v, _ = _pair(S, H, D, T, seed=1000 + case)
        x = {"q": synth.normal_bf16(20 + case, "q", E).reshape(S, H, D), "k": synth.normal_bf16(20 + case, "k", E).reshape(S, H, D),
             "v": cur_v}
        w = {"q": synth.normal_bf16(20 + case, "wq", D, 1.0, 0.1), "k": synth.normal_bf16(20 + case, "wk", D, 1.0, 0.1)}
        pos = rng.integers(0, 150, (S, 2)).astype(np.int32)
        cs_ref, cs = oracle.rope_table_2d(pos, D, 10000.0), rope_table(pos, D, 10000.0)
        old = {t: synth.normal_bf16(9, "old" + t, E).reshape(H, S, D) for t in "qkv"}
        comp = {t: Guarded(E) for t in "qkv"}
        cache = {t: Guarded(E, fill=old[t]) for t in "qkv"}
        sel = Selector(P, S, H, D, T)
        d = {t: dev(x[t]) for t in "qkv"}
        sq = torch.cuda.Stream()
        sv = torch.cuda.Stream() if two else sq
        torch.cuda.synchronize()
        binding.selective_prologue(dev(prev), d["q"], d["k"], d["v"], dev(w["q"]), dev(w["k"]), 1e-6, cs, P, S, H, D, T,
                                   r, n_groups, sel.metric, sel.mask, sel.idx, sel.n_active,
                                   comp["q"].t, comp["k"].t, comp["v"].t, cache["q"].t, cache["k"].t, cache["v"].t,
                                   sel.ws, sel.ws_bytes, order=order, stream_qk=sq, stream_v=sv)
        sq.synchronize()
        m_ref = oracle.vmajor_metric(prev, cur_v, P, T)
        mask_ref, idx_ref, na_ref = oracle.vmajor_select(m_ref, n_groups, r)
        assert np.array_equal(sel.metric.cpu().numpy().view(np.uint64)[:n], m_ref), what
        assert int(sel.n_active.item()) == na_ref, what
        assert np.array_equal(sel.mask.cpu().numpy()[:n], mask_ref), what
        assert np.array_equal(sel.idx.cpu().numpy()[:na_ref], idx_ref), what
        tok = (idx_ref[:, None] * T + np.arange(T)[None, :]).reshape(-1).astype(np.int64)
        for t in "qkv":
            if t == "v":
                ref, ref_f = x["v"], None
            else:
                ref, ref_f = oracle.norm_rope(x[t], w[t], 1e-6, cs_ref, want_f32=True)
            comp_ref = oracle.pack_active(ref, idx_ref, P, T)
            got_c = comp[t].host()[:comp_ref.size].reshape(comp_ref.shape)
            want_cache = oracle.unpack(comp_ref, idx_ref, old[t].copy(), P, T)
            got_cache = cache[t].host((H, S, D))
            if t == "v":
                assert np.array_equal(got_c, comp_ref) and np.array_equal(got_cache, want_cache), what
            else:
                if na_ref:
                    assert_norm_rope_close(got_c, comp_ref, np.ascontiguousarray(ref_f[tok].transpose(1, 0, 2)), f"{t} {what}")
                    assert np.array_equal(got_cache[:, tok], got_c), what
                untouched = np.ones(S, bool)
                untouched[tok] = False
                assert np.array_equal(got_cache[:, untouched], want_cache[:, untouched]), what
            assert np.all(comp[t].host()[comp_ref.size:] == 0x5A5A), what
            comp[t].assert_guards()
            cache[t].assert_guards()


def _direct_cases():
    cases = [(4, 768, 4, 64, 16, 0.8, 1), (2, 256, 6, 128, 1, 0.5, 2), (3, 99, 3, 32, 11, 0.0, 1),
             (2, 384, 2, 256, 64, 1.0, 1), (4, 2400, 4, 40, 1, 0.8, 1), (2, 1024, 8, 128, 256, 0.5, 1)]
    rng = np.random.default_rng(311)
    for _ in range(12):
        P = int(rng.choice([1, 2, 3, 4, 6]))
        H = P * int(rng.integers(1, 4))
        D = int(rng.choice([8, 24, 32, 48, 64, 104, 128, 200, 256]))
        T = int(rng.choice([1, 2, 3, 5, 16, 64]))
        S = P * T * int(rng.integers(1, 40 if T < 16 else 6))
        n = S // T
        cases.append((P, S, H, D, T, float(rng.choice([0.0, 1.0, 0.5, 0.8, rng.random()])),
                      int(rng.choice([g for g in (1, 2, P, n) if n % g == 0]))))
    return cases


def test_selective_prologue_direct_delivery():
    """Without compact buffers the active rows go straight to the caches: the caches
    match the oracle's select -> extract -> scatter and carry the very bits the call with
    compact buffers leaves there; selection outputs are the same; nothing else is touched."""
    orders = [(binding.LUMP, False), (binding.V_FIRST, True), (binding.V_FIRST, False)]
    for case, (P, S, H, D, T, r, n_groups) in enumerate(_direct_cases()):
        order, two = orders[case % 3]
        what = dict(case=case, P=P, S=S, H=H, D=D, T=T, r=r, n_groups=n_groups, order=order, two_streams=two)
        E, n = S * H * D, S // T
        rng = np.random.default_rng(900 + case)
        prev, cur_v, _ = _pair(S, H, D, T, seed=500 + case)
        x = {"q": synth.normal_bf16(40 + case, "q", E).reshape(S, H, D),
             "k": synth.normal_bf16(40 + case, "k", E).reshape(S, H, D), "v": cur_v}
        w = {"q": synth.normal_bf16(40 + case, "wq", D, 1.0, 0.1), "k": synth.normal_bf16(40 + case, "wk", D, 1.0, 0.1)}
        pos = rng.integers(0, 150, (S, 2)).astype(np.int32)
        cs_ref, cs = oracle.rope_table_2d(pos, D, 10000.0), rope_table(pos, D, 10000.0)
        old = {t: synth.normal_bf16(9, "old" + t, E).reshape(H, S, D) for t in "qkv"}
        d = {t: dev(x[t]) for t in "qkv"}
        sq = torch.cuda.Stream()
        sv = torch.cuda.Stream() if two else sq
        runs = {}
        for mode in ("compact", "direct"):
            comp = {t: Guarded(E) for t in "qkv"}
            cache = {t: Guarded(E, fill=old[t]) for t in "qkv"}
            sel = Selector(P, S, H, D, T)
            cb = [comp[t].t if mode == "compact" else None for t in "qkv"]
            torch.cuda.synchronize()
            for _ in range(2):
                binding.selective_prologue(dev(prev), d["q"], d["k"], d["v"], dev(w["q"]), dev(w["k"]), 1e-6, cs,
                                           P, S, H, D, T, r, n_groups, sel.metric, sel.mask, sel.idx, sel.n_active,
                                           *cb, cache["q"].t, cache["k"].t, cache["v"].t, sel.ws, sel.ws_bytes,
                                           order=order, stream_qk=sq, stream_v=sv)
            sq.synchronize()
            runs[mode] = (sel, comp, cache)
        m_ref = oracle.vmajor_metric(prev, cur_v, P, T)
        mask_ref, idx_ref, na_ref = oracle.vmajor_select(m_ref, n_groups, r)
        sel, comp, cache = runs["direct"]
        assert np.array_equal(sel.metric.cpu().numpy().view(np.uint64)[:n], m_ref), what
        assert int(sel.n_active.item()) == na_ref, what
        assert np.array_equal(sel.mask.cpu().numpy()[:n], mask_ref), what
        assert np.array_equal(sel.idx.cpu().numpy()[:na_ref], idx_ref), what
        tok = (idx_ref[:, None] * T + np.arange(T)[None, :]).reshape(-1).astype(np.int64)
        untouched = np.ones(S, bool)
        untouched[tok] = False
        for t in "qkv":
            if t == "v":
                ref, ref_f = x["v"], None
            else:
                ref, ref_f = oracle.norm_rope(x[t], w[t], 1e-6, cs_ref, want_f32=True)
            want_cache = oracle.unpack(oracle.pack_active(ref, idx_ref, P, T), idx_ref, old[t].copy(), P, T)
            got = cache[t].host((H, S, D))
            assert np.array_equal(got[:, untouched], want_cache[:, untouched]), what
            if t == "v":
                assert np.array_equal(got, want_cache), what
            elif na_ref:
                assert_norm_rope_close(got[:, tok], want_cache[:, tok],
                                       np.ascontiguousarray(ref_f[tok].transpose(1, 0, 2)), f"{t} {what}")
            assert np.array_equal(got, runs["compact"][2][t].host((H, S, D))), "both modes leave the same bits"
            assert np.all(comp[t].host() == 0x5A5A), "no compact buffer is written"
            cache[t].assert_guards()
