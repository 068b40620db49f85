"""GPU parity of the exchange, norm + RoPE and the fused prologue against the
CPU oracle, element by element, through the C ABI.  Moves are bit-exact; normed
and rotated values are within 2 bf16 ulp of the oracle's rounded result."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

import oracle
from paper_2604_14561_b200 import binding, synth

from gpu_util import Guarded, dev, rope_table, run_prologue, u16
from helpers import assert_norm_rope_close, bits_to_f32, exact_norm_rope_rows, note, parity_stats, ulp_bf16


def _layer(P, S, H, D, seed, grid=None):
    rng = np.random.default_rng(seed)
    L = {n: synth.normal_bf16(seed, n, S * H * D).reshape(S, H, D) for n in ("q", "k", "v")}
    L["wq"] = synth.normal_bf16(seed, "wq", D, 1.0, 0.1)
    L["wk"] = synth.normal_bf16(seed, "wk", D, 1.0, 0.1)
    L["pos"] = rng.integers(0, 150, (S, 2)).astype(np.int32)
    return L, dict(P=P, S=S, H=H, D=D, eps=1e-6, theta=10000.0)


def _check_prologue(L, cfg, report=None, **kw):
    """Runs the prologue, compares with the oracle element by element.  With `report`
    the distance statistics of Q and K go into the run record, and the elements that
    lie beyond 2 ulp of their own magnitude (cancelled rotations: the tolerance's floor
    applies there) are judged against a float64 evaluation of the textbook formula."""
    qh, kh, vh = run_prologue(L, cfg, **kw)
    cs = oracle.rope_table_2d(L["pos"], cfg["D"], cfg["theta"])
    assert np.array_equal(vh, oracle.ulysses_a2a(L["v"], cfg["P"])), "V must be moved bit-exactly"
    stats = {}
    for name, got, w in (("q", qh, L["wq"]), ("k", kh, L["wk"])):
        ref, ref_f = oracle.norm_rope(L[name], w, cfg["eps"], cs, want_f32=True)
        ref_h = oracle.ulysses_a2a(ref, cfg["P"])
        ref_fh = np.ascontiguousarray(ref_f.transpose(1, 0, 2))
        diff = got != ref_h
        frac = diff.mean()
        assert frac < 0.01, f"{name}: {frac:.4%} of elements differ from the oracle's rounding"
        if not diff.any():
            continue
        # tolerance evaluated on the rows that differ (pairs stay intact)
        rows = np.unique(np.argwhere(diff)[:, :2], axis=0)            # (head, token)
        g, r, rf = got[rows[:, 0], rows[:, 1]], ref_h[rows[:, 0], rows[:, 1]], ref_fh[rows[:, 0], rows[:, 1]]
        st = assert_norm_rope_close(g, r, rf, f"{name}_head")
        st["n"] = int(diff.size)
        st["ulp_hist"]["0"] += int(diff.size) - int(g.size)           # rows without any difference
        stats[name] = st
        if report is None:
            continue
        # strict outliers against the truth: is the kernel farther from it than the oracle is?
        gf, rfv = bits_to_f32(g).astype(np.float64), bits_to_f32(r).astype(np.float64)
        strict = np.abs(gf - rfv) > 2.0 * ulp_bf16(np.maximum(np.abs(rfv), 2.0 ** -126))
        bad_rows = np.unique(np.argwhere(strict)[:, 0])
        if len(bad_rows):
            tok, head = rows[bad_rows, 1], rows[bad_rows, 0]
            exact = exact_norm_rope_rows(L[name][tok, head], w, cfg["eps"], L["pos"][tok], cfg["theta"])
            m = strict[bad_rows]
            e_gpu, e_ora = np.abs(gf[bad_rows] - exact)[m], np.abs(rfv[bad_rows] - exact)[m]
            pair = exact.reshape(len(bad_rows), -1, 2)
            rho = np.sqrt((pair * pair).sum(axis=2)).repeat(2, axis=1)[m]
            # both sides: half a bf16 ulp of the true value plus a few fp32 roundings relative to the pair
            bound = 0.5 * ulp_bf16(np.maximum(np.abs(exact[m]), 2.0 ** -126)) + 8.0 * 2.0 ** -24 * rho
            assert np.all(e_gpu <= bound), f"{name}: kernel farther from the float64 value than fp32 arithmetic explains"
            assert np.all(e_ora <= bound)
            st["strict_outliers_vs_float64"] = dict(n=int(m.sum()), gpu_closer_or_equal=int((e_gpu <= e_ora).sum()),
                                                     worst_gpu_err_over_bound=float((e_gpu / bound).max()),
                                                     worst_oracle_err_over_bound=float((e_ora / bound).max()))
        note(f"{report} {name}: {st}")
    return (qh, kh, vh), stats


def test_rope_table_matches_oracle():
    for name in ("tiny", "qwen768"):
        cfg = synth.config(name)
        pos = synth.positions(*cfg["grid"], cfg["n_text"])
        got = rope_table(pos, cfg["D"], cfg["theta"]).cpu().numpy()
        ref = oracle.rope_table_2d(pos, cfg["D"], cfg["theta"])
        assert np.abs(got - ref).max() <= 6e-8       # at most one float ulp below 1
        assert (got != ref).mean() < 1e-3


@pytest.mark.parametrize("name", ["tiny", "sd3", "qwen768"])
@pytest.mark.parametrize("order", [binding.LUMP, binding.V_FIRST])
def test_prologue_parity_configs(name, order):
    cfg = synth.config(name)
    _check_prologue(synth.make_layer(cfg), cfg, order=order, report=name if order == binding.V_FIRST else None)


def test_prologue_parity_full_size_21k_tokens():
    cfg = synth.config("qwen2304")
    L = synth.make_layer(cfg)
    a, _ = _check_prologue(L, cfg, order=binding.V_FIRST, report="qwen2304")
    for b in (run_prologue(L, cfg, order=binding.LUMP), run_prologue(L, cfg, order=binding.V_FIRST, two_streams=False)):
        for x, y in zip(a, b):
            assert np.array_equal(x, y), "the order of issue must not change any value"


@pytest.mark.parametrize("P,S,H,D", [(1, 37, 1, 32), (1, 5, 3, 64), (3, 33, 3, 128), (2, 1002, 6, 256),
                                      (4, 4, 4, 64), (5, 535, 10, 32), (2, 130, 2, 128),
                                      # head dimensions that are not a power of two, and the smallest ones
                                      (2, 258, 4, 96), (3, 99, 3, 72), (1, 41, 2, 40), (2, 66, 2, 24), (2, 70, 4, 16),
                                      (1, 300, 3, 8), (2, 34, 2, 200), (1, 19, 5, 248)])
def test_prologue_ragged_and_degenerate_shapes(P, S, H, D):
    L, cfg = _layer(P, S, H, D, seed=100 + S)
    _check_prologue(L, cfg, order=binding.V_FIRST)
    _check_prologue(L, cfg, order=binding.LUMP, two_streams=False)
    _check_prologue(L, cfg, order=binding.V_FIRST, two_streams=False)      # V first on one stream


def test_empty_sequence_is_a_no_op():
    out = Guarded(64)
    x = torch.zeros(64, dtype=torch.int16, device="cuda")
    binding.ulysses_a2a(x, None, None, out.t, None, None, 2, 0, 4, 64)
    torch.cuda.synchronize()
    out.assert_guards()
    assert np.all(out.host() == 0x5A5A)


@pytest.mark.parametrize("P,S,H,D", [(2, 256, 4, 64), (4, 1000, 8, 128), (1, 77, 5, 32),
                                      (24, 9216, 24, 128)])      # the size the benchmark times the inverse at
def test_exchange_bit_exact_bijection_and_skips(P, S, H, D):
    L, cfg = _layer(P, S, H, D, seed=7)
    E = S * H * D
    ins = [dev(L[n]) for n in "qkv"]
    outs = [Guarded(E) for _ in range(3)]
    binding.ulysses_a2a(*ins, *(o.t for o in outs), P, S, H, D, order=binding.V_FIRST,
                        stream_qk=torch.cuda.Stream(), stream_v=torch.cuda.Stream())
    torch.cuda.synchronize()
    for n, o in zip("qkv", outs):
        assert np.array_equal(o.host((H, S, D)), oracle.ulysses_a2a(L[n], P))
        o.assert_guards()
    back = [Guarded(E) for _ in range(3)]
    binding.ulysses_a2a_inverse(*(o.t for o in outs), *(b.t for b in back), P, S, H, D)
    torch.cuda.synchronize()
    for n, b in zip("qkv", back):
        assert np.array_equal(b.host((S, H, D)), L[n])
        assert np.array_equal(b.host((S, H, D)), oracle.ulysses_a2a_inverse(oracle.ulysses_a2a(L[n], P), P))
        b.assert_guards()
    # only K
    only = Guarded(E)
    binding.ulysses_a2a(None, ins[1], None, None, only.t, None, P, S, H, D, order=binding.LUMP)
    torch.cuda.synchronize()
    assert np.array_equal(only.host((H, S, D)), oracle.ulysses_a2a(L["k"], P))


@pytest.mark.parametrize("S,H,D", [(256, 4, 64), (333, 3, 128), (64, 2, 256), (50, 7, 32), (45, 3, 80), (31, 2, 8)])
def test_qk_norm_rope_alone_and_in_place(S, H, D):
    L, cfg = _layer(1, S, H, D, seed=11)
    cs_ref = oracle.rope_table_2d(L["pos"], D, 10000.0)
    cs = rope_table(L["pos"], D, 10000.0)
    q, k = dev(L["q"]), dev(L["k"])
    qo, ko = Guarded(S * H * D), Guarded(S * H * D)
    binding.qk_norm_rope(q, k, qo.t, ko.t, dev(L["wq"]), dev(L["wk"]), 1e-6, cs, S, H, D)
    torch.cuda.synchronize()
    for name, out, w in (("q", qo, L["wq"]), ("k", ko, L["wk"])):
        ref, ref_f = oracle.norm_rope(L[name], w, 1e-6, cs_ref, want_f32=True)
        assert_norm_rope_close(out.host((S, H, D)), ref, ref_f, name)
        out.assert_guards()
    first = qo.host((S, H, D)).copy()
    binding.qk_norm_rope(q, None, q, None, dev(L["wq"]), None, 1e-6, cs, S, H, D)      # in place
    torch.cuda.synchronize()
    assert np.array_equal(u16(q).reshape(S, H, D), first)
    # no table: normalisation only
    binding.qk_norm_rope(None, k, None, ko.t, None, dev(L["wk"]), 1e-6, None, S, H, D)
    torch.cuda.synchronize()
    ref, ref_f = oracle.norm_rope(L["k"], L["wk"], 1e-6, None, want_f32=True)
    assert_norm_rope_close(ko.host((S, H, D)), ref, ref_f, "k norm only")


@pytest.mark.parametrize("name", ["tiny", "qwen768"])      # one chunk / eight pipelined token chunks
def test_prologue_host_buffers_match_device_path(name):
    cfg = synth.config(name)
    L = synth.make_layer(cfg)
    S, H, D, P = cfg["S"], cfg["H"], cfg["D"], cfg["P"]
    E = S * H * D
    want = run_prologue(L, cfg)
    hin = [torch.from_numpy(L[n].view(np.int16).copy()).pin_memory() for n in "qkv"]
    hout = [torch.empty(E, dtype=torch.int16).pin_memory() for _ in range(3)]
    dev_in = torch.empty(3 * E, dtype=torch.int16, device="cuda")
    dev_out = torch.empty(3 * E, dtype=torch.int16, device="cuda")
    cs = rope_table(L["pos"], D, cfg["theta"])
    for order in (binding.V_FIRST, binding.LUMP):
        sq, sv = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()
        binding.prologue_host(*hin, *hout, dev_in, dev_out, dev(L["wq"]), dev(L["wk"]), cfg["eps"], cs,
                              P, S, H, D, order=order, stream_qk=sq, stream_v=sv)
        sq.synchronize()
        for got, ref in zip(hout, want):
            assert np.array_equal(got.numpy().view(np.uint16).reshape(H, S, D), ref)
            got.zero_()


def test_exchange_and_norm_beyond_2_31_elements():
    """One tensor of 2.4e9 elements (4.8 GB): offsets no longer fit 32 bits.
    Checked on the device against what holds at any size: the exchange is the
    axis swap HEAD[h][s] = SEQ[s][h], its inverse restores the input, and a
    normalised row (weight 1, no rotation) has unit RMS."""
    P, S, H, D = 16, 1179648, 16, 128
    E = S * H * D
    assert E > 2 ** 31
    g = torch.Generator(device="cuda").manual_seed(0)
    x = torch.empty(E, dtype=torch.int16, device="cuda")
    for lo in range(0, E, 1 << 28):        # bf16 patterns of N(0,1) values, generated on the device
        hi = min(E, lo + (1 << 28))
        x[lo:hi] = torch.randn(hi - lo, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16).view(torch.int16)
    y = torch.empty(E, dtype=torch.int16, device="cuda")
    binding.ulysses_a2a(None, None, x, None, None, y, P, S, H, D, order=binding.LUMP)
    torch.cuda.synchronize()
    xv, yv = x.view(S, H, D), y.view(H, S, D)
    for h in range(H):
        assert torch.equal(yv[h], xv[:, h, :]), h
    back = torch.empty(E, dtype=torch.int16, device="cuda")
    binding.ulysses_a2a_inverse(None, None, y, None, None, back, P, S, H, D)
    torch.cuda.synchronize()
    assert torch.equal(back, x)
    del back
    w = torch.full((D,), 0x3F80, dtype=torch.int16, device="cuda")        # bf16 1.0
    # normalisation only (no table): SEQ -> SEQ
    binding.qk_norm_rope(x, None, y, None, w, None, 1e-6, None, S, H, D)
    torch.cuda.synchronize()
    rows = y.view(torch.bfloat16).view(S * H, D)
    for lo in (0, S * H // 2 - 1000, S * H - 4096):                        # first, middle and last rows
        r = rows[lo:lo + 4096].float()
        rms = r.pow(2).mean(dim=1).sqrt()
        assert torch.all((rms - 1.0).abs() < 2.0 ** -8), lo
    # and the normalised rows are the right rows: same signs as the input rows they came from
    assert torch.equal((y.view(S * H, D)[-4096:] < 0), (x.view(S * H, D)[-4096:] < 0))


def test_two_host_threads_call_the_library_at_once():
    """The library keeps no shared mutable state beyond guarded per-device caches and
    per-thread events: two host threads, each with its own streams and buffers, issue
    V-first prologues and selective steps concurrently and both get the oracle's results."""
    import threading
    cfg = synth.config("tiny")
    cfg.update(T=16, r=0.5)
    L = synth.make_layer(cfg)
    P, S, H, D, T = cfg["P"], cfg["S"], cfg["H"], cfg["D"], cfg["T"]
    E, n = S * H * D, S // T
    cs_ref = oracle.rope_table_2d(L["pos"], D, cfg["theta"])
    want = oracle.prologue(L["q"], L["k"], L["v"], L["wq"], L["wk"], cfg["eps"], cs_ref, P)
    prev = synth.normal_bf16(3, "prev", E).reshape(S, H, D)
    m_ref = oracle.vmajor_metric(prev, L["v"], P, T)
    mask_ref, idx_ref, na_ref = oracle.vmajor_select(m_ref, 1, cfg["r"])
    errors = []

    def worker(seed):
        try:
            torch.cuda.set_device(0)
            q, k, v, p_v = dev(L["q"]), dev(L["k"]), dev(L["v"]), dev(prev)
            wq, wk = dev(L["wq"]), dev(L["wk"])
            cs = rope_table(L["pos"], D, cfg["theta"])
            out = [torch.zeros(E, dtype=torch.int16, device="cuda") for _ in range(3)]
            comp = [torch.zeros(E, dtype=torch.int16, device="cuda") for _ in range(3)]
            metric = torch.zeros(n, dtype=torch.int64, device="cuda")
            mask = torch.zeros(n, dtype=torch.uint8, device="cuda")
            idx = torch.zeros(n, dtype=torch.int32, device="cuda")
            na = torch.zeros(1, dtype=torch.int32, device="cuda")
            ws_bytes = binding.vmajor_workspace_bytes(P, S, H, D, T)
            ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
            sq, sv = torch.cuda.Stream(), torch.cuda.Stream()
            for _ in range(200):
                binding.prologue(q, k, v, *out, wq, wk, cfg["eps"], cs, P, S, H, D, order=binding.V_FIRST,
                                 stream_qk=sq, stream_v=sv)
                binding.selective_prologue(p_v, q, k, v, wq, wk, cfg["eps"], cs, P, S, H, D, T, cfg["r"], 1, metric, mask,
                                           idx, na, *comp, None, None, None, ws, ws_bytes, order=binding.V_FIRST,
                                           stream_qk=sq, stream_v=sv)
            sq.synchronize()
            assert np.array_equal(u16(out[2]).reshape(H, S, D), want[2])
            assert (u16(out[0]).reshape(H, S, D) != want[0]).mean() < 0.01
            assert int(na.item()) == na_ref and np.array_equal(idx.cpu().numpy()[:na_ref], idx_ref)
            assert np.array_equal(mask.cpu().numpy(), mask_ref)
        except Exception as exc:      # reported by the main thread
            errors.append((seed, repr(exc)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors


@pytest.mark.parametrize("P,S,H,D", [(4, 1000, 8, 128), (24, 9216, 24, 128)])
def test_calls_chained_on_one_stream_keep_their_order(P, S, H, D):
    """Consecutive calls on one stream are launched as programmatic dependents of one another
    (a call's first kernel may become resident while the previous call's last kernel drains).
    Here every call reads what the call before it wrote, twelve calls without a host
    synchronisation in between, in both orders of issue: exchange -> inverse -> exchange -> ...
    must return the input bit for bit, and a stale read anywhere would not."""
    L, _ = _layer(P, S, H, D, seed=11)
    E = S * H * D
    x0 = [dev(L[n]) for n in "qkv"]
    seq = [[torch.zeros(E, dtype=torch.int16, device="cuda") for _ in range(3)] for _ in range(2)]
    head = [[torch.zeros(E, dtype=torch.int16, device="cuda") for _ in range(3)] for _ in range(2)]
    st = torch.cuda.Stream()
    torch.cuda.synchronize()
    src = x0
    for i in range(6):
        order = binding.V_FIRST if i % 2 == 0 else binding.LUMP
        binding.ulysses_a2a(*src, *head[i % 2], P, S, H, D, order=order, stream_qk=st, stream_v=st)
        binding.ulysses_a2a_inverse(*head[i % 2], *seq[i % 2], P, S, H, D, stream=st)
        src = seq[i % 2]
    st.synchronize()
    for n, got in zip("qkv", src):
        assert np.array_equal(u16(got).reshape(S, H, D), L[n]), n
    # the selective chain: scatter into the caches, read them back through the inverse, use that as prev_v
    T, r = (64, 0.5) if S % (P * 64) == 0 else (1, 0.5)      # 144 units ranked inside the mover / 1000 by the selection kernel
    n_units = S // T
    wq, wk = dev(L["wq"]), dev(L["wk"])
    cs = rope_table(L["pos"], D, 10000.0)
    cache = [torch.zeros(E, dtype=torch.int16, device="cuda") for _ in range(3)]
    prev_b = torch.zeros(E, dtype=torch.int16, device="cuda")
    metric = torch.zeros(n_units, dtype=torch.int64, device="cuda")
    mask = torch.zeros(n_units, dtype=torch.uint8, device="cuda")
    idx = torch.zeros(n_units, dtype=torch.int32, device="cuda")
    na = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws_bytes = binding.vmajor_workspace_bytes(P, S, H, D, T)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    binding.prologue(*x0, *cache, wq, wk, 1e-6, cs, P, S, H, D, order=binding.V_FIRST, stream_qk=st, stream_v=st)
    for i in range(3):
        binding.ulysses_a2a_inverse(None, None, cache[2], None, None, prev_b, P, S, H, D, stream=st)
        binding.selective_prologue(prev_b, *x0, wq, wk, 1e-6, cs, P, S, H, D, T, r, 1, metric, mask, idx, na,
                                   None, None, None, *cache, ws, ws_bytes, order=binding.LUMP, stream_qk=st, stream_v=st)
    st.synchronize()
    # prev_b always equalled V exactly (the full step filled the cache, selective steps rewrite the same
    # bits), so every distance is zero and the rule caches the lowest-numbered half
    assert np.array_equal(u16(prev_b).reshape(S, H, D), L["v"])
    assert not metric.any().item()
    n_cached = int(np.floor(r * n_units))
    assert int(na.item()) == n_units - n_cached
    assert np.array_equal(idx.cpu().numpy()[:n_units - n_cached], np.arange(n_cached, n_units))
    assert np.array_equal(u16(cache[2]).reshape(H, S, D), oracle.ulysses_a2a(L["v"], P))


def test_chained_calls_replayed_as_a_cuda_graph_keep_their_order():
    """The same dependent chain captured into a CUDA graph (the dependent launches become
    programmatic edges of the graph) and replayed: still the input, bit for bit."""
    P, S, H, D = 4, 2048, 8, 128
    L, _ = _layer(P, S, H, D, seed=13)
    E = S * H * D
    x0 = [dev(L[n]) for n in "qkv"]
    seq = [[torch.zeros(E, dtype=torch.int16, device="cuda") for _ in range(3)] for _ in range(2)]
    head = [[torch.zeros(E, dtype=torch.int16, device="cuda") for _ in range(3)] for _ in range(2)]
    st = torch.cuda.Stream()

    def chain():
        src = x0
        for i in range(4):
            order = binding.V_FIRST if i % 2 == 0 else binding.LUMP
            binding.ulysses_a2a(*src, *head[i % 2], P, S, H, D, order=order, stream_qk=st, stream_v=st)
            binding.ulysses_a2a_inverse(*head[i % 2], *seq[i % 2], P, S, H, D, stream=st)
            src = seq[i % 2]
        return src
    chain()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        last = chain()
    for t in seq[0] + seq[1] + head[0] + head[1]:
        t.zero_()
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        g.replay()
        g.replay()
    st.synchronize()
    for n, got in zip("qkv", last):
        assert np.array_equal(u16(got).reshape(S, H, D), L[n]), n
