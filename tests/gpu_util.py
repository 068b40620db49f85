"""Helpers for the GPU parity tests: host <-> device plumbing and guard bands.
torch only allocates device memory and streams here."""
import numpy as np
import torch

from paper_2604_14561_b200 import binding

CANARY = 0x5A5A
GUARD = 4096        # elements on each side of a guarded buffer


def dev(a):
    """numpy array -> CUDA tensor with the same bits (uint16/uint64 via signed views)."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    elif a.dtype == np.uint64:
        a = a.view(np.int64)
    return torch.from_numpy(a).cuda()


def u16(t):
    return t.detach().cpu().numpy().view(np.uint16)


class Guarded:
    """A 2-byte-element device buffer of `n` elements between two canary bands."""

    def __init__(self, n, fill=None):
        self.n = n
        self.raw = torch.full((n + 2 * GUARD,), CANARY - 0x10000 if CANARY > 0x7FFF else CANARY,
                              dtype=torch.int16, device="cuda")
        self.t = self.raw[GUARD:GUARD + n]
        if fill is not None:
            self.t.copy_(dev(fill).reshape(-1))

    def host(self, shape=None):
        a = u16(self.t)
        return a if shape is None else a.reshape(shape)

    def assert_guards(self, what=""):
        r = u16(self.raw)
        assert np.all(r[:GUARD] == CANARY) and np.all(r[GUARD + self.n:] == CANARY), f"guard band overwritten: {what}"


def rope_table(pos, D, theta):
    S = pos.shape[0]
    cs = torch.empty((S, D // 2, 2), dtype=torch.float32, device="cuda")
    binding.rope_table_2d(cs, dev(pos), S, D, theta)
    return cs


def run_prologue(L, cfg, order=binding.V_FIRST, two_streams=True):
    """Full prologue through the C ABI; returns (q_head, k_head, v_head) as
    uint16 arrays [H][S][D] and checks the guard bands."""
    S, H, D, P = cfg["S"], cfg["H"], cfg["D"], cfg["P"]
    E = S * H * D
    q, k, v = dev(L["q"]), dev(L["k"]), dev(L["v"])
    wq, wk = dev(L["wq"]), dev(L["wk"])
    cs = rope_table(L["pos"], D, cfg["theta"])
    out = [Guarded(E) for _ in range(3)]
    sq = torch.cuda.Stream()
    sv = torch.cuda.Stream() if two_streams else sq
    torch.cuda.synchronize()
    binding.prologue(q, k, v, out[0].t, out[1].t, out[2].t, wq, wk, cfg["eps"], cs, P, S, H, D,
                     order=order, stream_qk=sq, stream_v=sv)
    sq.synchronize()          # the call orders everything on stream_qk
    res = [o.host((H, S, D)) for o in out]
    for o in out:
        o.assert_guards("prologue")
    return res
