"""Seeded synthetic inputs for the Ulysses attention-prologue path.

This module holds the input recipe only: a counter-based random stream, the
bf16 bit-pattern rounding of generated numbers, token positions and the five
workload shapes.  It contains none of the method's arithmetic (no norm, no
rotation, no exchange, no selection) and imports neither the CUDA binding nor
the CPU oracle; both sides consume the arrays it returns.

The workloads stand in for DiT activations (the paper's models need trained
weights): Q, K, V ~ N(0, 1) stored as bf16, RMSNorm weights ~ N(1, 0.1) stored
as bf16, image tokens on a square grid in row-major order followed by text
tokens.  The grid sides follow the paper's rule "resolution / 16" (Section IV,
discussion of the absent 8-node bars): 768 -> 48, 1536 -> 96, 2304 -> 144.

Everything is numpy on the host; bf16 tensors are uint16 bit patterns.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 output function applied elementwise to a uint64 array."""
    x = (x ^ (x >> np.uint64(30))) * _M1
    x = (x ^ (x >> np.uint64(27))) * _M2
    return x ^ (x >> np.uint64(31))


def stream_key(seed: int, stream: str | int) -> np.uint64:
    """Key of an independent sub-stream: hash of (seed, stream name)."""
    if isinstance(stream, str):
        sid = 0
        for ch in stream.encode():
            sid = (sid * 131 + ch) & 0xFFFFFFFFFFFFFFFF
    else:
        sid = int(stream) & 0xFFFFFFFFFFFFFFFF
    with np.errstate(over="ignore"):
        a = _mix64(np.array([seed & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64) + _GOLDEN)
        b = _mix64(a ^ (np.array([sid], dtype=np.uint64) * _GOLDEN + _GOLDEN))
    return b[0]


def random_bits(key: np.uint64, start: int, n: int) -> np.ndarray:
    """64 random bits for counters start .. start+n-1 of the stream `key`."""
    with np.errstate(over="ignore"):
        ctr = np.arange(start + 1, start + n + 1, dtype=np.uint64)
        return _mix64(key + ctr * _GOLDEN)


def _normal_chunk(key, s0: int, m: int, mean: float, std: float, out: np.ndarray) -> None:
    bits = random_bits(key, s0, m)
    u1 = ((bits >> np.uint64(32)).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)
    u2 = ((bits & np.uint64(0xFFFFFFFF)).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    out[s0:s0 + m] = (mean + std * z).astype(np.float32)


def normal_f32(seed: int, stream: str | int, n: int, mean: float = 0.0,
               std: float = 1.0) -> np.ndarray:
    """n draws of N(mean, std) as float32 (Box-Muller on one 64-bit draw each).

    The value at index i depends only on (seed, stream, i); large requests are
    filled chunk by chunk on a few host threads (numpy releases the interpreter
    lock inside its loops), which changes no value.
    """
    key = stream_key(seed, stream)
    out = np.empty(n, dtype=np.float32)
    chunks = [(s0, min(_CHUNK, n - s0)) for s0 in range(0, n, _CHUNK)]
    if len(chunks) <= 1:
        for s0, m in chunks:
            _normal_chunk(key, s0, m, mean, std, out)
        return out
    with ThreadPoolExecutor(max_workers=min(8, len(chunks), os.cpu_count() or 1)) as pool:
        list(pool.map(lambda c: _normal_chunk(key, c[0], c[1], mean, std, out), chunks))
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bf16 (ties to even); returns uint16 bits.

    Storage-format conversion of generated inputs (finite values only).
    """
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(seed: int, stream: str | int, n: int, mean: float = 0.0,
                std: float = 1.0) -> np.ndarray:
    return f32_to_bf16_bits(normal_f32(seed, stream, n, mean, std))


def positions(grid_h: int, grid_w: int, n_text: int) -> np.ndarray:
    """pos[S][2] = (row, col), int32.

    Image tokens first in row-major order (row = s // W, col = s % W); text
    token j follows with the 1-D position j on both axes, (j, j).
    """
    s = np.arange(grid_h * grid_w, dtype=np.int32)
    img = np.stack([s // grid_w, s % grid_w], axis=1)
    j = np.arange(n_text, dtype=np.int32)
    txt = np.stack([j, j], axis=1)
    return np.ascontiguousarray(np.concatenate([img, txt], axis=0), dtype=np.int32)


# The five synthetic workloads.  S = grid_h * grid_w + n_text.
CONFIGS = {
    "tiny": dict(P=2, grid=(16, 16), n_text=0, H=4, D=64, seed=0),
    "sd3": dict(P=4, grid=(64, 64), n_text=256, H=24, D=64, seed=1),
    "qwen768": dict(P=8, grid=(48, 48), n_text=256, H=24, D=128, seed=2),
    "qwen2304": dict(P=12, grid=(144, 144), n_text=288, H=24, D=128, seed=3),
    "temporal": dict(P=24, grid=(96, 96), n_text=0, H=24, D=128, seed=4,
                     T=64, steps=8, r=0.8, n_groups=1,
                     sigma_small=1e-3, sigma_large=0.5, frac_large=0.2),
}
EPS = 1e-6
THETA = 10000.0


def config(name: str) -> dict:
    c = dict(CONFIGS[name])
    c["name"] = name
    c["S"] = c["grid"][0] * c["grid"][1] + c["n_text"]
    c["eps"] = EPS
    c["theta"] = THETA
    return c


def make_layer(cfg: dict) -> dict:
    """One layer's inputs: q, k, v in the sequence-parallel layout [S][H][D]
    (uint16 bf16 bits), wq, wk [D] (uint16 bf16 bits), pos [S][2] int32."""
    S, H, D, seed = cfg["S"], cfg["H"], cfg["D"], cfg["seed"]
    E = S * H * D
    out = {n: normal_bf16(seed, n, E).reshape(S, H, D) for n in ("q", "k", "v")}
    out["wq"] = normal_bf16(seed, "wq", D, 1.0, 0.1)
    out["wk"] = normal_bf16(seed, "wk", D, 1.0, 0.1)
    out["pos"] = positions(cfg["grid"][0], cfg["grid"][1], cfg["n_text"])
    return out


def perturbed_tiles(seed: int, step: int, n_tiles: int, frac: float) -> np.ndarray:
    """The ceil(frac * n_tiles) tiles that change strongly at `step`: drawn
    without replacement, re-drawn every step; returned ascending (int32)."""
    k = int(np.ceil(frac * n_tiles - 1e-9))
    bits = random_bits(stream_key(seed + step, "tiles"), 0, n_tiles)
    order = np.argsort(bits, kind="stable")
    return np.sort(order[:k]).astype(np.int32)


class TemporalSequence:
    """Consecutive denoising steps of the temporal-redundancy workload.

    float32 masters of Q, K, V are kept; step t+1 = step t + N(0, sigma_small)
    everywhere, plus N(0, sigma_large) on a seeded `frac_large` of the T-token
    tiles (the same tiles in Q, K and V: they stand for the same tokens).  Each
    step is re-rounded to bf16 from the master, because 1e-3 added directly to
    a bf16 value near 1 would mostly vanish under its 2^-7 spacing.
    """

    def __init__(self, cfg: dict):
        self.cfg = cfg
        S, H, D, seed = cfg["S"], cfg["H"], cfg["D"], cfg["seed"]
        self.E = S * H * D
        self.n_tiles = S // cfg["T"]
        self.tile_elems = cfg["T"] * H * D
        self.master = {n: normal_f32(seed, n, self.E) for n in ("q", "k", "v")}
        self.step = 0
        self.wq = normal_bf16(seed, "wq", D, 1.0, 0.1)
        self.wk = normal_bf16(seed, "wk", D, 1.0, 0.1)
        self.pos = positions(cfg["grid"][0], cfg["grid"][1], cfg["n_text"])
        self.large = np.zeros(0, dtype=np.int32)

    def current(self) -> dict:
        S, H, D = self.cfg["S"], self.cfg["H"], self.cfg["D"]
        return {n: f32_to_bf16_bits(self.master[n]).reshape(S, H, D) for n in ("q", "k", "v")}

    def advance(self) -> np.ndarray:
        """Move the masters to the next step; returns the perturbed tiles."""
        cfg = self.cfg
        self.step += 1
        t = self.step
        self.large = perturbed_tiles(cfg["seed"], t, self.n_tiles, cfg["frac_large"])
        for n in ("q", "k", "v"):
            m = self.master[n]
            m += normal_f32(cfg["seed"], f"{n}.small.{t}", self.E, 0.0, cfg["sigma_small"])
            big = normal_f32(cfg["seed"], f"{n}.large.{t}", len(self.large) * self.tile_elems,
                             0.0, cfg["sigma_large"]).reshape(len(self.large), self.tile_elems)
            mv = m.reshape(self.n_tiles, self.tile_elems)
            mv[self.large] += big
        return self.large
