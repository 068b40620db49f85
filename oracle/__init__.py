"""ctypes access to the CPU oracle (oracle/cocodiff_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg; never by the product package.  This file only
compiles the C source with gcc and marshals numpy arrays; all arithmetic is in
the C file.  bf16 tensors are numpy uint16 bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cocodiff_oracle.c")
_SO = os.path.join(_HERE, "libcocodiff_oracle.so")
_SO_OMP = os.path.join(_HERE, "libcocodiff_oracle_omp.so")     # the same source, all host cores
_lib = None
_lib_omp = None


def build(force: bool = False, openmp: bool = False) -> str:
    """Compile the oracle with gcc (no FMA contraction, no fast-math).  openmp=True
    builds the same source with -fopenmp beside it (used by the benchmark only)."""
    out = _SO_OMP if openmp else _SO
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(_SRC):
        tmp = out + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math"] +
                              (["-fopenmp"] if openmp else []) + ["-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, out)
    return out


def _declare(handle):
    handle.oracle_bf16_to_f32.restype = C.c_float
    handle.oracle_bf16_to_f32.argtypes = [C.c_uint16]
    handle.oracle_f32_to_bf16.restype = C.c_uint16
    handle.oracle_f32_to_bf16.argtypes = [C.c_float]
    handle.oracle_head_shard_elems.restype = C.c_int64
    handle.oracle_seq_shard_elems.restype = C.c_int64
    return handle


def lib():
    global _lib
    if _lib is None:
        _lib = _declare(C.CDLL(build()))
    return _lib


def use_all_cores(on: bool) -> None:
    """Route the calls of this module to the OpenMP build (True) or back to the
    single-threaded build (False).  For the benchmark's CPU-baseline leg."""
    global _lib, _lib_omp
    if on:
        if _lib_omp is None:
            _lib_omp = _declare(C.CDLL(build(openmp=True)))
        _lib = _lib_omp
    else:
        _lib = None
        lib()


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _check(rc, what):
    if rc != 0:
        raise ValueError(f"oracle {what}: bad arguments (rc={rc})")


def bf16_to_f32(bits: int) -> float:
    return float(lib().oracle_bf16_to_f32(int(bits)))


def f32_to_bf16(x: float) -> int:
    return int(lib().oracle_f32_to_bf16(float(x)))


def head_shard_elems(P, S, H, D) -> int:
    return int(lib().oracle_head_shard_elems(P, S, H, D))


def seq_shard_elems(P, S, H, D) -> int:
    return int(lib().oracle_seq_shard_elems(P, S, H, D))


def rope_table_2d(pos: np.ndarray, D: int, theta: float) -> np.ndarray:
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    S = pos.shape[0]
    cs = np.empty((S, D // 2, 2), dtype=np.float32)
    _check(lib().oracle_rope_table_2d(_p(cs), _p(pos), S, D, C.c_double(theta)), "rope_table_2d")
    return cs


def norm_rope(x, w, eps, cs, want_f32=False):
    """x: [S][H][D] uint16.  Returns bf16 bits (and the unrounded fp32)."""
    x = _u16(x)
    S, H, D = x.shape
    w = None if w is None else _u16(w)
    cs = None if cs is None else np.ascontiguousarray(cs, dtype=np.float32)
    y = np.empty_like(x)
    yf = np.empty(x.shape, dtype=np.float32) if want_f32 else None
    _check(lib().oracle_norm_rope(_p(x), _p(w), C.c_float(eps), _p(cs), S, H, D, _p(y), _p(yf)),
           "norm_rope")
    return (y, yf) if want_f32 else y


def ulysses_a2a(seq, P):
    seq = _u16(seq)
    S, H, D = seq.shape
    head = np.empty((H, S, D), dtype=np.uint16)
    _check(lib().oracle_ulysses_a2a(_p(seq), _p(head), P, S, H, D), "ulysses_a2a")
    return head


def ulysses_a2a_inverse(head, P):
    head = _u16(head)
    H, S, D = head.shape
    seq = np.empty((S, H, D), dtype=np.uint16)
    _check(lib().oracle_ulysses_a2a_inverse(_p(head), _p(seq), P, S, H, D), "ulysses_a2a_inverse")
    return seq


def tapa_phase1(seq, P):
    """seq [S][H][D] -> p1 [2][S][H][D] (p1[t] = the copies held by the tiles of ring t)."""
    seq = _u16(seq)
    S, H, D = seq.shape
    p1 = np.empty((2, S, H, D), dtype=np.uint16)
    _check(lib().oracle_tapa_phase1(_p(seq), _p(p1), P, S, H, D), "tapa_phase1")
    return p1


def tapa_phase2(p1, P):
    p1 = _u16(p1)
    _, S, H, D = p1.shape
    head = np.empty((H, S, D), dtype=np.uint16)
    _check(lib().oracle_tapa_phase2(_p(p1), _p(head), P, S, H, D), "tapa_phase2")
    return head


def vmajor_metric(prev_v, cur_v, P, T):
    prev_v, cur_v = _u16(prev_v), _u16(cur_v)
    S, H, D = cur_v.shape
    if T < 1 or S % T:
        raise ValueError("oracle vmajor_metric: T must divide S")
    m = np.empty(S // T, dtype=np.uint64)
    _check(lib().oracle_vmajor_metric(_p(prev_v), _p(cur_v), P, S, H, D, T, _p(m)), "vmajor_metric")
    return m


def vmajor_select(metric, n_groups, r):
    metric = np.ascontiguousarray(metric, dtype=np.uint64)
    n = metric.shape[0]
    mask = np.empty(n, dtype=np.uint8)
    idx = np.full(n, -1, dtype=np.int32)
    na = C.c_int32(0)
    _check(lib().oracle_vmajor_select(_p(metric), n, n_groups, C.c_double(r), _p(mask), _p(idx),
                                      C.byref(na)), "vmajor_select")
    return mask, idx[:na.value].copy(), int(na.value)


def pack_active(x_seq, idx, P, T):
    """x_seq [S][H][D] -> compact [H][n_active*T][D]."""
    x_seq = _u16(x_seq)
    S, H, D = x_seq.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    na = idx.shape[0]
    out = np.empty((H, na * T, D), dtype=np.uint16)
    _check(lib().oracle_pack_active(_p(x_seq), _p(idx), na, _p(out), P, S, H, D, T), "pack_active")
    return out


def unpack(compact, idx, cache_head, P, T):
    """Scatter compact [H][n_active*T][D] over cache_head [H][S][D] in place."""
    compact = _u16(compact)
    assert cache_head.dtype == np.uint16 and cache_head.flags.c_contiguous
    H, S, D = cache_head.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    _check(lib().oracle_unpack(_p(compact), _p(idx), idx.shape[0], _p(cache_head), P, S, H, D, T),
           "unpack")
    return cache_head


def prologue(q, k, v, wq, wk, eps, cs, P):
    q, k, v = _u16(q), _u16(k), _u16(v)
    S, H, D = q.shape
    cs = np.ascontiguousarray(cs, dtype=np.float32)
    qh, kh, vh = (np.empty((H, S, D), dtype=np.uint16) for _ in range(3))
    scratch = np.empty((S, H, D), dtype=np.uint16)
    _check(lib().oracle_prologue(_p(q), _p(k), _p(v), _p(_u16(wq)), _p(_u16(wk)), C.c_float(eps),
                                 _p(cs), P, S, H, D, _p(qh), _p(kh), _p(vh), _p(scratch)), "prologue")
    return qh, kh, vh


def cache_schedule(step, total_steps, warmup, sync_interval):
    """(full_exchange, r) of a denoising step."""
    full, r = C.c_int(0), C.c_double(0.0)
    _check(lib().oracle_cache_schedule(step, total_steps, warmup, sync_interval, C.byref(full), C.byref(r)),
           "cache_schedule")
    return bool(full.value), float(r.value)
