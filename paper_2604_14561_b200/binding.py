"""Thin ctypes binding over libcocodiff.so: same names as the C ABI, argument
marshalling only.  Every step of the path runs in the CUDA library; there is
no fallback - if the library is missing or fails to load, `lib()` raises.

Tensors may be torch CUDA tensors (any 2-byte dtype for bf16 bit patterns),
raw integer device addresses, or None.  Streams may be torch.cuda.Stream,
raw cudaStream_t integers, or None (default stream).  Host-buffer arguments
of `prologue_host` take pinned torch CPU tensors or numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os

LUMP = 0
V_FIRST = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcocodiff.so")
_lib = None

STATUS = {0: "OK", -1: "INVALID_ARG", -2: "BAD_SHAPE", -3: "MISALIGNED", -4: "WORKSPACE_TOO_SMALL",
          -5: "CUDA_ERROR", -6: "ALIASING"}

# name -> (restype, argtypes); mirrors include/cocodiff.h
_P, _I, _F, _D, _Z = C.c_void_p, C.c_int, C.c_float, C.c_double, C.c_size_t
SIGNATURES = {
    "cocodiff_status_string": (C.c_char_p, [_I]),
    "cocodiff_version": (_I, []),
    "cocodiff_last_cuda_error": (_I, []),
    "cocodiff_rope_table_2d": (_I, [_P, _P, _I, _I, _D, _P]),
    "cocodiff_qk_norm_rope": (_I, [_P, _P, _P, _P, _P, _P, _F, _P, _I, _I, _I, _P]),
    "cocodiff_ulysses_a2a": (_I, [_P] * 6 + [_I] * 5 + [_P, _P]),
    "cocodiff_ulysses_a2a_inverse": (_I, [_P] * 6 + [_I] * 4 + [_P]),
    "cocodiff_prologue": (_I, [_P] * 8 + [_F, _P] + [_I] * 5 + [_P, _P]),
    "cocodiff_prologue_host": (_I, [_P] * 10 + [_F, _P] + [_I] * 5 + [_P, _P]),
    "cocodiff_vmajor_workspace_bytes": (_Z, [_I] * 5),
    "cocodiff_vmajor_select_compact": (_I, [_P, _P] + [_I] * 5 + [_D, _I] + [_P] * 6 + [_Z, _P]),
    "cocodiff_vmajor_select": (_I, [_P, _I, _D, _I, _P, _P, _P, _P]),
    "cocodiff_pack_active": (_I, [_P, _P, _F, _P, _P, _P, _P] + [_I] * 5 + [_P]),
    "cocodiff_unpack": (_I, [_P, _P, _P, _P] + [_I] * 5 + [_P]),
    "cocodiff_pack_active_qkv": (_I, [_P] * 5 + [_F] + [_P] * 6 + [_I] * 5 + [_P]),
    "cocodiff_unpack_qkv": (_I, [_P] * 8 + [_I] * 5 + [_P]),
    "cocodiff_vmajor_select_compact_static": (_I, [_P, _P] + [_I] * 5 + [_D, _I] + [_P] * 5 + [_P]),
    "cocodiff_cache_schedule": (_I, [_I] * 4 + [_P, _P]),
    "cocodiff_layer_step": (_I, [_I] * 4 + [_P] * 6 + [_F, _P] + [_I] * 6 + [_P] * 11 + [_Z, _I, _P, _P, _P]),
    "cocodiff_tapa_phase1": (_I, [_P] * 6 + [_I] * 4 + [_P]),
    "cocodiff_tapa_phase2": (_I, [_P] * 6 + [_I] * 4 + [_P]),
    "cocodiff_debug_bounds_violations": (C.c_longlong, []),
    "cocodiff_debug_bounds_selftest": (C.c_longlong, [_P, _P, _I, _I, _I, _P]),
    "cocodiff_selective_prologue": (_I, [_P] * 6 + [_F, _P] + [_I] * 5 + [_D, _I] + [_P] * 11 + [_Z, _I, _P, _P]),
}


class CocodiffError(RuntimeError):
    def __init__(self, fn, status):
        self.status = status
        extra = ""
        if status == -5 and _lib is not None:
            extra = f" (cudaError {_lib.cocodiff_last_cuda_error()})"
        super().__init__(f"{fn}: {STATUS.get(status, status)}{extra}")


def lib():
    """Load libcocodiff.so (built in-tree by `build.build()`); no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run paper_2604_14561_b200/build.py "
                               "(there is no CPU or PyTorch fallback for this path)")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):          # torch tensor (device or pinned host)
        return x.data_ptr()
    if hasattr(x, "ctypes"):            # numpy array (host)
        return x.ctypes.data
    raise TypeError(type(x))


def _stream(s):
    if s is None:
        return None
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _call(name, *args, check=True):
    rc = getattr(lib(), name)(*args)
    if check and rc != 0:
        raise CocodiffError(name, rc)
    return rc


def version() -> int:
    return lib().cocodiff_version()


def status_string(status: int) -> str:
    return lib().cocodiff_status_string(status).decode()


def rope_table_2d(cs, pos, S, D, theta, stream=None, check=True):
    return _call("cocodiff_rope_table_2d", _ptr(cs), _ptr(pos), S, D, theta, _stream(stream), check=check)


def qk_norm_rope(q, k, q_out, k_out, wq, wk, eps, cs, S, H, D, stream=None, check=True):
    return _call("cocodiff_qk_norm_rope", _ptr(q), _ptr(k), _ptr(q_out), _ptr(k_out), _ptr(wq), _ptr(wk),
                 eps, _ptr(cs), S, H, D, _stream(stream), check=check)


def ulysses_a2a(q, k, v, q_head, k_head, v_head, P, S, H, D, order=V_FIRST, stream_qk=None,
                stream_v=None, check=True):
    return _call("cocodiff_ulysses_a2a", _ptr(q), _ptr(k), _ptr(v), _ptr(q_head), _ptr(k_head),
                 _ptr(v_head), P, S, H, D, order, _stream(stream_qk), _stream(stream_v), check=check)


def ulysses_a2a_inverse(q_head, k_head, v_head, q, k, v, P, S, H, D, stream=None, check=True):
    return _call("cocodiff_ulysses_a2a_inverse", _ptr(q_head), _ptr(k_head), _ptr(v_head), _ptr(q),
                 _ptr(k), _ptr(v), P, S, H, D, _stream(stream), check=check)


def prologue(q, k, v, q_head, k_head, v_head, wq, wk, eps, cs, P, S, H, D, order=V_FIRST,
             stream_qk=None, stream_v=None, check=True):
    return _call("cocodiff_prologue", _ptr(q), _ptr(k), _ptr(v), _ptr(q_head), _ptr(k_head), _ptr(v_head),
                 _ptr(wq), _ptr(wk), eps, _ptr(cs), P, S, H, D, order, _stream(stream_qk),
                 _stream(stream_v), check=check)


def prologue_host(q_host, k_host, v_host, q_head_host, k_head_host, v_head_host, dev_in, dev_out,
                  wq, wk, eps, cs, P, S, H, D, order=V_FIRST, stream_qk=None, stream_v=None, check=True):
    return _call("cocodiff_prologue_host", _ptr(q_host), _ptr(k_host), _ptr(v_host), _ptr(q_head_host),
                 _ptr(k_head_host), _ptr(v_head_host), _ptr(dev_in), _ptr(dev_out), _ptr(wq), _ptr(wk),
                 eps, _ptr(cs), P, S, H, D, order, _stream(stream_qk), _stream(stream_v), check=check)


def vmajor_workspace_bytes(P, S, H, D, T) -> int:
    return int(lib().cocodiff_vmajor_workspace_bytes(P, S, H, D, T))


def vmajor_select_compact(prev_v, cur_v, P, S, H, D, T, r, n_groups, metric, mask, idx, n_active,
                          v_compact, workspace, workspace_bytes, stream=None, check=True):
    return _call("cocodiff_vmajor_select_compact", _ptr(prev_v), _ptr(cur_v), P, S, H, D, T, r, n_groups,
                 _ptr(metric), _ptr(mask), _ptr(idx), _ptr(n_active), _ptr(v_compact), _ptr(workspace),
                 workspace_bytes, _stream(stream), check=check)


def vmajor_select(metric, n, r, n_groups, mask, idx, n_active, stream=None, check=True):
    return _call("cocodiff_vmajor_select", _ptr(metric), n, r, n_groups, _ptr(mask), _ptr(idx),
                 _ptr(n_active), _stream(stream), check=check)


def pack_active(x, w, eps, cs, idx, n_active, x_compact, P, S, H, D, T, stream=None, check=True):
    return _call("cocodiff_pack_active", _ptr(x), _ptr(w), eps, _ptr(cs), _ptr(idx), _ptr(n_active),
                 _ptr(x_compact), P, S, H, D, T, _stream(stream), check=check)


def unpack(x_compact, idx, n_active, x_cache, P, S, H, D, T, stream=None, check=True):
    return _call("cocodiff_unpack", _ptr(x_compact), _ptr(idx), _ptr(n_active), _ptr(x_cache),
                 P, S, H, D, T, _stream(stream), check=check)


def pack_active_qkv(q, k, v, wq, wk, eps, cs, idx, n_active, q_compact, k_compact, v_compact,
                    P, S, H, D, T, stream=None, check=True):
    return _call("cocodiff_pack_active_qkv", _ptr(q), _ptr(k), _ptr(v), _ptr(wq), _ptr(wk), eps, _ptr(cs),
                 _ptr(idx), _ptr(n_active), _ptr(q_compact), _ptr(k_compact), _ptr(v_compact),
                 P, S, H, D, T, _stream(stream), check=check)


def unpack_qkv(q_compact, k_compact, v_compact, idx, n_active, q_cache, k_cache, v_cache,
               P, S, H, D, T, stream=None, check=True):
    return _call("cocodiff_unpack_qkv", _ptr(q_compact), _ptr(k_compact), _ptr(v_compact), _ptr(idx),
                 _ptr(n_active), _ptr(q_cache), _ptr(k_cache), _ptr(v_cache), P, S, H, D, T,
                 _stream(stream), check=check)


def selective_prologue(prev_v, q, k, v, wq, wk, eps, cs, P, S, H, D, T, r, n_groups, metric, mask, idx,
                       n_active, q_compact, k_compact, v_compact, q_cache, k_cache, v_cache,
                       workspace, workspace_bytes, order=V_FIRST, stream_qk=None, stream_v=None, check=True):
    return _call("cocodiff_selective_prologue", _ptr(prev_v), _ptr(q), _ptr(k), _ptr(v), _ptr(wq), _ptr(wk),
                 eps, _ptr(cs), P, S, H, D, T, r, n_groups, _ptr(metric), _ptr(mask), _ptr(idx),
                 _ptr(n_active), _ptr(q_compact), _ptr(k_compact), _ptr(v_compact), _ptr(q_cache),
                 _ptr(k_cache), _ptr(v_cache), _ptr(workspace), workspace_bytes, order,
                 _stream(stream_qk), _stream(stream_v), check=check)


STATIC_MAX_UNITS = 32768     # COCODIFF_STATIC_MAX_UNITS of include/cocodiff.h (a test keeps the two equal)


def vmajor_select_compact_static(prev_v, cur_v, P, S, H, D, T, r, n_groups, metric, mask, idx, n_active,
                                 v_compact, stream=None, check=True):
    """`vmajor_select_compact` without a workspace argument, for callers that cannot
    allocate device memory: the scratch is a fixed array inside the library (at most
    STATIC_MAX_UNITS selection units).  Calls on one device share that array, so calls
    that may overlap on the GPU must be ordered by the caller."""
    return _call("cocodiff_vmajor_select_compact_static", _ptr(prev_v), _ptr(cur_v), P, S, H, D, T, r,
                 n_groups, _ptr(metric), _ptr(mask), _ptr(idx), _ptr(n_active), _ptr(v_compact),
                 _stream(stream), check=check)


def tapa_phase1(q, k, v, q_p1, k_p1, v_p1, P, S, H, D, stream=None, check=True):
    return _call("cocodiff_tapa_phase1", _ptr(q), _ptr(k), _ptr(v), _ptr(q_p1), _ptr(k_p1), _ptr(v_p1),
                 P, S, H, D, _stream(stream), check=check)


def tapa_phase2(q_p1, k_p1, v_p1, q_head, k_head, v_head, P, S, H, D, stream=None, check=True):
    return _call("cocodiff_tapa_phase2", _ptr(q_p1), _ptr(k_p1), _ptr(v_p1), _ptr(q_head), _ptr(k_head),
                 _ptr(v_head), P, S, H, D, _stream(stream), check=check)


def cache_schedule(step, total_steps, warmup, sync_interval):
    """(full_exchange, r) of a denoising step; host-only."""
    full, r = C.c_int(0), C.c_double(0.0)
    _call("cocodiff_cache_schedule", step, total_steps, warmup, sync_interval,
          C.cast(C.byref(full), C.c_void_p), C.cast(C.byref(r), C.c_void_p))
    return bool(full.value), float(r.value)


def layer_step(step, total_steps, warmup, sync_interval, prev_v, q, k, v, wq, wk, eps, cs, P, S, H, D, T,
               n_groups, metric, mask, idx, n_active, q_compact, k_compact, v_compact, q_cache, k_cache,
               v_cache, workspace, workspace_bytes, order=V_FIRST, stream_qk=None, stream_v=None, check=True):
    """Returns (status, elements of Q, K, V that cross the exchange in this step)."""
    sent = C.c_int64(0)
    rc = _call("cocodiff_layer_step", step, total_steps, warmup, sync_interval, _ptr(prev_v), _ptr(q), _ptr(k),
               _ptr(v), _ptr(wq), _ptr(wk), eps, _ptr(cs), P, S, H, D, T, n_groups, _ptr(metric), _ptr(mask),
               _ptr(idx), _ptr(n_active), _ptr(q_compact), _ptr(k_compact), _ptr(v_compact), _ptr(q_cache),
               _ptr(k_cache), _ptr(v_cache), _ptr(workspace), workspace_bytes, order, _stream(stream_qk),
               _stream(stream_v), C.cast(C.byref(sent), C.c_void_p), check=check)
    return rc, int(sent.value)


def debug_bounds_violations() -> int:
    """Out-of-bounds accesses caught (and skipped) by the bounds-checked build since the
    last call; -1 when the loaded library is the normal build."""
    return int(lib().cocodiff_debug_bounds_violations())


def debug_bounds_selftest(x, y, S, H, D, stream=None) -> int:
    """Bounds-checked build only: a move told that its buffers end after S/2 tokens;
    returns how many accesses the checker caught and skipped (-1 in the normal build)."""
    return int(lib().cocodiff_debug_bounds_selftest(_ptr(x), _ptr(y), S, H, D, _stream(stream)))
