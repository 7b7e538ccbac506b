"""ctypes front-end of the fp64 CPU oracle (``sla_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the benchmark's CPU
baseline leg.  Nothing on the product path imports this module, and this module imports nothing
from the CUDA package.  It only marshals numpy arrays into the C routines; all of the method's
arithmetic lives in ``sla_oracle.c``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sla_oracle.c")
_LIB = os.path.join(_HERE, "libsla_oracle.so")

F32, BF16, F64 = 0, 1, 2
UNION, PER_SPAN = 0, 1

_lib = None


def build(force: bool = False) -> str:
    """Compile ``sla_oracle.c`` into ``libsla_oracle.so`` next to it (gcc, -O2, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        i64, i32, dbl, vp = C.c_int64, C.c_int, C.c_double, C.c_void_p
        _lib.sla_oracle_isqrt.restype = i64
        _lib.sla_oracle_isqrt.argtypes = [i64]
        _lib.sla_oracle_ceil_isqrt.restype = i64
        _lib.sla_oracle_ceil_isqrt.argtypes = [i64]
        _lib.sla_oracle_base_len.restype = i64
        _lib.sla_oracle_base_len.argtypes = [i64, i64, dbl]
        _lib.sla_oracle_stride_offset.restype = i64
        _lib.sla_oracle_stride_offset.argtypes = [i64, dbl]
        _lib.sla_oracle_n_strides.restype = i64
        _lib.sla_oracle_n_strides.argtypes = [i64, dbl]
        _lib.sla_oracle_anchors.restype = i64
        _lib.sla_oracle_anchors.argtypes = [i64, i64, dbl, vp, vp, i64]
        _lib.sla_oracle_span.restype = None
        _lib.sla_oracle_span.argtypes = [i64, i64, i64, i64, i64, vp, vp]
        _lib.sla_oracle_threads.restype = i32
        _lib.sla_oracle_span_search.restype = i32
        _lib.sla_oracle_span_search.argtypes = (
            [vp, vp, i32, i32, i32, i32, i32, i64, i64, i64, i64, i32, i64, dbl, dbl, vp, i64, vp, vp, vp, vp]
        )
        _lib.sla_oracle_span_attention.restype = i32
        _lib.sla_oracle_span_attention.argtypes = (
            [vp, vp, vp, i32, i32, i32, i32, i32, i64, i64, i64, i64, i32, i64, i64, i64, i64, i32, dbl, dbl,
             vp, i64, vp, vp, vp, vp, vp, vp]
        )
        _lib.sla_oracle_decode_step.restype = i32
        _lib.sla_oracle_decode_step.argtypes = (
            [vp, vp, vp, vp, i32, i32, i32, i32, i32, i64, i64, i32, i64, i64, i64, i64, i32, dbl, dbl, dbl, dbl,
             vp, vp, vp, vp, vp, vp, vp]
        )
    return _lib


def threads() -> int:
    return int(lib().sla_oracle_threads())


# ----------------------------------------------------------------------------- scalar helpers
def isqrt(x: int) -> int:
    return int(lib().sla_oracle_isqrt(int(x)))


def ceil_isqrt(x: int) -> int:
    return int(lib().sla_oracle_ceil_isqrt(int(x)))


def base_len(i: int, span_len: int = 0, span_exponent: float = 0.5) -> int:
    return int(lib().sla_oracle_base_len(int(i), int(span_len), float(span_exponent)))


def stride_offset(s: int, search_exponent: float = 0.5) -> int:
    """Distance of the stride-s anchor from position i + 1."""
    return int(lib().sla_oracle_stride_offset(int(s), float(search_exponent)))


def n_strides(i: int, search_exponent: float = 0.5) -> int:
    return int(lib().sla_oracle_n_strides(int(i), float(search_exponent)))


def anchors(i: int, window: int = 0, search_exponent: float = 0.5):
    """Candidate anchor positions of query ``i`` and their stride indices, nearest first."""
    p = float(search_exponent)
    n = int(lib().sla_oracle_anchors(int(i), int(window), p, None, None, 0))
    t = np.zeros(max(n, 1), dtype=np.int64)
    s = np.zeros(max(n, 1), dtype=np.int64)
    lib().sla_oracle_anchors(int(i), int(window), p, t.ctypes.data, s.ctypes.data, n)
    return t[:n], s[:n]


def span(i: int, t: int, ell: int, b: int = 2, f: int = 0):
    lo, hi = C.c_int64(), C.c_int64()
    lib().sla_oracle_span(int(i), int(t), int(ell), int(b), int(f), C.byref(lo), C.byref(hi))
    return int(lo.value), int(hi.value)


# ----------------------------------------------------------------------------- array marshalling
def _as_input(a: np.ndarray, dtype_code: int) -> np.ndarray:
    """fp32 / fp64 arrays pass as they are; bf16 arrays pass as their uint16 bit patterns."""
    want = {F32: np.float32, BF16: np.uint16, F64: np.float64}[dtype_code]
    if a.dtype != want:
        raise TypeError(f"expected {want} for dtype code {dtype_code}, got {a.dtype}")
    if not a.flags["C_CONTIGUOUS"]:
        raise ValueError("oracle inputs must be C-contiguous")
    return a


def _rows(rows):
    if rows is None:
        return None, 0, None
    r = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    return r, int(r.size), r.ctypes.data


def span_search(q_s, k, dtype, *, top_k, q_pos0=0, Lkv=None, window=0, search_scale=1.0, rows=None,
                search_exponent=0.5):
    """q_s [B,Hq,Lq,D], k [B,Hkv,cap,D] -> dict(anchor, score, gap, n_dots); see the C header comment."""
    q_s, k = _as_input(q_s, dtype), _as_input(k, dtype)
    B, Hq, Lq, D = q_s.shape
    _, Hkv, cap, _ = k.shape
    Lkv = cap if Lkv is None else int(Lkv)
    rr, n_rows, rptr = _rows(rows)
    R = n_rows if rr is not None else Lq
    anchor = np.empty((B, Hq, R, top_k), dtype=np.int32)
    score = np.empty((B, Hq, R, top_k), dtype=np.float64)
    gap = np.empty((B, Hq, R), dtype=np.float64)
    n_dots = C.c_int64(0)
    rc = lib().sla_oracle_span_search(
        q_s.ctypes.data, k.ctypes.data, dtype, B, Hq, Hkv, D, Lq, int(q_pos0), Lkv, cap, int(top_k),
        int(window), float(search_scale), float(search_exponent), rptr, n_rows, anchor.ctypes.data, score.ctypes.data,
        gap.ctypes.data, C.addressof(n_dots))
    if rc:
        raise ValueError("sla_oracle_span_search rejected its arguments")
    return dict(anchor=anchor, score=score, gap=gap, n_dots=int(n_dots.value))


def span_attention(q, k, v, dtype, anchor, *, span_len, back_factor=2, fwd_factor=0, window=0,
                   mode=UNION, softmax_scale=None, q_pos0=0, Lkv=None, rows=None, score=None,
                   span_exponent=0.5):
    """q [B,Hq,Lq,D], k/v [B,Hkv,cap,D], anchor [B,Hq,R,k] -> dict(out, lse, lse_span, n_pairs)."""
    q, k, v = _as_input(q, dtype), _as_input(k, dtype), _as_input(v, dtype)
    B, Hq, Lq, D = q.shape
    _, Hkv, cap, _ = k.shape
    Lkv = cap if Lkv is None else int(Lkv)
    rr, n_rows, rptr = _rows(rows)
    R = n_rows if rr is not None else Lq
    anchor = np.ascontiguousarray(anchor, dtype=np.int32)
    top_k = anchor.shape[-1]
    assert anchor.shape == (B, Hq, R, top_k), (anchor.shape, (B, Hq, R, top_k))
    if score is not None:
        score = np.ascontiguousarray(score, dtype=np.float64)
        assert score.shape == anchor.shape
    if softmax_scale is None:
        softmax_scale = 1.0 / float(np.sqrt(D))
    out = np.empty((B, Hq, R, D), dtype=np.float64)
    lse = np.empty((B, Hq, R), dtype=np.float64)
    lse_span = np.empty((B, Hq, R, top_k), dtype=np.float64)
    n_pairs = C.c_int64(0)
    rc = lib().sla_oracle_span_attention(
        q.ctypes.data, k.ctypes.data, v.ctypes.data, dtype, B, Hq, Hkv, D, Lq, int(q_pos0), Lkv, cap,
        int(top_k), int(span_len), int(back_factor), int(fwd_factor), int(window), int(mode),
        float(softmax_scale), float(span_exponent), rptr, n_rows, anchor.ctypes.data,
        None if score is None else score.ctypes.data, out.ctypes.data, lse.ctypes.data,
        lse_span.ctypes.data, C.addressof(n_pairs))
    if rc:
        raise ValueError("sla_oracle_span_attention rejected its arguments")
    return dict(out=out, lse=lse, lse_span=lse_span, n_pairs=int(n_pairs.value))


def decode_step(q_s, q, k_cache, v_cache, dtype, *, n_ctx, top_k, span_len, back_factor=2,
                fwd_factor=0, window=0, mode=UNION, search_scale=1.0, softmax_scale=None,
                search_exponent=0.5, span_exponent=0.5):
    """q_s,q [B,Hq,D]; caches [B,Hkv,cap,D] -> dict(out, lse, anchor, score, gap, n_dots, n_pairs)."""
    q_s, q = _as_input(q_s, dtype), _as_input(q, dtype)
    k_cache, v_cache = _as_input(k_cache, dtype), _as_input(v_cache, dtype)
    B, Hq, D = q.shape
    _, Hkv, cap, _ = k_cache.shape
    if softmax_scale is None:
        softmax_scale = 1.0 / float(np.sqrt(D))
    anchor = np.empty((B, Hq, top_k), dtype=np.int32)
    score = np.empty((B, Hq, top_k), dtype=np.float64)
    gap = np.empty((B, Hq), dtype=np.float64)
    out = np.empty((B, Hq, D), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    n_dots, n_pairs = C.c_int64(0), C.c_int64(0)
    rc = lib().sla_oracle_decode_step(
        q_s.ctypes.data, q.ctypes.data, k_cache.ctypes.data, v_cache.ctypes.data, dtype, B, Hq, Hkv, D,
        int(n_ctx), cap, int(top_k), int(span_len), int(back_factor), int(fwd_factor), int(window),
        int(mode), float(search_scale), float(softmax_scale), float(search_exponent), float(span_exponent),
        anchor.ctypes.data, score.ctypes.data,
        gap.ctypes.data, out.ctypes.data, lse.ctypes.data, C.addressof(n_dots), C.addressof(n_pairs))
    if rc:
        raise ValueError("sla_oracle_decode_step rejected its arguments")
    return dict(out=out, lse=lse, anchor=anchor, score=score, gap=gap,
                n_dots=int(n_dots.value), n_pairs=int(n_pairs.value))
