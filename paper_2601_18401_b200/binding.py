"""Thin ctypes binding of ``libsla.so``: argument marshalling only.

Every function here has the name and the meaning of the C entry point it forwards to (see
``include/sla.h``); torch is used for device memory and streams, nothing else.  There is no
fallback: if the CUDA library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsla.so")

SLA_OK = 0
SLA_F32, SLA_BF16 = 0, 1
SLA_UNION, SLA_PER_SPAN = 0, 1
SLA_ERR_INVALID_ARG = -1

EXPORTS = [
    "sla_create", "sla_destroy", "sla_workspace_bytes", "sla_status_string", "sla_last_error",
    "sla_poll_status", "sla_span_search", "sla_span_attention", "sla_decode_step",
    "sla_host_staging_bytes", "sla_prefill_host", "sla_kernel_launches", "sla_set_kernel_timing",
    "sla_kernel_time_ms", "sla_decode_step_static", "sla_span_attention_gated",
    "sla_decode_shard_search", "sla_decode_shard_attend", "sla_decode_shard_merge",
    "sla_pattern_offsets", "sla_pattern_len_steps", "sla_probe_l2_read", "sla_selftest_wait_expiry",
    "sla_set_debug_canaries", "sla_selftest_canary_trip", "sla_attention_tile_stats",
]


class SlaError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{message} (status {status})")
        self.status = status


class sla_layout_t(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("dtype", C.c_int32), ("reserved", C.c_int32),
                ("q_stride_b", C.c_int64), ("q_stride_h", C.c_int64), ("q_stride_t", C.c_int64),
                ("kv_stride_b", C.c_int64), ("kv_stride_h", C.c_int64), ("kv_stride_t", C.c_int64)]


class sla_params_t(C.Structure):
    _fields_ = [("top_k", C.c_int32), ("span_len", C.c_int32), ("back_factor", C.c_int32),
                ("fwd_factor", C.c_int32), ("window", C.c_int32), ("mode", C.c_int32),
                ("search_scale", C.c_float), ("softmax_scale", C.c_float),
                ("search_exponent", C.c_double), ("span_exponent", C.c_double)]


_lib = None


def load_library():
    """Loads ``libsla.so`` from the package directory; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2601_18401_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i64, i32, sz = C.c_void_p, C.c_int64, C.c_int, C.c_size_t
    LP, PP = C.POINTER(sla_layout_t), C.POINTER(sla_params_t)
    lib.sla_create.restype = i32
    lib.sla_create.argtypes = [C.POINTER(vp), i32, sz]
    lib.sla_destroy.restype = i32
    lib.sla_destroy.argtypes = [vp]
    lib.sla_workspace_bytes.restype = sz
    lib.sla_workspace_bytes.argtypes = [LP, PP, i64, i64]
    lib.sla_status_string.restype = C.c_char_p
    lib.sla_status_string.argtypes = [i32]
    lib.sla_last_error.restype = C.c_char_p
    lib.sla_last_error.argtypes = [vp]
    lib.sla_poll_status.restype = i32
    lib.sla_poll_status.argtypes = [vp, vp]
    lib.sla_span_search.restype = i32
    lib.sla_span_search.argtypes = [vp, vp, vp, i64, i64, i64, LP, PP, vp, vp, vp]
    lib.sla_span_attention.restype = i32
    lib.sla_span_attention.argtypes = [vp, vp, vp, vp, i64, i64, i64, LP, PP, vp, vp, vp, vp]
    lib.sla_span_attention_gated.restype = i32
    lib.sla_span_attention_gated.argtypes = [vp, vp, vp, vp, i64, i64, i64, LP, PP, vp, vp, vp, vp, vp, vp]
    lib.sla_decode_shard_search.restype = i32
    lib.sla_decode_shard_search.argtypes = [vp, vp, vp, i64, i64, i64, LP, PP, vp, vp, vp]
    lib.sla_decode_shard_attend.restype = i32
    lib.sla_decode_shard_attend.argtypes = [vp, vp, vp, vp, i64, i64, i64, LP, PP, i32, vp, vp, vp, vp, vp, vp]
    lib.sla_decode_shard_merge.restype = i32
    lib.sla_decode_shard_merge.argtypes = [vp, i32, vp, LP, vp, vp, vp]
    lib.sla_decode_step.restype = i32
    lib.sla_decode_step.argtypes = [vp, vp, vp, vp, vp, i64, LP, PP, vp, vp, vp, vp, vp]
    lib.sla_decode_step_static.restype = i32
    lib.sla_decode_step_static.argtypes = [vp, vp, vp, vp, i64, LP, PP, vp, vp, vp, vp, vp]
    lib.sla_kernel_launches.restype = i64
    lib.sla_kernel_launches.argtypes = [vp]
    lib.sla_set_kernel_timing.restype = i32
    lib.sla_set_kernel_timing.argtypes = [vp, i32]
    lib.sla_kernel_time_ms.restype = i32
    lib.sla_kernel_time_ms.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.sla_host_staging_bytes.restype = sz
    lib.sla_host_staging_bytes.argtypes = [LP, PP, i64]
    lib.sla_prefill_host.restype = i32
    lib.sla_prefill_host.argtypes = [vp, vp, vp, vp, vp, i64, LP, PP, vp, vp, vp, vp, vp]
    lib.sla_attention_tile_stats.restype = i32
    lib.sla_attention_tile_stats.argtypes = [vp, vp, vp]
    lib.sla_set_debug_canaries.restype = i32
    lib.sla_set_debug_canaries.argtypes = [vp, i32]
    lib.sla_selftest_canary_trip.restype = i32
    lib.sla_selftest_canary_trip.argtypes = [vp, vp]
    lib.sla_probe_l2_read.restype = i32
    lib.sla_probe_l2_read.argtypes = [vp, vp, sz, C.c_int32, vp, vp]
    lib.sla_selftest_wait_expiry.restype = i32
    lib.sla_selftest_wait_expiry.argtypes = [vp, C.c_int32, vp, vp]
    lib.sla_pattern_offsets.restype = C.c_int32
    lib.sla_pattern_offsets.argtypes = [C.c_double, i64, vp, C.c_int32]
    lib.sla_pattern_len_steps.restype = C.c_int32
    lib.sla_pattern_len_steps.argtypes = [C.c_double, i64, vp, C.c_int32]
    _lib = lib
    return lib


def _pattern_table(fn, exponent: float, reach: int):
    n = fn(float(exponent), int(reach), None, 0)
    if n < 0:
        raise SlaError(SLA_ERR_INVALID_ARG, "exponent outside [0.2, 0.8] or more than 65536 entries")
    buf = (C.c_int32 * max(n, 1))()
    fn(float(exponent), int(reach), buf, n)
    return list(buf[:n])


def sla_pattern_offsets(search_exponent: float, reach: int):
    """Stride offsets ceil((s+1)^(1/p)) up to `reach`, as the library derives them (host-only)."""
    return _pattern_table(load_library().sla_pattern_offsets, search_exponent, reach)


def sla_pattern_len_steps(span_exponent: float, reach: int):
    """Positions at which l(i) = ceil(i^p) steps up, as the library derives them (host-only)."""
    return _pattern_table(load_library().sla_pattern_len_steps, span_exponent, reach)


def make_params(top_k: int, span_len: int, back_factor: int = 2, fwd_factor: int = 0, window: int = 0,
                mode: int = SLA_UNION, search_scale: float = 1.0,
                softmax_scale: Optional[float] = None, head_dim: int = 128,
                search_exponent: float = 0.5, span_exponent: float = 0.5) -> sla_params_t:
    if softmax_scale is None:
        softmax_scale = 1.0 / math.sqrt(head_dim)
    return sla_params_t(top_k, span_len, back_factor, fwd_factor, window, mode, search_scale, softmax_scale,
                        search_exponent, span_exponent)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SLA_F32
    if t.dtype == torch.bfloat16:
        return SLA_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def make_layout(q: torch.Tensor, k: torch.Tensor, decode: bool = False) -> sla_layout_t:
    """Layout struct from a query tensor ([B,Hq,L,D], or [B,Hq,D] for decode) and a key tensor [B,Hkv,L,D]."""
    if q.stride(-1) != 1 or k.stride(-1) != 1:
        raise ValueError("head_dim axis must be contiguous")
    B, Hq, D = q.shape[0], q.shape[1], q.shape[-1]
    Hkv = k.shape[1]
    return sla_layout_t(B, Hq, Hkv, D, _dtype_code(q), 0,
                        q.stride(0), q.stride(1), 0 if decode else q.stride(2),
                        k.stride(0), k.stride(1), k.stride(2))


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


class Handle:
    """Owns an ``sla_handle_t`` (and with it the library's device workspace)."""

    def __init__(self, device: int = 0, workspace_bytes: int = 64 << 20):
        self._lib = load_library()
        self._h = C.c_void_p()
        self.device = int(device)
        with torch.cuda.device(self.device):
            rc = self._lib.sla_create(C.byref(self._h), self.device, int(workspace_bytes))
        if rc != SLA_OK:
            raise SlaError(rc, "sla_create failed: " + self._lib.sla_status_string(rc).decode())
        self.workspace_bytes = int(workspace_bytes)

    def check(self, rc: int, what: str):
        if rc != SLA_OK:
            raise SlaError(rc, f"{what}: {self._lib.sla_status_string(rc).decode()}: "
                               f"{self._lib.sla_last_error(self._h).decode()}")

    @property
    def ptr(self):
        return self._h

    def close(self):
        if self._h:
            self._lib.sla_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def sla_workspace_bytes(layout: sla_layout_t, params: sla_params_t, Lq: int, Lkv: int) -> int:
    return int(load_library().sla_workspace_bytes(C.byref(layout), C.byref(params), int(Lq), int(Lkv)))


def sla_host_staging_bytes(layout: sla_layout_t, params: sla_params_t, L: int) -> int:
    return int(load_library().sla_host_staging_bytes(C.byref(layout), C.byref(params), int(L)))


def sla_kernel_launches(handle: Handle) -> int:
    return int(handle._lib.sla_kernel_launches(handle.ptr))


def sla_set_kernel_timing(handle: Handle, enable: bool) -> None:
    handle.check(handle._lib.sla_set_kernel_timing(handle.ptr, int(bool(enable))), "sla_set_kernel_timing")


def sla_kernel_time_ms(handle: Handle):
    """(milliseconds, launches) of the main attention kernel since the previous read."""
    ms, n = C.c_float(0.0), C.c_int32(0)
    handle.check(handle._lib.sla_kernel_time_ms(handle.ptr, C.byref(ms), C.byref(n)), "sla_kernel_time_ms")
    return float(ms.value), int(n.value)


def sla_attention_tile_stats(handle: Handle, stream=None) -> dict:
    """Tiles, pieces and key blocks walked by the most recent tensor-core span-attention call (last chunk)."""
    buf = (C.c_int64 * 4)()
    handle.check(handle._lib.sla_attention_tile_stats(handle.ptr, buf, _stream_ptr(stream)), "sla_attention_tile_stats")
    return {"tiles": int(buf[0]), "pieces": int(buf[1]), "tile_blocks": int(buf[2]), "piece_blocks": int(buf[3])}


def sla_set_debug_canaries(handle: Handle, enable: bool) -> None:
    handle.check(handle._lib.sla_set_debug_canaries(handle.ptr, int(bool(enable))), "sla_set_debug_canaries")


def sla_selftest_canary_trip(handle: Handle, stream=None) -> None:
    handle.check(handle._lib.sla_selftest_canary_trip(handle.ptr, _stream_ptr(stream)), "sla_selftest_canary_trip")


def sla_probe_l2_read(handle: Handle, buf: torch.Tensor, iters: int, stream=None) -> int:
    """Launches the read-only L2 probe over `buf` (device, contiguous); returns the bytes it reads."""
    nbytes = buf.numel() * buf.element_size()
    handle.check(handle._lib.sla_probe_l2_read(handle.ptr, buf.data_ptr(), nbytes, int(iters), None, _stream_ptr(stream)),
                 "sla_probe_l2_read")
    sms = torch.cuda.get_device_properties(buf.device).multi_processor_count
    return 4 * sms * nbytes * int(iters)


def sla_selftest_wait_expiry(handle: Handle, max_polls: int = 2000, polls_done: Optional[torch.Tensor] = None,
                             stream=None) -> None:
    """Makes a bounded device-side wait run out on purpose-built barrier nothing arrives on (see sla.h)."""
    handle.check(handle._lib.sla_selftest_wait_expiry(handle.ptr, int(max_polls),
                                                     None if polls_done is None else polls_done.data_ptr(),
                                                     _stream_ptr(stream)), "sla_selftest_wait_expiry")


def sla_poll_status(handle: Handle, stream=None) -> int:
    return int(handle._lib.sla_poll_status(handle.ptr, _stream_ptr(stream)))


def sla_span_search(handle: Handle, q_s: torch.Tensor, k: torch.Tensor, params: sla_params_t, *,
                    q_pos0: int = 0, Lkv: Optional[int] = None, out_anchor=None, out_score=None, stream=None):
    """q_s [B,Hq,Lq,D], k [B,Hkv,>=Lkv,D] (device) -> anchors int32 [B,Hq,Lq,k], scores fp32 [B,Hq,Lq,k]."""
    B, Hq, Lq, _ = q_s.shape
    Lkv = k.shape[2] if Lkv is None else int(Lkv)
    if out_anchor is None:
        out_anchor = torch.empty(B, Hq, Lq, params.top_k, dtype=torch.int32, device=q_s.device)
    if out_score is None:
        out_score = torch.empty(B, Hq, Lq, params.top_k, dtype=torch.float32, device=q_s.device)
    layout = make_layout(q_s, k)
    rc = handle._lib.sla_span_search(handle.ptr, q_s.data_ptr(), k.data_ptr(), Lq, int(q_pos0), Lkv,
                                     C.byref(layout), C.byref(params), out_anchor.data_ptr(),
                                     out_score.data_ptr(), _stream_ptr(stream))
    handle.check(rc, "sla_span_search")
    return out_anchor, out_score


def sla_span_attention(handle: Handle, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                       anchor: torch.Tensor, params: sla_params_t, *, q_pos0: int = 0,
                       Lkv: Optional[int] = None, out=None, lse=None, stream=None):
    """q [B,Hq,Lq,D], k/v [B,Hkv,>=Lkv,D], anchor int32 [B,Hq,Lq,k] -> out (q's dtype and strides), lse fp32."""
    B, Hq, Lq, _ = q.shape
    Lkv = k.shape[2] if Lkv is None else int(Lkv)
    if k.stride() != v.stride():
        raise ValueError("k and v must share their strides")
    if not anchor.is_contiguous() or anchor.dtype != torch.int32:
        raise ValueError("anchor must be a contiguous int32 tensor")
    if out is None:
        out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=q.device)
    if lse is None:
        lse = torch.empty(B, Hq, Lq, dtype=torch.float32, device=q.device)
    layout = make_layout(q, k)
    rc = handle._lib.sla_span_attention(handle.ptr, q.data_ptr(), k.data_ptr(), v.data_ptr(), Lq,
                                        int(q_pos0), Lkv, C.byref(layout), C.byref(params),
                                        anchor.data_ptr(), out.data_ptr(), lse.data_ptr(), _stream_ptr(stream))
    handle.check(rc, "sla_span_attention")
    return out, lse


def sla_span_attention_gated(handle: Handle, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                             anchor: torch.Tensor, score: torch.Tensor, params: sla_params_t, *,
                             q_pos0: int = 0, Lkv: Optional[int] = None, out=None, lse=None, lse_span=None,
                             stream=None):
    """Per-span softmax and gate (params.mode = SLA_PER_SPAN): anchor int32 and score fp32 [B,Hq,Lq,k]
    -> out (q's dtype and strides), lse fp32 [B,Hq,Lq], lse_span fp32 [B,Hq,Lq,k]."""
    B, Hq, Lq, D = q.shape
    Lkv = k.shape[2] if Lkv is None else int(Lkv)
    assert anchor.dtype == torch.int32 and anchor.is_contiguous() and anchor.shape[:3] == (B, Hq, Lq)
    assert score.dtype == torch.float32 and score.is_contiguous() and score.shape == anchor.shape
    if out is None:
        out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=q.device)
    if lse is None:
        lse = torch.empty(B, Hq, Lq, dtype=torch.float32, device=q.device)
    if lse_span is None:
        lse_span = torch.empty(anchor.shape, dtype=torch.float32, device=q.device)
    layout = make_layout(q, k)
    rc = handle._lib.sla_span_attention_gated(handle.ptr, q.data_ptr(), k.data_ptr(), v.data_ptr(), Lq,
                                              int(q_pos0), Lkv, C.byref(layout), C.byref(params),
                                              anchor.data_ptr(), score.data_ptr(), out.data_ptr(),
                                              lse.data_ptr(), lse_span.data_ptr(), _stream_ptr(stream))
    handle.check(rc, "sla_span_attention_gated")
    return out, lse, lse_span


def sla_decode_step(handle: Handle, q_s: torch.Tensor, q: torch.Tensor, k_cache: torch.Tensor,
                    v_cache: torch.Tensor, n_ctx: int, params: sla_params_t, *, out=None, lse=None,
                    out_anchor=None, out_score=None, stream=None):
    """q_s, q [B,Hq,D]; caches [B,Hkv,cap,D] -> out [B,Hq,D], lse [B,Hq], anchors/scores [B,Hq,k]."""
    B, Hq, _ = q.shape
    if q_s.stride() != q.stride() or k_cache.stride() != v_cache.stride():
        raise ValueError("q_s/q and k_cache/v_cache must share their strides")
    dev = q.device
    out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=dev) if out is None else out
    lse = torch.empty(B, Hq, dtype=torch.float32, device=dev) if lse is None else lse
    out_anchor = torch.empty(B, Hq, params.top_k, dtype=torch.int32, device=dev) if out_anchor is None else out_anchor
    out_score = torch.empty(B, Hq, params.top_k, dtype=torch.float32, device=dev) if out_score is None else out_score
    layout = make_layout(q, k_cache, decode=True)
    rc = handle._lib.sla_decode_step(handle.ptr, q_s.data_ptr(), q.data_ptr(), k_cache.data_ptr(),
                                     v_cache.data_ptr(), int(n_ctx), C.byref(layout), C.byref(params),
                                     out.data_ptr(), lse.data_ptr(), out_anchor.data_ptr(),
                                     out_score.data_ptr(), _stream_ptr(stream))
    handle.check(rc, "sla_decode_step")
    return out, lse, out_anchor, out_score


def sla_decode_step_static(q_s: torch.Tensor, q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                           n_ctx: int, params: sla_params_t, *, out, lse, out_anchor, out_score, stream=None):
    """The decode step for callers that may not allocate: no handle, scratch inside the library image,
    and every output buffer supplied by the caller (this wrapper allocates nothing either)."""
    if q_s.stride() != q.stride() or k_cache.stride() != v_cache.stride() or out.stride() != q.stride():
        raise ValueError("q_s/q/out and k_cache/v_cache must share their strides")
    lib = load_library()
    layout = make_layout(q, k_cache, decode=True)
    rc = lib.sla_decode_step_static(q_s.data_ptr(), q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), int(n_ctx),
                                    C.byref(layout), C.byref(params), out.data_ptr(), lse.data_ptr(),
                                    out_anchor.data_ptr(), out_score.data_ptr(), _stream_ptr(stream))
    if rc != SLA_OK:
        what = {-3: "the step needs more scratch than the fixed array inside the library holds"}.get(rc, "call rejected")
        raise SlaError(rc, f"sla_decode_step_static: {lib.sla_status_string(rc).decode()}: {what}")
    return out, lse, out_anchor, out_score


def sla_prefill_host(handle: Handle, q_s: torch.Tensor, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                     params: sla_params_t, *, out=None, lse=None, anchor=None, score=None, stream=None):
    """Host tensors in (ideally pinned), host tensors out; copies both ways happen inside the C call."""
    for t in (q_s, q, k, v):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("sla_prefill_host takes contiguous host tensors")
    B, Hq, L, D = q.shape
    pin = q.is_pinned()
    out = torch.empty(q.shape, dtype=q.dtype, pin_memory=pin) if out is None else out
    lse = torch.empty(B, Hq, L, dtype=torch.float32, pin_memory=pin) if lse is None else lse
    anchor = torch.empty(B, Hq, L, params.top_k, dtype=torch.int32, pin_memory=pin) if anchor is None else anchor
    score = torch.empty(B, Hq, L, params.top_k, dtype=torch.float32, pin_memory=pin) if score is None else score
    layout = make_layout(q, k)
    rc = handle._lib.sla_prefill_host(handle.ptr, q_s.data_ptr(), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                      L, C.byref(layout), C.byref(params), out.data_ptr(), lse.data_ptr(),
                                      anchor.data_ptr(), score.data_ptr(), _stream_ptr(stream))
    handle.check(rc, "sla_prefill_host")
    return out, lse, anchor, score


def sla_decode_shard_search(handle: Handle, q_s: torch.Tensor, k_local: torch.Tensor, shard_lo: int, n_ctx: int,
                            params: sla_params_t, *, shard_len: Optional[int] = None, stream=None):
    """q_s [B,Hq,D]; k_local [B,Hkv,>=shard_len,D] holds positions shard_lo.. -> this rank's candidates
    (anchor int32, score fp32) [B,Hq,k]."""
    B, Hq, _ = q_s.shape
    shard_len = k_local.shape[2] if shard_len is None else int(shard_len)
    anchor = torch.empty(B, Hq, params.top_k, dtype=torch.int32, device=q_s.device)
    score = torch.empty(B, Hq, params.top_k, dtype=torch.float32, device=q_s.device)
    layout = make_layout(q_s, k_local, decode=True)
    rc = handle._lib.sla_decode_shard_search(handle.ptr, q_s.data_ptr(), k_local.data_ptr(), int(shard_lo), shard_len,
                                             int(n_ctx), C.byref(layout), C.byref(params), anchor.data_ptr(),
                                             score.data_ptr(), _stream_ptr(stream))
    handle.check(rc, "sla_decode_shard_search")
    return anchor, score


def sla_decode_shard_attend(handle: Handle, q: torch.Tensor, k_local: torch.Tensor, v_local: torch.Tensor,
                            shard_lo: int, n_ctx: int, params: sla_params_t, all_anchor: torch.Tensor,
                            all_score: torch.Tensor, *, shard_len: Optional[int] = None, stream=None):
    """all_anchor / all_score [n_shards,B,Hq,k] (gathered candidates) -> out_anchor, out_score [B,Hq,k] and
    this rank's partial result [B,Hq,D+2] fp32."""
    B, Hq, D = q.shape
    n_shards = all_anchor.shape[0]
    assert all_anchor.is_contiguous() and all_score.is_contiguous() and all_anchor.dtype == torch.int32
    assert all_score.dtype == torch.float32 and all_anchor.shape == (n_shards, B, Hq, params.top_k) == all_score.shape
    shard_len = k_local.shape[2] if shard_len is None else int(shard_len)
    out_anchor = torch.empty(B, Hq, params.top_k, dtype=torch.int32, device=q.device)
    out_score = torch.empty(B, Hq, params.top_k, dtype=torch.float32, device=q.device)
    partial = torch.empty(B, Hq, D + 2, dtype=torch.float32, device=q.device)
    layout = make_layout(q, k_local, decode=True)
    rc = handle._lib.sla_decode_shard_attend(handle.ptr, q.data_ptr(), k_local.data_ptr(), v_local.data_ptr(),
                                             int(shard_lo), shard_len, int(n_ctx), C.byref(layout), C.byref(params),
                                             n_shards, all_anchor.data_ptr(), all_score.data_ptr(),
                                             out_anchor.data_ptr(), out_score.data_ptr(), partial.data_ptr(),
                                             _stream_ptr(stream))
    handle.check(rc, "sla_decode_shard_attend")
    return out_anchor, out_score, partial


def sla_decode_shard_merge(handle: Handle, all_partial: torch.Tensor, q_like: torch.Tensor, *, stream=None):
    """all_partial [n_shards,B,Hq,D+2] fp32 (gathered) -> out [B,Hq,D] (dtype and strides of q_like), lse [B,Hq]."""
    n_shards, B, Hq, D2 = all_partial.shape
    assert all_partial.is_contiguous() and all_partial.dtype == torch.float32 and D2 == q_like.shape[-1] + 2
    out = torch.empty_strided(q_like.shape, q_like.stride(), dtype=q_like.dtype, device=q_like.device)
    lse = torch.empty(B, Hq, dtype=torch.float32, device=q_like.device)
    layout = make_layout(q_like, q_like.new_empty(B, 1, 1, q_like.shape[-1]), decode=True)
    rc = handle._lib.sla_decode_shard_merge(handle.ptr, n_shards, all_partial.data_ptr(), C.byref(layout),
                                            out.data_ptr(), lse.data_ptr(), _stream_ptr(stream))
    handle.check(rc, "sla_decode_shard_merge")
    return out, lse
