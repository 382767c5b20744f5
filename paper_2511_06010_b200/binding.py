"""Thin ctypes binding of libmoska.so: one Python function per C entry point, same names.

Argument marshalling only: tensors are passed as device pointers, the stream is torch's current
stream unless given.  There is no fallback: if the CUDA library cannot be loaded, importing this
module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MOSKA_LIB names another build of the library (same ABI) to load instead of the in-tree one.
LIB_PATH = os.environ.get("MOSKA_LIB") or os.path.join(_HERE, "csrc", "libmoska.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2511_06010_b200.build` "
        "(there is no CPU or PyTorch fallback)")

_lib = ctypes.CDLL(LIB_PATH)


class MoskaShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "Hq", "Hkv", "D", "C", "L", "k", "shared_slots", "n_unique_splits")] + \
               [("unique_tokens", ctypes.c_int64), ("q_len", ctypes.c_int32)]


class MoskaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status}: {last_error()}")


OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
ERR_CORRUPT = -6

_vp, _sz, _f, _i = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_float, ctypes.c_int
_sp = ctypes.POINTER(MoskaShape)

EXPORTS = {
    "moska_version": (_i, []),
    "moska_last_error": (ctypes.c_char_p, []),
    "moska_device_status": (_i, [ctypes.POINTER(ctypes.c_int32)]),
    "moska_partial_slots": (_i, [_sp]),
    "moska_workspace_bytes": (_sz, [_sp]),
    "moska_default_unique_splits": (_i, [ctypes.c_int32] * 3),
    "moska_default_unique_splits_fp8": (_i, [ctypes.c_int32] * 3),
    "moska_build_chunk_summaries": (_i, [_vp, _vp, _sp, _vp]),
    "moska_build_chunk_summaries_attn": (_i, [_vp, _vp, _f, _sp, _vp]),
    "moska_route": (_i, [_vp, _vp, _vp, _vp, _sp, _vp, _sz, _vp]),
    "moska_group_by_chunk": (_i, [_vp, _vp, _vp, _sp, _vp, _sz, _vp]),
    "moska_group_by_chunk_noalloc": (_i, [_vp, _vp, _vp, _sp, _vp]),
    "moska_debug_check_workspace": (_i, [_vp, _sz, _sp, _vp]),
    "moska_shared_attn": (_i, [_vp] * 8 + [_f, _sp, _vp, _sz, _vp]),
    "moska_shared_attn_fp8": (_i, [_vp] * 10 + [_f, _sp, _vp, _sz, _vp]),
    "moska_unique_attn": (_i, [_vp] * 7 + [_f, _sp, _vp]),
    "moska_unique_attn_fp8": (_i, [_vp] * 9 + [_f, _sp, _vp]),
    "moska_merge": (_i, [_vp] * 5 + [_sp, _vp]),
    "moska_gemv_baseline": (_i, [_vp] * 6 + [_f, _sp, _vp]),
    "moska_decode_step": (_i, [_vp] * 15 + [_f, _sp, _vp, _sz, _vp, _vp, _vp]),
    "moska_decode_step_fp8kv": (_i, [_vp] * 17 + [_f, _sp, _vp, _sz, _vp, _vp, _vp]),
    "moska_decode_step_fp8shared": (_i, [_vp] * 17 + [_f, _sp, _vp, _sz, _vp, _vp, _vp]),
    "moska_decode_step_fp8": (_i, [_vp] * 19 + [_f, _sp, _vp, _sz, _vp, _vp, _vp]),
    "moska_decode_step_host": (_i, [_vp] * 16 + [_f, _sp, _vp, _sz, _vp, _vp, _vp]),
    "moska_decode_step_fp8_host": (_i, [_vp] * 20 + [_f, _sp, _vp, _sz, _vp, _vp, _vp]),
    "moska_profiler_create": (_i, [ctypes.POINTER(_vp), ctypes.c_int32]),
    "moska_profiler_destroy": (None, [_vp]),
    "moska_profiler_select": (_i, [_vp, ctypes.c_uint32]),
    "moska_profiler_read": (_i, [_vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)]),
}
for _name, (_res, _args) in EXPORTS.items():
    _fn = getattr(_lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


def shape(B, Hq, Hkv, D, C, L, k, shared_slots=None, n_unique_splits=1, q_len=0) -> MoskaShape:
    return MoskaShape(B, Hq, Hkv, D, C, L, k, k if shared_slots is None else shared_slots,
                      n_unique_splits, 0, q_len)


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a tensor, None for NULL, or a raw integer address."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors cross the C ABI as dense row-major buffers"
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(status: int, where: str) -> None:
    if status != OK:
        raise MoskaError(status, where)


def version() -> int:
    return _lib.moska_version()


def last_error() -> str:
    return _lib.moska_last_error().decode()


def device_status() -> int:
    """Synchronises the device; returns (and clears) the sticky device-side status word."""
    v = ctypes.c_int32(0)
    _check(_lib.moska_device_status(ctypes.byref(v)), "moska_device_status")
    return v.value


def partial_slots(s: MoskaShape) -> int:
    n = _lib.moska_partial_slots(ctypes.byref(s))
    if n < 0:
        raise MoskaError(n, "moska_partial_slots")
    return n


def workspace_bytes(s: MoskaShape) -> int:
    return _lib.moska_workspace_bytes(ctypes.byref(s))


def default_unique_splits(B: int, Hkv: int, max_len: int) -> int:
    return _lib.moska_default_unique_splits(B, Hkv, max_len)


def default_unique_splits_fp8(B: int, Hkv: int, max_len: int) -> int:
    return _lib.moska_default_unique_splits_fp8(B, Hkv, max_len)


def build_chunk_summaries(k_shared, summaries, s, stream=None) -> None:
    _check(_lib.moska_build_chunk_summaries(_ptr(k_shared), _ptr(summaries), ctypes.byref(s),
                                            _stream(stream)), "moska_build_chunk_summaries")


def build_chunk_summaries_attn(k_shared, summaries, probe_scale, s, stream=None) -> None:
    _check(_lib.moska_build_chunk_summaries_attn(_ptr(k_shared), _ptr(summaries), probe_scale,
                                                 ctypes.byref(s), _stream(stream)),
           "moska_build_chunk_summaries_attn")


def route(q, summaries, topk_idx, topk_score, s, ws=None, stream=None) -> None:
    _check(_lib.moska_route(_ptr(q), _ptr(summaries), _ptr(topk_idx), _ptr(topk_score),
                            ctypes.byref(s), _ptr(ws),
                            0 if ws is None else ws.numel() * ws.element_size(),
                            _stream(stream)), "moska_route")


def group_by_chunk(topk_idx, seg_offsets, seg_entries, s, ws, stream=None) -> None:
    _check(_lib.moska_group_by_chunk(_ptr(topk_idx), _ptr(seg_offsets), _ptr(seg_entries),
                                     ctypes.byref(s), _ptr(ws), ws.numel() * ws.element_size(),
                                     _stream(stream)), "moska_group_by_chunk")


def group_by_chunk_noalloc(topk_idx, seg_offsets, seg_entries, s, stream=None) -> None:
    """Grouping with the library's built-in scratch buffer: for callers that must not allocate
    device memory (no workspace argument; shapes beyond the buffer raise ERR_WORKSPACE)."""
    _check(_lib.moska_group_by_chunk_noalloc(_ptr(topk_idx), _ptr(seg_offsets), _ptr(seg_entries),
                                             ctypes.byref(s), _stream(stream)),
           "moska_group_by_chunk_noalloc")


def debug_check_workspace(ws, s, stream=None) -> None:
    """Debug build of the library only: compares the workspace's guard words (a mismatch shows as
    ERR_CORRUPT in device_status()); the regular build raises ERR_UNSUPPORTED."""
    _check(_lib.moska_debug_check_workspace(_ptr(ws), ws.numel() * ws.element_size(), ctypes.byref(s),
                                            _stream(stream)), "moska_debug_check_workspace")


def shared_attn(q, k_shared, v_shared, topk_idx, seg_offsets, seg_entries, o_part, lse_part,
                softmax_scale, s, ws, stream=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(_lib.moska_shared_attn(_ptr(q), _ptr(k_shared), _ptr(v_shared), _ptr(topk_idx),
                                  _ptr(seg_offsets), _ptr(seg_entries), _ptr(o_part),
                                  _ptr(lse_part), softmax_scale, ctypes.byref(s), _ptr(ws),
                                  ws_bytes, _stream(stream)), "moska_shared_attn")


def shared_attn_fp8(q, k8_shared, v8_shared, k_scale, v_scale, topk_idx, seg_offsets, seg_entries, o_part,
                    lse_part, softmax_scale, s, ws, stream=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(_lib.moska_shared_attn_fp8(_ptr(q), _ptr(k8_shared), _ptr(v8_shared), _ptr(k_scale), _ptr(v_scale),
                                      _ptr(topk_idx), _ptr(seg_offsets), _ptr(seg_entries), _ptr(o_part),
                                      _ptr(lse_part), softmax_scale, ctypes.byref(s), _ptr(ws), ws_bytes,
                                      _stream(stream)), "moska_shared_attn_fp8")


def unique_attn(q, k_unique, v_unique, kv_start, kv_len, o_part, lse_part, softmax_scale, s,
                stream=None) -> None:
    _check(_lib.moska_unique_attn(_ptr(q), _ptr(k_unique), _ptr(v_unique), _ptr(kv_start),
                                  _ptr(kv_len), _ptr(o_part), _ptr(lse_part), softmax_scale,
                                  ctypes.byref(s), _stream(stream)), "moska_unique_attn")


def unique_attn_fp8(q, k8, v8, k_scale, v_scale, kv_start, kv_len, o_part, lse_part, softmax_scale,
                    s, stream=None) -> None:
    _check(_lib.moska_unique_attn_fp8(_ptr(q), _ptr(k8), _ptr(v8), _ptr(k_scale), _ptr(v_scale),
                                      _ptr(kv_start), _ptr(kv_len), _ptr(o_part), _ptr(lse_part),
                                      softmax_scale, ctypes.byref(s), _stream(stream)),
           "moska_unique_attn_fp8")


def merge(o_part, lse_part, out, out_f32, lse_out, s, stream=None) -> None:
    _check(_lib.moska_merge(_ptr(o_part), _ptr(lse_part), _ptr(out), _ptr(out_f32),
                            _ptr(lse_out), ctypes.byref(s), _stream(stream)), "moska_merge")


def gemv_baseline(q, k_shared, v_shared, topk_idx, o_part, lse_part, softmax_scale, s,
                  stream=None) -> None:
    _check(_lib.moska_gemv_baseline(_ptr(q), _ptr(k_shared), _ptr(v_shared), _ptr(topk_idx),
                                    _ptr(o_part), _ptr(lse_part), softmax_scale, ctypes.byref(s),
                                    _stream(stream)), "moska_gemv_baseline")


def decode_step(q, summaries, k_shared, v_shared, k_unique, v_unique, kv_start, kv_len, topk_idx,
                seg_offsets, seg_entries, o_part, lse_part, out, lse_out, softmax_scale, s, ws,
                stream=None, side_stream=None, prof=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(_lib.moska_decode_step(
        _ptr(q), _ptr(summaries), _ptr(k_shared), _ptr(v_shared), _ptr(k_unique), _ptr(v_unique),
        _ptr(kv_start), _ptr(kv_len), _ptr(topk_idx), _ptr(seg_offsets), _ptr(seg_entries),
        _ptr(o_part), _ptr(lse_part), _ptr(out), _ptr(lse_out), softmax_scale, ctypes.byref(s),
        _ptr(ws), ws_bytes, _stream(stream),
        None if side_stream is None else _stream(side_stream), prof), "moska_decode_step")


def decode_step_fp8kv(q, summaries, k_shared, v_shared, k8_unique, v8_unique, k_scale, v_scale,
                      kv_start, kv_len, topk_idx, seg_offsets, seg_entries, o_part, lse_part, out,
                      lse_out, softmax_scale, s, ws, stream=None, side_stream=None, prof=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(_lib.moska_decode_step_fp8kv(
        _ptr(q), _ptr(summaries), _ptr(k_shared), _ptr(v_shared), _ptr(k8_unique), _ptr(v8_unique),
        _ptr(k_scale), _ptr(v_scale), _ptr(kv_start), _ptr(kv_len), _ptr(topk_idx),
        _ptr(seg_offsets), _ptr(seg_entries), _ptr(o_part), _ptr(lse_part), _ptr(out),
        _ptr(lse_out), softmax_scale, ctypes.byref(s), _ptr(ws), ws_bytes, _stream(stream),
        None if side_stream is None else _stream(side_stream), prof), "moska_decode_step_fp8kv")


def decode_step_fp8shared(q, summaries, k8_shared, v8_shared, k_scale_shared, v_scale_shared, k_unique,
                          v_unique, kv_start, kv_len, topk_idx, seg_offsets, seg_entries, o_part, lse_part, out,
                          lse_out, softmax_scale, s, ws, stream=None, side_stream=None, prof=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(_lib.moska_decode_step_fp8shared(
        _ptr(q), _ptr(summaries), _ptr(k8_shared), _ptr(v8_shared), _ptr(k_scale_shared),
        _ptr(v_scale_shared), _ptr(k_unique), _ptr(v_unique), _ptr(kv_start), _ptr(kv_len), _ptr(topk_idx),
        _ptr(seg_offsets), _ptr(seg_entries), _ptr(o_part), _ptr(lse_part), _ptr(out), _ptr(lse_out),
        softmax_scale, ctypes.byref(s), _ptr(ws), ws_bytes, _stream(stream),
        None if side_stream is None else _stream(side_stream), prof), "moska_decode_step_fp8shared")


def decode_step_fp8(q, summaries, k8_shared, v8_shared, k_scale_shared, v_scale_shared, k8_unique, v8_unique,
                    k_scale_unique, v_scale_unique, kv_start, kv_len, topk_idx, seg_offsets, seg_entries,
                    o_part, lse_part, out, lse_out, softmax_scale, s, ws, stream=None, side_stream=None,
                    prof=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(_lib.moska_decode_step_fp8(
        _ptr(q), _ptr(summaries), _ptr(k8_shared), _ptr(v8_shared), _ptr(k_scale_shared),
        _ptr(v_scale_shared), _ptr(k8_unique), _ptr(v8_unique), _ptr(k_scale_unique), _ptr(v_scale_unique),
        _ptr(kv_start), _ptr(kv_len), _ptr(topk_idx), _ptr(seg_offsets), _ptr(seg_entries), _ptr(o_part),
        _ptr(lse_part), _ptr(out), _ptr(lse_out), softmax_scale, ctypes.byref(s), _ptr(ws), ws_bytes,
        _stream(stream), None if side_stream is None else _stream(side_stream), prof),
        "moska_decode_step_fp8")


def decode_step_host(q_host, q_dev, summaries, k_shared, v_shared, k_unique, v_unique, kv_start,
                     kv_len, topk_idx, seg_offsets, seg_entries, o_part, lse_part, out_dev,
                     out_host, softmax_scale, s, ws, stream=None, side_stream=None,
                     prof=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(_lib.moska_decode_step_host(
        _ptr(q_host), _ptr(q_dev), _ptr(summaries), _ptr(k_shared), _ptr(v_shared),
        _ptr(k_unique), _ptr(v_unique), _ptr(kv_start), _ptr(kv_len), _ptr(topk_idx),
        _ptr(seg_offsets), _ptr(seg_entries), _ptr(o_part), _ptr(lse_part), _ptr(out_dev),
        _ptr(out_host), softmax_scale, ctypes.byref(s), _ptr(ws), ws_bytes, _stream(stream),
        None if side_stream is None else _stream(side_stream), prof), "moska_decode_step_host")


def bind_decode_step_host(q_host, q_dev, summaries, k_shared, v_shared, k_unique, v_unique, kv_start,
                          kv_len, topk_idx, seg_offsets, seg_entries, o_part, lse_part, out_dev,
                          out_host, softmax_scale, s, ws, stream=None, side_stream=None, prof=None):
    """decode_step_host with its arguments marshalled once: returns a callable for a serving loop
    that repeats the call on the same buffers (the tensors must stay alive and in place; the shape
    struct is passed by reference, so later changes of its fields are seen)."""
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    args = (_ptr(q_host), _ptr(q_dev), _ptr(summaries), _ptr(k_shared), _ptr(v_shared),
            _ptr(k_unique), _ptr(v_unique), _ptr(kv_start), _ptr(kv_len), _ptr(topk_idx),
            _ptr(seg_offsets), _ptr(seg_entries), _ptr(o_part), _ptr(lse_part), _ptr(out_dev),
            _ptr(out_host), softmax_scale, ctypes.byref(s), _ptr(ws), ws_bytes, _stream(stream),
            None if side_stream is None else _stream(side_stream), prof)
    fn = _lib.moska_decode_step_host

    def call() -> None:
        status = fn(*args)
        if status != OK:
            raise MoskaError(status, "moska_decode_step_host")

    return call


def decode_step_fp8_host(q_host, q_dev, summaries, k8_shared, v8_shared, k_scale_shared, v_scale_shared,
                         k8_unique, v8_unique, k_scale_unique, v_scale_unique, kv_start, kv_len, topk_idx,
                         seg_offsets, seg_entries, o_part, lse_part, out_dev, out_host, softmax_scale, s, ws,
                         stream=None, side_stream=None, prof=None) -> None:
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check(_lib.moska_decode_step_fp8_host(
        _ptr(q_host), _ptr(q_dev), _ptr(summaries), _ptr(k8_shared), _ptr(v8_shared), _ptr(k_scale_shared),
        _ptr(v_scale_shared), _ptr(k8_unique), _ptr(v8_unique), _ptr(k_scale_unique), _ptr(v_scale_unique),
        _ptr(kv_start), _ptr(kv_len), _ptr(topk_idx), _ptr(seg_offsets), _ptr(seg_entries), _ptr(o_part),
        _ptr(lse_part), _ptr(out_dev), _ptr(out_host), softmax_scale, ctypes.byref(s), _ptr(ws), ws_bytes,
        _stream(stream), None if side_stream is None else _stream(side_stream), prof),
        "moska_decode_step_fp8_host")


def bind_decode_step_fp8_host(q_host, q_dev, summaries, k8_shared, v8_shared, k_scale_shared, v_scale_shared,
                              k8_unique, v8_unique, k_scale_unique, v_scale_unique, kv_start, kv_len,
                              topk_idx, seg_offsets, seg_entries, o_part, lse_part, out_dev, out_host,
                              softmax_scale, s, ws, stream=None, side_stream=None, prof=None):
    """decode_step_fp8_host with its arguments marshalled once (see bind_decode_step_host)."""
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    args = (_ptr(q_host), _ptr(q_dev), _ptr(summaries), _ptr(k8_shared), _ptr(v8_shared),
            _ptr(k_scale_shared), _ptr(v_scale_shared), _ptr(k8_unique), _ptr(v8_unique),
            _ptr(k_scale_unique), _ptr(v_scale_unique), _ptr(kv_start), _ptr(kv_len), _ptr(topk_idx),
            _ptr(seg_offsets), _ptr(seg_entries), _ptr(o_part), _ptr(lse_part), _ptr(out_dev),
            _ptr(out_host), softmax_scale, ctypes.byref(s), _ptr(ws), ws_bytes, _stream(stream),
            None if side_stream is None else _stream(side_stream), prof)
    fn = _lib.moska_decode_step_fp8_host

    def call() -> None:
        status = fn(*args)
        if status != OK:
            raise MoskaError(status, "moska_decode_step_fp8_host")

    return call


STAGES = ("route", "group", "shared", "unique", "merge")


def profiler_create(max_steps: int):
    """-> opaque profiler handle (pass as `prof=` to decode_step)."""
    h = _vp()
    _check(_lib.moska_profiler_create(ctypes.byref(h), max_steps), "moska_profiler_create")
    return h


def profiler_destroy(prof) -> None:
    _lib.moska_profiler_destroy(prof)


def profiler_select(prof, stages) -> None:
    """Record only the named stages (an iterable of names from STAGES)."""
    mask = 0
    for name in stages:
        mask |= 1 << STAGES.index(name)
    _check(_lib.moska_profiler_select(prof, mask), "moska_profiler_select")


def profiler_read(prof):
    """-> ({stage: summed milliseconds}, number of recorded steps); clears the profiler."""
    ms = (ctypes.c_float * len(STAGES))()
    n = ctypes.c_int32(0)
    _check(_lib.moska_profiler_read(prof, ms, ctypes.byref(n)), "moska_profiler_read")
    return {name: float(ms[i]) for i, name in enumerate(STAGES)}, int(n.value)
