"""ctypes access to the fp64 CPU oracle (moska_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the benchmark's CPU-baseline
leg, never by the product package.  This file only marshals arguments (torch/numpy -> pointers);
all arithmetic is in the C file.  bf16 tensors are handed over as their raw 16-bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moska_oracle.c")
_LIB = os.path.join(_HERE, "libmoska_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile moska_oracle.c with gcc (OpenMP) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
             "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _bits(t) -> np.ndarray:
    """Raw bf16 bit patterns of a torch bf16 tensor (or a uint16 numpy array) as uint16."""
    if isinstance(t, np.ndarray):
        assert t.dtype == np.uint16
        return np.ascontiguousarray(t)
    assert t.dtype == torch.bfloat16
    return np.ascontiguousarray(t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def _i32(t) -> np.ndarray:
    if isinstance(t, torch.Tensor):
        t = t.detach().cpu().numpy()
    return np.ascontiguousarray(t, dtype=np.int32)


def _i64(t) -> np.ndarray:
    if isinstance(t, torch.Tensor):
        t = t.detach().cpu().numpy()
    return np.ascontiguousarray(t, dtype=np.int64)


def _f64(t) -> np.ndarray:
    if isinstance(t, torch.Tensor):
        t = t.detach().cpu().numpy()
    return np.ascontiguousarray(t, dtype=np.float64)


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def chunk_summaries(k_shared) -> np.ndarray:
    Hkv, C, L, D = k_shared.shape
    kb = _bits(k_shared)
    out = np.empty((Hkv, C, D), dtype=np.float64)
    _load().oracle_chunk_summaries(_p(kb), _p(out), Hkv, C, L, D)
    return out


def chunk_summaries_attn(k_shared, scale: float) -> np.ndarray:
    """Attention-pooled chunk embedding: softmax(scale * <mean key, k_t>)-weighted mean of the keys."""
    Hkv, C, L, D = k_shared.shape
    kb = _bits(k_shared)
    out = np.empty((Hkv, C, D), dtype=np.float64)
    _load().oracle_chunk_summaries_attn(_p(kb), _p(out), ctypes.c_double(scale), Hkv, C, L, D)
    return out


def route(q, summaries, k: int, return_all: bool = False):
    """-> (topk_idx int32 [B][Hkv][k] ascending, topk_score f64 [B][Hkv][k][, scores_all])."""
    B, Hq, D = q.shape
    s = _f64(summaries)
    Hkv, C, _ = s.shape
    qb = _bits(q)
    idx = np.empty((B, Hkv, k), dtype=np.int32)
    sc = np.empty((B, Hkv, k), dtype=np.float64)
    allsc = np.empty((B, Hkv, C), dtype=np.float64)
    _load().oracle_route(_p(qb), _p(s), _p(idx), _p(sc), _p(allsc), B, Hq, Hkv, D, C, k)
    return (idx, sc, allsc) if return_all else (idx, sc)


def group_by_chunk(topk_idx, C: int, fast: bool = False):
    """-> (seg_offsets int32 [Hkv*C+1], seg_entries int32 [B*Hkv*k])."""
    idx = _i32(topk_idx)
    B, Hkv, k = idx.shape
    off = np.empty(Hkv * C + 1, dtype=np.int32)
    ent = np.empty(B * Hkv * k, dtype=np.int32)
    fn = _load().oracle_group_by_chunk_fast if fast else _load().oracle_group_by_chunk
    fn(_p(idx), _p(off), _p(ent), B, Hkv, C, k)
    return off, ent


def attend_direct(q, k_shared, v_shared, k_unique, v_unique, kv_start, kv_len, topk_idx,
                  scale: float, use_shared: bool = True, use_unique: bool = True):
    """One softmax per row over [routed shared chunks || unique tokens] -> (out, lse) in f64."""
    B, Hq, D = q.shape
    Hkv, C, L, _ = k_shared.shape
    idx = _i32(topk_idx)
    k = idx.shape[2]
    out = np.empty((B, Hq, D), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    qb, ks, vs, ku, vu = _bits(q), _bits(k_shared), _bits(v_shared), _bits(k_unique), _bits(v_unique)
    st, ln = _i64(kv_start), _i32(kv_len)
    _load().oracle_attend_direct(
        _p(qb), _p(ks), _p(vs), _p(ku), _p(vu), _p(st), _p(ln), _p(idx), _p(out), _p(lse),
        ctypes.c_double(scale), B, Hq, Hkv, D, C, L, k, int(use_shared), int(use_unique))
    return out, lse


def shared_partials(q, k_shared, v_shared, topk_idx, scale: float):
    """-> (o_part f64 [B][Hq][k][D], lse_part f64 [B][Hq][k]), slot j = j-th routed chunk."""
    B, Hq, D = q.shape
    Hkv, C, L, _ = k_shared.shape
    idx = _i32(topk_idx)
    k = idx.shape[2]
    o = np.empty((B, Hq, k, D), dtype=np.float64)
    lse = np.empty((B, Hq, k), dtype=np.float64)
    qb, ks, vs = _bits(q), _bits(k_shared), _bits(v_shared)
    _load().oracle_shared_partials(_p(qb), _p(ks), _p(vs), _p(idx), _p(o), _p(lse),
                                   ctypes.c_double(scale), B, Hq, Hkv, D, C, L, k)
    return o, lse


def merge(o_part, lse_part):
    """[..., n_slots, D], [..., n_slots] -> (out [..., D], lse [...]) in f64."""
    o = _f64(o_part)
    l = _f64(lse_part)
    n_slots, D = o.shape[-2], o.shape[-1]
    lead = o.shape[:-2]
    rows = int(np.prod(lead)) if lead else 1
    out = np.empty((rows, D), dtype=np.float64)
    lse = np.empty((rows,), dtype=np.float64)
    _load().oracle_merge(_p(o), _p(l), _p(out), _p(lse), ctypes.c_long(rows), n_slots, D)
    return out.reshape(*lead, D), lse.reshape(lead)


def e4m3_values() -> np.ndarray:
    """The 256 values of the FP8 E4M3 format as the oracle decodes them (NaN for the two NaN codes)."""
    lib = _load()
    lib.oracle_e4m3_value.restype = ctypes.c_double
    lib.oracle_e4m3_value.argtypes = [ctypes.c_uint8]
    return np.array([lib.oracle_e4m3_value(c) for c in range(256)], dtype=np.float64)


def attend_unique_fp8(q, k8, v8, k_scale, v_scale, kv_start, kv_len, scale: float):
    """Attention of every query row over its request's FP8 private KV -> (out, lse) in f64."""
    B, Hq, D = q.shape
    Hkv = k8.shape[1]

    def _u8(t):
        if isinstance(t, torch.Tensor):
            t = t.detach().cpu().numpy()
        return np.ascontiguousarray(t, dtype=np.uint8)

    def _f32(t):
        if isinstance(t, torch.Tensor):
            t = t.detach().cpu().numpy()
        return np.ascontiguousarray(t, dtype=np.float32)

    out = np.empty((B, Hq, D), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    qb, kk, vv, ks, vs = _bits(q), _u8(k8), _u8(v8), _f32(k_scale), _f32(v_scale)
    st, ln = _i64(kv_start), _i32(kv_len)
    _load().oracle_attend_unique_fp8(_p(qb), _p(kk), _p(vv), _p(ks), _p(vs), _p(st), _p(ln), _p(out),
                                     _p(lse), ctypes.c_double(scale), B, Hq, Hkv, D)
    return out, lse


def shared_partials_fp8(q, k8, v8, k_scale, v_scale, topk_idx, scale: float):
    """Per-(row, routed chunk) partials over an FP8 shared store (codes [Hkv][C][L][D], one scale
    per (KV head, chunk) for K and for V) -> (o_part f64 [B][Hq][k][D], lse_part f64 [B][Hq][k])."""
    B, Hq, D = q.shape
    Hkv, C, L, _ = k8.shape
    idx = _i32(topk_idx)
    k = idx.shape[2]

    def _u8(t):
        if isinstance(t, torch.Tensor):
            t = t.detach().cpu().numpy()
        return np.ascontiguousarray(t, dtype=np.uint8)

    def _f32(t):
        if isinstance(t, torch.Tensor):
            t = t.detach().cpu().numpy()
        return np.ascontiguousarray(t, dtype=np.float32)

    o = np.empty((B, Hq, k, D), dtype=np.float64)
    lse = np.empty((B, Hq, k), dtype=np.float64)
    qb, kk, vv, ks, vs = _bits(q), _u8(k8), _u8(v8), _f32(k_scale), _f32(v_scale)
    assert ks.shape == (Hkv, C) and vs.shape == (Hkv, C)
    _load().oracle_shared_partials_fp8(_p(qb), _p(kk), _p(vv), _p(ks), _p(vs), _p(idx), _p(o), _p(lse),
                                       ctypes.c_double(scale), B, Hq, Hkv, D, C, L, k)
    return o, lse
