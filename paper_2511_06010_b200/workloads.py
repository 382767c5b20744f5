"""Seeded synthetic inputs for the MoSKA decode-attention hot path.

This module only draws random tensors with the shapes, value distributions and structure of the
five benchmark workloads (clustered shared keys, uniform or Zipf-skewed query targets, ragged
unique contexts).  It holds none of the method's arithmetic: no summaries, scores, softmax or
merge are computed here.  Both the CUDA path and the CPU oracle are fed from it.

The paper evaluates on no dataset (Section IV describes a workload of a 1M-16M token shared
context plus a private context per request); these generators stand in for that workload.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and distribution parameters of one synthetic decode workload."""

    name: str
    B: int                  # concurrent requests
    Hq: int                 # query heads
    Hkv: int                # KV heads
    D: int                  # head dimension
    C: int                  # shared chunks
    L: int                  # tokens per chunk
    k: int                  # routed chunks per (request, KV head); k == C means dense (no routing)
    unique_len: int         # unique tokens per request (lower bound if ragged)
    unique_len_max: int = 0  # > 0: ragged, length uniform in [unique_len, unique_len_max]
    zipf_s: float = 0.0     # > 0: query target chunk ~ Zipf(s) over chunk rank c+1; else uniform
    steps: int = 1          # consecutive decode steps (re-routing every step)
    seed: int = 0
    shard: int = 0          # index of a KV-head shard of the workload: changes the drawn K/V values
                            # only, never the request structure (lengths, query targets)

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def dense(self) -> bool:
        return self.k == self.C

    @property
    def ragged(self) -> bool:
        return self.unique_len_max > 0


# The five workloads of the benchmark definition (index = config number).
CONFIGS = [
    Workload("cfg0_small", B=16, Hq=4, Hkv=1, D=64, C=8, L=512, k=2, unique_len=256),
    Workload("cfg1_llama8b_b64", B=64, Hq=32, Hkv=8, D=128, C=128, L=512, k=8, unique_len=4096),
    Workload("cfg2_corpus1m_b256", B=256, Hq=32, Hkv=8, D=128, C=2048, L=512, k=16,
             unique_len=8192, zipf_s=1.1),
    Workload("cfg3_dense_b512", B=512, Hq=32, Hkv=8, D=128, C=256, L=512, k=256, unique_len=2048),
    Workload("cfg4_serving70b_b1024", B=1024, Hq=64, Hkv=8, D=128, C=1024, L=512, k=32,
             unique_len=1024, unique_len_max=32768, zipf_s=1.3, steps=8),
]


def scaled(w: Workload, **overrides) -> Workload:
    """A copy of `w` with some fields replaced (used for reduced-size parity cases)."""
    return dataclasses.replace(w, **overrides)


@dataclasses.dataclass
class SharedStore:
    k_shared: torch.Tensor   # bf16 [Hkv][C][L][D]
    v_shared: torch.Tensor   # bf16 [Hkv][C][L][D]
    mu: torch.Tensor         # fp32 [Hkv][C][D]  cluster centres the keys and queries are drawn around


@dataclasses.dataclass
class UniqueStore:
    k_unique: torch.Tensor   # bf16 [T_total][Hkv][D]
    v_unique: torch.Tensor   # bf16 [T_total][Hkv][D]
    kv_start: torch.Tensor   # int64 [B]  first token of request b
    kv_len: torch.Tensor     # int32 [B]  tokens of request b at step 0
    capacity: torch.Tensor   # int64 [B]  tokens reserved for request b (kv_len + steps)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def kv_head_shard(w: Workload, rank: int, world: int) -> Workload:
    """The part of workload `w` that rank `rank` of `world` holds when ONE batch is split by KV
    head: the same requests (lengths, query targets), Hkv / world KV heads with their G query heads
    each, and that many heads' share of the shared and private stores."""
    if w.Hkv % world != 0:
        raise ValueError(f"{w.Hkv} KV heads do not split evenly over {world} ranks")
    return scaled(w, Hq=w.Hq // world, Hkv=w.Hkv // world, shard=rank)


def make_shared_store(w: Workload, device="cpu") -> SharedStore:
    """Keys of chunk c (per KV head) are mu[h][c] + 0.5 N(0, I); values are N(0, I); bf16."""
    g = _gen(w.seed * 1000 + 1 + 7919 * w.shard, device)
    mu = torch.randn(w.Hkv, w.C, w.D, generator=g, device=device, dtype=torch.float32)
    k_shared = torch.empty(w.Hkv, w.C, w.L, w.D, device=device, dtype=torch.bfloat16)
    v_shared = torch.empty(w.Hkv, w.C, w.L, w.D, device=device, dtype=torch.bfloat16)
    # Chunk by chunk groups so that the fp32 temporaries stay small for the multi-GB stores.
    step = max(1, (1 << 24) // (w.L * w.D))
    for h in range(w.Hkv):
        for c0 in range(0, w.C, step):
            c1 = min(w.C, c0 + step)
            noise = torch.randn(c1 - c0, w.L, w.D, generator=g, device=device, dtype=torch.float32)
            k_shared[h, c0:c1] = (mu[h, c0:c1, None, :] + 0.5 * noise).to(torch.bfloat16)
            v_shared[h, c0:c1] = torch.randn(
                c1 - c0, w.L, w.D, generator=g, device=device, dtype=torch.float32
            ).to(torch.bfloat16)
    return SharedStore(k_shared, v_shared, mu)


def shared_centres(w: Workload, device="cpu") -> torch.Tensor:
    """The cluster centres mu [Hkv][C][D] of make_shared_store(w) without the store itself (the
    first draw of the same generator): what a rank that holds no shared KV needs to draw queries."""
    g = _gen(w.seed * 1000 + 1 + 7919 * w.shard, device)
    return torch.randn(w.Hkv, w.C, w.D, generator=g, device=device, dtype=torch.float32)


def unique_lengths(w: Workload) -> np.ndarray:
    """Per-request unique context length at step 0 (host-side seeded draw)."""
    rng = np.random.default_rng(w.seed * 1000 + 2)
    if w.ragged:
        return rng.integers(w.unique_len, w.unique_len_max + 1, size=w.B).astype(np.int64)
    return np.full(w.B, w.unique_len, dtype=np.int64)


def make_unique_store(w: Workload, device="cpu", lengths: Optional[np.ndarray] = None) -> UniqueStore:
    """Ragged token-major private KV: K, V ~ N(0, I) in bf16, `steps` spare tokens per request."""
    lens = unique_lengths(w) if lengths is None else np.asarray(lengths, dtype=np.int64)
    cap = lens + w.steps
    start = np.concatenate([[0], np.cumsum(cap)[:-1]]).astype(np.int64)
    total = int(cap.sum())
    g = _gen(w.seed * 1000 + 3 + 7919 * w.shard, device)
    k_unique = torch.empty(max(total, 1), w.Hkv, w.D, device=device, dtype=torch.bfloat16)
    v_unique = torch.empty(max(total, 1), w.Hkv, w.D, device=device, dtype=torch.bfloat16)
    step = max(1, (1 << 25) // (w.Hkv * w.D))
    for t0 in range(0, total, step):
        t1 = min(total, t0 + step)
        k_unique[t0:t1].normal_(generator=g)
        v_unique[t0:t1].normal_(generator=g)
    if total == 0:
        k_unique.zero_()
        v_unique.zero_()
    return UniqueStore(
        k_unique,
        v_unique,
        torch.from_numpy(start).to(device),
        torch.from_numpy(lens.astype(np.int32)).to(device),
        torch.from_numpy(cap).to(device),
    )


def query_targets(w: Workload, step: int = 0) -> np.ndarray:
    """Target chunk of every request: uniform, or Zipf(s) over rank c+1 (identity rank->chunk)."""
    rng = np.random.default_rng(w.seed * 1000 + 10 + step)
    if w.zipf_s > 0:
        p = (np.arange(1, w.C + 1, dtype=np.float64)) ** (-w.zipf_s)
        p /= p.sum()
        return rng.choice(w.C, size=w.B, p=p).astype(np.int64)
    return rng.integers(0, w.C, size=w.B).astype(np.int64)


def make_queries(w: Workload, shared: SharedStore, step: int = 0, device="cpu") -> torch.Tensor:
    """q[b][hq] = mu[hq // G][target_b] + 0.5 N(0, I), independent noise per query head; bf16."""
    tgt = torch.from_numpy(query_targets(w, step)).to(device)
    g = _gen(w.seed * 1000 + 100 + step + 7919 * w.shard, device)
    noise = torch.randn(w.B, w.Hq, w.D, generator=g, device=device, dtype=torch.float32)
    head_of = torch.arange(w.Hq, device=device) // w.G
    centre = shared.mu[head_of[None, :], tgt[:, None], :]          # [B][Hq][D]
    return (centre + 0.5 * noise).to(torch.bfloat16).contiguous()


@dataclasses.dataclass
class UniqueStoreFp8:
    k8: torch.Tensor        # uint8 [T_total][Hkv][D]  FP8 E4M3 codes of the keys
    v8: torch.Tensor        # uint8 [T_total][Hkv][D]  FP8 E4M3 codes of the values
    k_scale: torch.Tensor   # fp32  [T_total][Hkv]     key = k_scale * e4m3(k8)
    v_scale: torch.Tensor   # fp32  [T_total][Hkv]


def quantize_unique_store_fp8(un: UniqueStore, release: bool = False) -> UniqueStoreFp8:
    """Storage-format conversion of a private KV store to FP8 E4M3 with one scale per (token, KV
    head): scale = max|x| / 448 (the largest E4M3 value), codes by torch's round-to-nearest cast.
    Input preparation only: the FP8 store is what both the CUDA path and the oracle are given.
    `release` drops each bf16 tensor of `un` as soon as it is converted (for stores that fill most
    of the device memory)."""
    def q8(x):
        codes = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
        scales = torch.empty(x.shape[:-1], dtype=torch.float32, device=x.device)
        step = max(1, (1 << 26) // (x.shape[1] * x.shape[2]))  # bounded temporaries
        for t0 in range(0, x.shape[0], step):
            xs = x[t0:t0 + step].float()
            amax = xs.abs().amax(dim=-1)
            scale = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax))
            codes[t0:t0 + step] = (xs / scale[..., None]).to(torch.float8_e4m3fn).view(torch.uint8)
            scales[t0:t0 + step] = scale
        return codes, scales

    k8, ks = q8(un.k_unique)
    if release:
        un.k_unique = None
    v8, vs = q8(un.v_unique)
    if release:
        un.v_unique = None
    return UniqueStoreFp8(k8, v8, ks, vs)


@dataclasses.dataclass
class SharedStoreFp8:
    k8: torch.Tensor        # uint8 [Hkv][C][L][D]  FP8 E4M3 codes of the shared keys
    v8: torch.Tensor        # uint8 [Hkv][C][L][D]  FP8 E4M3 codes of the shared values
    k_scale: torch.Tensor   # fp32  [Hkv][C]        key = k_scale[h][c] * e4m3(k8)
    v_scale: torch.Tensor   # fp32  [Hkv][C]


def quantize_shared_store_fp8(sh: SharedStore) -> SharedStoreFp8:
    """Storage-format conversion of a shared KV store to FP8 E4M3 with ONE scale per (KV head,
    chunk) for the keys and one for the values: scale = max|x| over the chunk / 448, codes by
    torch's round-to-nearest cast.  Input preparation only: the FP8 store is what both the CUDA
    path and the oracle are given (chunk embeddings for the router are built from whichever store
    the caller keeps in bf16; the benchmark builds them before it drops the bf16 copy)."""
    def q8(x):
        Hkv, C = x.shape[:2]
        codes = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
        scales = torch.empty(Hkv, C, dtype=torch.float32, device=x.device)
        step = max(1, (1 << 24) // (x.shape[2] * x.shape[3]))
        for h in range(Hkv):
            for c0 in range(0, C, step):
                xs = x[h, c0:c0 + step].float()
                amax = xs.abs().amax(dim=(-1, -2))
                scale = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax))
                codes[h, c0:c0 + step] = (xs / scale[:, None, None]).to(torch.float8_e4m3fn).view(torch.uint8)
                scales[h, c0:c0 + step] = scale
        return codes, scales

    k8, ks = q8(sh.k_shared)
    v8, vs = q8(sh.v_shared)
    return SharedStoreFp8(k8, v8, ks, vs)
