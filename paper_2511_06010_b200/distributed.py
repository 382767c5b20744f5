"""Host-side multi-process plumbing of the benchmark (torch.distributed; NCCL on GPUs, gloo on CPU).

The decode-attention path needs no data-path collective: routing, shared attention, unique
attention and the merge are independent per (request, KV head).  One batch is therefore split by
KV HEAD: rank r holds heads [h0, h1) of the shared store and of every request's private store,
receives those heads' queries and produces those heads' outputs, with no exchange on the path
(`kv_head_shard`, `slice_kv_heads`; the paper's point is that the shared store is NOT replicated,
Section I).  Replicas (every rank its own batch and its own copy of the shared store) remain
available to the benchmark behind a flag.  Only the timing is reduced over ranks.
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment (1 process if absent)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: every multi-GPU number is the max over ranks."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(units_this_rank: float, ms_this_rank: float, device="cpu") -> Tuple[float, float]:
    """(units of all ranks / slowest rank's time in seconds, that time in ms)."""
    ms = max_over_ranks(ms_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / (ms * 1e-3), ms


def kv_head_shard(Hkv: int, rank: int, world: int) -> Tuple[int, int]:
    """[h0, h1) KV heads of `rank` when a batch is split by KV head (exchange-free partition)."""
    per = (Hkv + world - 1) // world
    h0 = min(Hkv, rank * per)
    return h0, min(Hkv, h0 + per)


def slice_kv_heads(h0: int, h1: int, G: int, q, k_shared, v_shared, k_unique, v_unique):
    """The tensors of KV heads [h0, h1) of one batch, as dense buffers of their own (what the rank
    that owns those heads holds): q [B][(h1-h0)*G][D], shared K/V [h1-h0][C][L][D], private K/V
    [T][h1-h0][D].  Indexing only; request structure (kv_start, kv_len) is the same on every rank."""
    return (q[:, h0 * G:h1 * G].contiguous(), k_shared[h0:h1].contiguous(),
            v_shared[h0:h1].contiguous(), k_unique[:, h0:h1].contiguous(),
            v_unique[:, h0:h1].contiguous())


def finalize() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
