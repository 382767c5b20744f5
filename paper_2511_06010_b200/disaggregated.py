"""The decode step split over a Shared-KV rank and Unique-KV ranks (Section III-C in miniature).

The paper serves the two kinds of attention from different nodes because their resource profiles
differ: Shared KV Attention is compute-bound and batches across ALL requests, Unique KV Attention
is memory-bound and private to a request.  Here rank `shared_rank` holds the shared store and runs
routing, grouping and Shared KV Attention for every request of the step; each other rank holds the
private KV of a contiguous block of requests, owns their queries and produces their outputs.

Per step (one exchange each way, point to point, sizes independent of the context lengths):
  unique rank -> shared rank   q of its requests                      B_u * Hq * D * 2 bytes
  shared rank -> unique rank   the shared result of its requests,     B_u * Hq * (D + 1) * 4 bytes
                               already merged over the k routed chunks (o fp32 and lse)
The unique rank runs Unique KV Attention while the queries travel and the shared rank works, then
merges the returned partial with its own split-K partials.  The log-sum-exp merge is associative, so
the result equals the single-GPU step.

Only tensors cross this module's communication helpers, so they run on CPU tensors over gloo as
well as on CUDA tensors over NCCL; all arithmetic stays in the library's kernels.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist


def request_blocks(n_requests: int, unique_ranks: Sequence[int]) -> List[Tuple[int, int, int]]:
    """[(rank, b0, b1)]: the contiguous block of requests each unique rank owns."""
    n = len(unique_ranks)
    per = (n_requests + n - 1) // n
    out = []
    for i, r in enumerate(unique_ranks):
        b0 = min(n_requests, i * per)
        out.append((r, b0, min(n_requests, b0 + per)))
    return out


def send_queries(q_local: torch.Tensor, shared_rank: int, group=None):
    """Unique rank: start sending this rank's queries [B_u][Hq][D]; returns the work handle."""
    return dist.isend(q_local, dst=shared_rank, group=group)


def gather_queries(q_all: torch.Tensor, blocks: Sequence[Tuple[int, int, int]], group=None) -> None:
    """Shared rank: receive every unique rank's queries into its rows of q_all [B][Hq][D]."""
    works = [dist.irecv(q_all[b0:b1], src=r, group=group) for r, b0, b1 in blocks if b1 > b0]
    for w in works:
        w.wait()


def return_shared_partials(o_shared: torch.Tensor, lse_shared: torch.Tensor,
                           blocks: Sequence[Tuple[int, int, int]], group=None) -> None:
    """Shared rank: send rows [b0, b1) of the merged shared result (o fp32 [B][Hq][D], lse fp32
    [B][Hq]) to their owners."""
    works = []
    for r, b0, b1 in blocks:
        if b1 > b0:
            works.append(dist.isend(o_shared[b0:b1], dst=r, group=group))
            works.append(dist.isend(lse_shared[b0:b1], dst=r, group=group))
    for w in works:
        w.wait()


def receive_shared_partial(o_buf: torch.Tensor, lse_buf: torch.Tensor, shared_rank: int, group=None) -> None:
    """Unique rank: receive the shared result of this rank's requests (contiguous buffers)."""
    w0 = dist.irecv(o_buf, src=shared_rank, group=group)
    w1 = dist.irecv(lse_buf, src=shared_rank, group=group)
    w0.wait()
    w1.wait()


class SharedRank:
    """Routing, grouping and Shared KV Attention for all requests, merged over the routed chunks."""

    is_shared_rank = True

    def __init__(self, layer, k_shared, v_shared):
        # `layer`: a MoskaLayer for ALL requests with n_unique_splits = 1; its one unique slot stays
        # empty (lse = -inf), so the merge combines the shared slots only.
        assert layer.shape.n_unique_splits == 1
        self.layer, self.k_shared, self.v_shared = layer, k_shared, v_shared
        n_sh = layer.shape.shared_slots
        layer.lse_part[:, :, n_sh:].fill_(float("-inf"))
        layer.o_part[:, :, n_sh:].zero_()
        if not layer.dense:
            layer.build_summaries(k_shared)

    def compute(self, q_all: torch.Tensor):
        """-> (o fp32 [B][Hq][D], lse fp32 [B][Hq]) of the shared part of every request."""
        L = self.layer
        if not L.dense:
            L.route(q_all)
            L.group()
        L.shared(q_all, self.k_shared, self.v_shared)
        L.merge()
        return L.out_f32, L.lse_out


class UniqueRank:
    """Unique KV Attention of this rank's requests and the final merge with the shared result."""

    is_shared_rank = False

    def __init__(self, layer, k_unique, v_unique, kv_start):
        # `layer`: a MoskaLayer for this rank's requests with shared_slots = 1: slot 0 takes the
        # shared result that comes back from the shared rank.
        assert layer.shape.shared_slots == 1
        self.layer, self.k_unique, self.v_unique, self.kv_start = layer, k_unique, v_unique, kv_start
        B, Hq, D = layer.out.shape
        self.o_in = torch.empty(B, Hq, D, dtype=torch.float32, device=layer.device)
        self.lse_in = torch.empty(B, Hq, dtype=torch.float32, device=layer.device)

    def start(self, q_local: torch.Tensor, kv_len: torch.Tensor) -> None:
        self.layer.unique(q_local, self.k_unique, self.v_unique, self.kv_start, kv_len)

    def finish(self, o_shared: Optional[torch.Tensor] = None, lse_shared: Optional[torch.Tensor] = None):
        """Places the shared result (default: what receive_shared_partial left in o_in / lse_in)
        in slot 0 and merges -> out bf16 [B_u][Hq][D]."""
        L = self.layer
        L.o_part[:, :, 0, :].copy_(self.o_in if o_shared is None else o_shared)
        L.lse_part[:, :, 0].copy_(self.lse_in if lse_shared is None else lse_shared)
        L.merge()
        return L.out


def step(role, q_local, kv_len, shared_rank: int, blocks, q_all=None, group=None):
    """One decode step on this rank.  `role` is a SharedRank (pass q_all, its [B][Hq][D] buffer)
    or a UniqueRank (pass q_local and kv_len); returns the outputs of the rank's own requests
    (None on the shared rank)."""
    if getattr(role, "is_shared_rank", False):
        gather_queries(q_all, blocks, group)
        o, lse = role.compute(q_all)
        return_shared_partials(o, lse, blocks, group)
        return None
    send = send_queries(q_local, shared_rank, group)
    role.start(q_local, kv_len)
    receive_shared_partial(role.o_in, role.lse_in, shared_rank, group)
    send.wait()
    return role.finish()
