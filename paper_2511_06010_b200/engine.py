"""Device-buffer bookkeeping for one MoSKA attention layer (no arithmetic: every step of the path
runs in the CUDA library; torch only owns the memory and the streams)."""
from __future__ import annotations

import math
from typing import Optional

import torch

from . import binding as M


class MoskaLayer:
    """Owns the scratch of a decode step for a fixed shape and calls the C ABI in path order."""

    def __init__(self, B, Hq, Hkv, D, C, L, k, max_unique_len, dense=False, dense_slots=None,
                 n_unique_splits=None, device="cuda", fp8_unique=False, q_len=1):
        """B counts batch rows; with q_len > 1 they are B / q_len requests of q_len query tokens."""
        self.device = torch.device(device)
        self.dense = dense
        if n_unique_splits is None:
            default = M.default_unique_splits_fp8 if fp8_unique else M.default_unique_splits
            n_unique_splits = default(B // max(1, q_len), Hkv, max(1, max_unique_len))
        if dense:
            shared_slots = dense_slots if dense_slots is not None else min(C, 16)
            k = C
        else:
            shared_slots = k
        self.shape = M.shape(B, Hq, Hkv, D, C, L, k, shared_slots, n_unique_splits, q_len)
        self.n_slots = M.partial_slots(self.shape)
        self.scale = 1.0 / math.sqrt(D)
        dev = self.device
        P = B * Hkv * k
        self.summaries = torch.empty(Hkv, C, D, dtype=torch.float32, device=dev)
        self.topk_idx = None if dense else torch.empty(B, Hkv, k, dtype=torch.int32, device=dev)
        self.topk_score = None if dense else torch.empty(B, Hkv, k, dtype=torch.float32, device=dev)
        self.seg_offsets = None if dense else torch.empty(Hkv * C + 1, dtype=torch.int32, device=dev)
        self.seg_entries = None if dense else torch.empty(max(P, 1), dtype=torch.int32, device=dev)
        self.o_part = torch.empty(B, Hq, self.n_slots, D, dtype=torch.float32, device=dev)
        self.lse_part = torch.empty(B, Hq, self.n_slots, dtype=torch.float32, device=dev)
        self.out = torch.empty(B, Hq, D, dtype=torch.bfloat16, device=dev)
        self.out_f32 = torch.empty(B, Hq, D, dtype=torch.float32, device=dev)
        self.lse_out = torch.empty(B, Hq, dtype=torch.float32, device=dev)
        ws_bytes = M.workspace_bytes(self.shape)
        self.ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=dev)
        self.side_stream: Optional[torch.cuda.Stream] = None
        # Routing, grouping and the streaming shared-attention tiles run on a second, high-priority
        # stream beside unique attention (which stages K/V through shared memory and therefore
        # keeps its bandwidth whatever shares the SM with it).
        self.overlap_routing = True

    # -- offline ---------------------------------------------------------------------------------
    def build_summaries(self, k_shared, attention_pooled=False, probe_scale=None):
        """Chunk embeddings for the router: the mean key, or (attention_pooled) the mean key's
        softmax-weighted pooling of the chunk's keys."""
        if attention_pooled:
            M.build_chunk_summaries_attn(k_shared, self.summaries,
                                         self.scale if probe_scale is None else probe_scale, self.shape)
        else:
            M.build_chunk_summaries(k_shared, self.summaries, self.shape)
        return self.summaries

    # -- the individual stages (used by the per-stage parity tests and per-kernel timing) --------
    def route(self, q):
        M.route(q, self.summaries, self.topk_idx, self.topk_score, self.shape, self.ws)

    def group(self):
        M.group_by_chunk(self.topk_idx, self.seg_offsets, self.seg_entries, self.shape, self.ws)

    def shared(self, q, k_shared, v_shared):
        M.shared_attn(q, k_shared, v_shared, self.topk_idx, self.seg_offsets, self.seg_entries,
                      self.o_part, self.lse_part, self.scale, self.shape, self.ws)

    def shared_fp8(self, q, sf8):
        """Shared KV Attention over an FP8 shared store (`sf8`: codes and per-chunk scales)."""
        M.shared_attn_fp8(q, sf8.k8, sf8.v8, sf8.k_scale, sf8.v_scale, self.topk_idx, self.seg_offsets,
                          self.seg_entries, self.o_part, self.lse_part, self.scale, self.shape, self.ws)

    def gemv_baseline(self, q, k_shared, v_shared):
        M.gemv_baseline(q, k_shared, v_shared, self.topk_idx, self.o_part, self.lse_part,
                        self.scale, self.shape)

    def unique(self, q, k_unique, v_unique, kv_start, kv_len, stream=None):
        M.unique_attn(q, k_unique, v_unique, kv_start, kv_len, self.o_part, self.lse_part,
                      self.scale, self.shape, stream)

    def unique_fp8(self, q, f8, kv_start, kv_len, stream=None):
        M.unique_attn_fp8(q, f8.k8, f8.v8, f8.k_scale, f8.v_scale, kv_start, kv_len, self.o_part,
                          self.lse_part, self.scale, self.shape, stream)

    def merge(self):
        M.merge(self.o_part, self.lse_part, self.out, self.out_f32, self.lse_out, self.shape)

    # -- the whole step --------------------------------------------------------------------------
    def step(self, q, k_shared, v_shared, k_unique, v_unique, kv_start, kv_len, two_streams=False,
             prof=None, unique_tokens=0):
        self.shape.unique_tokens = int(unique_tokens)
        two_streams = two_streams and self.overlap_routing
        if two_streams and self.side_stream is None:
            self.side_stream = torch.cuda.Stream(device=self.device, priority=-1)
        M.decode_step(q, None if self.dense else self.summaries, k_shared, v_shared, k_unique,
                      v_unique, kv_start, kv_len, self.topk_idx, self.seg_offsets,
                      self.seg_entries, self.o_part, self.lse_part, self.out, self.lse_out,
                      self.scale, self.shape, self.ws, None,
                      self.side_stream if two_streams else None, prof)
        return self.out

    def step_fp8kv(self, q, k_shared, v_shared, f8, kv_start, kv_len, two_streams=False, prof=None,
                   unique_tokens=0):
        """One decode step with the private KV store in FP8 (`f8`: codes and per-token scales)."""
        self.shape.unique_tokens = int(unique_tokens)
        two_streams = two_streams and self.overlap_routing
        if two_streams and self.side_stream is None:
            self.side_stream = torch.cuda.Stream(device=self.device, priority=-1)
        M.decode_step_fp8kv(q, None if self.dense else self.summaries, k_shared, v_shared, f8.k8,
                            f8.v8, f8.k_scale, f8.v_scale, kv_start, kv_len, self.topk_idx,
                            self.seg_offsets, self.seg_entries, self.o_part, self.lse_part,
                            self.out, self.lse_out, self.scale, self.shape, self.ws, None,
                            self.side_stream if two_streams else None, prof)
        return self.out

    def step_fp8shared(self, q, sf8, k_unique, v_unique, kv_start, kv_len, two_streams=False, prof=None,
                       unique_tokens=0):
        """One decode step with the SHARED store in FP8 (`sf8`: codes and per-chunk scales)."""
        self.shape.unique_tokens = int(unique_tokens)
        two_streams = two_streams and self.overlap_routing
        if two_streams and self.side_stream is None:
            self.side_stream = torch.cuda.Stream(device=self.device, priority=-1)
        M.decode_step_fp8shared(q, None if self.dense else self.summaries, sf8.k8, sf8.v8, sf8.k_scale, sf8.v_scale, k_unique,
                                v_unique, kv_start, kv_len, self.topk_idx, self.seg_offsets, self.seg_entries,
                                self.o_part, self.lse_part, self.out, self.lse_out, self.scale, self.shape,
                                self.ws, None, self.side_stream if two_streams else None, prof)
        return self.out

    def step_fp8(self, q, sf8, f8, kv_start, kv_len, two_streams=False, prof=None, unique_tokens=0):
        """One decode step with both stores in FP8 (`sf8`: shared codes and per-chunk scales, `f8`:
        private codes and per-token scales)."""
        self.shape.unique_tokens = int(unique_tokens)
        two_streams = two_streams and self.overlap_routing
        if two_streams and self.side_stream is None:
            self.side_stream = torch.cuda.Stream(device=self.device, priority=-1)
        M.decode_step_fp8(q, None if self.dense else self.summaries, sf8.k8, sf8.v8, sf8.k_scale, sf8.v_scale, f8.k8, f8.v8,
                          f8.k_scale, f8.v_scale, kv_start, kv_len, self.topk_idx, self.seg_offsets,
                          self.seg_entries, self.o_part, self.lse_part, self.out, self.lse_out, self.scale,
                          self.shape, self.ws, None, self.side_stream if two_streams else None, prof)
        return self.out

    def step_fp8_host(self, q_host, q_dev, out_host, sf8, f8, kv_start, kv_len, two_streams=False,
                      prof=None, unique_tokens=0):
        """step_fp8 with the queries taken from and the result delivered to host memory."""
        self.shape.unique_tokens = int(unique_tokens)
        two_streams = two_streams and self.overlap_routing
        if two_streams and self.side_stream is None:
            self.side_stream = torch.cuda.Stream(device=self.device, priority=-1)
        M.decode_step_fp8_host(q_host, q_dev, None if self.dense else self.summaries, sf8.k8, sf8.v8, sf8.k_scale, sf8.v_scale,
                               f8.k8, f8.v8, f8.k_scale, f8.v_scale, kv_start, kv_len, self.topk_idx,
                               self.seg_offsets, self.seg_entries, self.o_part, self.lse_part, self.out,
                               out_host, self.scale, self.shape, self.ws, None,
                               self.side_stream if two_streams else None, prof)
        return out_host

    def bind_step_fp8_host(self, q_host, q_dev, out_host, sf8, f8, kv_start, kv_len, two_streams=False,
                           unique_tokens=0):
        """step_fp8_host for a loop over fixed buffers: arguments marshalled once (see bind_step_host)."""
        self.shape.unique_tokens = int(unique_tokens)
        two_streams = two_streams and self.overlap_routing
        if two_streams and self.side_stream is None:
            self.side_stream = torch.cuda.Stream(device=self.device, priority=-1)
        return M.bind_decode_step_fp8_host(q_host, q_dev, None if self.dense else self.summaries, sf8.k8, sf8.v8, sf8.k_scale,
                                           sf8.v_scale, f8.k8, f8.v8, f8.k_scale, f8.v_scale, kv_start,
                                           kv_len, self.topk_idx, self.seg_offsets, self.seg_entries,
                                           self.o_part, self.lse_part, self.out, out_host, self.scale,
                                           self.shape, self.ws, None,
                                           self.side_stream if two_streams else None)

    def bind_step_host(self, q_host, q_dev, out_host, k_shared, v_shared, k_unique, v_unique,
                       kv_start, kv_len, two_streams=False, unique_tokens=0):
        """step_host for a loop over fixed buffers: marshals the arguments once and returns a
        callable that only makes the C call (no per-call Python work between two steps)."""
        self.shape.unique_tokens = int(unique_tokens)
        two_streams = two_streams and self.overlap_routing
        if two_streams and self.side_stream is None:
            self.side_stream = torch.cuda.Stream(device=self.device, priority=-1)
        return M.bind_decode_step_host(q_host, q_dev, None if self.dense else self.summaries, k_shared,
                                       v_shared, k_unique, v_unique, kv_start, kv_len, self.topk_idx,
                                       self.seg_offsets, self.seg_entries, self.o_part, self.lse_part,
                                       self.out, out_host, self.scale, self.shape, self.ws, None,
                                       self.side_stream if two_streams else None)

    def step_host(self, q_host, q_dev, out_host, k_shared, v_shared, k_unique, v_unique,
                  kv_start, kv_len, two_streams=False, prof=None, unique_tokens=0):
        self.shape.unique_tokens = int(unique_tokens)
        two_streams = two_streams and self.overlap_routing
        if two_streams and self.side_stream is None:
            self.side_stream = torch.cuda.Stream(device=self.device, priority=-1)
        M.decode_step_host(q_host, q_dev, None if self.dense else self.summaries, k_shared,
                           v_shared, k_unique, v_unique, kv_start, kv_len, self.topk_idx,
                           self.seg_offsets, self.seg_entries, self.o_part, self.lse_part,
                           self.out, out_host, self.scale, self.shape, self.ws, None,
                           self.side_stream if two_streams else None, prof)
        return out_host
