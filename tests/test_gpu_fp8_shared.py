"""GPU parity of Shared KV Attention over an FP8 (E4M3, one scale per (KV head, chunk)) shared store:
the tensor-core kernel fed with code tiles, against the fp64 oracle that decodes the same codes from
the format's definition.  Tolerances are those of the bf16 path (tests/parity_utils.py)."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2511_06010_b200 import workloads as W
from tests import parity_utils as PU

pytestmark = pytest.mark.gpu


def _mods():
    from paper_2511_06010_b200 import binding as M
    from paper_2511_06010_b200.engine import MoskaLayer

    return M, MoskaLayer


def _case(w, lengths=None, n_unique_splits=2, sample=None, two_streams=False, unique_tokens=0):
    M, MoskaLayer = _mods()
    sh = W.make_shared_store(w, "cuda")
    un = W.make_unique_store(w, "cuda", lengths)
    q = W.make_queries(w, sh, 0, "cuda")
    f8 = W.quantize_shared_store_fp8(sh)
    max_len = int(un.kv_len.max().item()) if w.B else 1
    layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, max_len, n_unique_splits=n_unique_splits)
    layer.build_summaries(sh.k_shared)        # offline, from the bf16 copy of the keys
    layer.route(q)
    layer.group()
    sample = np.arange(w.B) if sample is None else np.asarray(sample)
    topk = layer.topk_idx.cpu().numpy()
    # staged oracle on the same codes: one partial per (row, routed chunk)
    o_ref, l_ref = O.shared_partials_fp8(q[sample].cpu(), f8.k8.cpu(), f8.v8.cpu(), f8.k_scale.cpu(),
                                         f8.v_scale.cpu(), topk[sample], layer.scale)
    layer.o_part.fill_(float("nan"))
    layer.lse_part.fill_(float("nan"))
    layer.shared_fp8(q, f8)
    torch.cuda.synchronize()
    n_sh = layer.shape.shared_slots
    PU.check_lse(layer.lse_part[sample][:, :, :n_sh].cpu().numpy(), l_ref, "fp8 shared lse")
    PU.check_attention(layer.o_part[sample][:, :, :n_sh].cpu().numpy(), o_ref, "fp8 shared partial o")
    assert torch.isfinite(layer.o_part[:, :, :n_sh]).all(), "a shared slot was left unwritten"
    # the whole step: shared partials of the oracle merged with its unique partial
    out = layer.step_fp8shared(q, f8, un.k_unique, un.v_unique, un.kv_start, un.kv_len,
                               two_streams=two_streams, unique_tokens=unique_tokens)
    torch.cuda.synchronize()
    dummy = torch.zeros(w.Hkv, 1, 128, w.D, dtype=torch.bfloat16)
    lens = un.kv_len.cpu().numpy()[sample]
    starts = un.kv_start.cpu().numpy()[sample]
    o_un, l_un = O.attend_direct(q[sample].cpu(), dummy, dummy, un.k_unique.cpu(), un.v_unique.cpu(), starts, lens,
                                 np.zeros((len(sample), w.Hkv, 1), dtype=np.int32), layer.scale, use_shared=False)
    o_all = np.concatenate([o_ref, o_un[:, :, None, :]], axis=2)
    l_all = np.concatenate([l_ref, l_un[:, :, None]], axis=2)
    want, want_lse = O.merge(o_all, l_all)
    PU.check_attention(out[sample].float().cpu().numpy(), want, "fp8-shared decode step out")
    PU.check_lse(layer.lse_out[sample].cpu().numpy(), want_lse, "fp8-shared decode step lse")
    assert M.device_status() == 0


def test_fp8_shared_small_and_large_segments_every_element():
    """Segments of one request up to hundreds of rows (8-row items, single-tile items as pairs and
    split, two-tile items), chunks of one to five K/V tiles, G = 4 and 8, ragged private contexts."""
    lens = np.array([0, 1, 100, 257, 64, 33, 700, 15], dtype=np.int64)
    for Hq, Hkv, B, C, L, k in ((8, 2, 12, 32, 512, 4), (8, 2, 96, 4, 256, 2), (16, 2, 70, 3, 128, 2),
                                (8, 2, 200, 4, 640, 2), (8, 2, 64, 256, 256, 8)):
        w = W.Workload("f8sh", B=B, Hq=Hq, Hkv=Hkv, D=128, C=C, L=L, k=k, unique_len=0, seed=91 + B)
        _case(w, lengths=np.resize(lens, B))


def test_fp8_shared_full_cfg1_sampled_two_streams():
    w = W.CONFIGS[1]
    _case(w, sample=[0, 7, 21, 40, 63], n_unique_splits=None, two_streams=True,
          unique_tokens=w.B * w.unique_len)


def test_decode_step_with_both_stores_in_fp8():
    """moska_decode_step_fp8: shared codes with per-chunk scales, private codes with per-token scales;
    the oracle merges its FP8 shared partials with its FP8 private-store attention.  One and two
    streams; segments on every work list; empty and ragged private contexts."""
    M, MoskaLayer = _mods()
    lens = np.array([300, 1, 0, 1000, 64, 17, 129, 511, 2048, 77, 5, 900, 33, 640, 256, 4], dtype=np.int64)
    for B, C, k in ((16, 16, 4), (80, 4, 2)):
        w = W.scaled(W.CONFIGS[1], B=B, C=C, k=k, unique_len=0)
        sh = W.make_shared_store(w, "cuda")
        un = W.make_unique_store(w, "cuda", np.resize(lens, B))
        q = W.make_queries(w, sh, 0, "cuda")
        sf8 = W.quantize_shared_store_fp8(sh)
        kv_start, kv_len = un.kv_start, un.kv_len
        f8 = W.quantize_unique_store_fp8(un)
        layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, int(lens.max()), n_unique_splits=3,
                           fp8_unique=True)
        layer.build_summaries(sh.k_shared)
        for two in (False, True):
            layer.out.zero_()
            out = layer.step_fp8(q, sf8, f8, kv_start, kv_len, two_streams=two,
                                 unique_tokens=int(kv_len.sum().item())).clone()
            torch.cuda.synchronize()
            topk = layer.topk_idx.cpu().numpy()
            o_sh, l_sh = O.shared_partials_fp8(q.cpu(), sf8.k8.cpu(), sf8.v8.cpu(), sf8.k_scale.cpu(),
                                               sf8.v_scale.cpu(), topk, layer.scale)
            o_u, l_u = O.attend_unique_fp8(q.cpu(), f8.k8.cpu(), f8.v8.cpu(), f8.k_scale.cpu(),
                                           f8.v_scale.cpu(), kv_start.cpu().numpy(), kv_len.cpu().numpy(),
                                           layer.scale)
            want, want_lse = O.merge(np.concatenate([o_sh, o_u[:, :, None, :]], axis=2),
                                     np.concatenate([l_sh, l_u[:, :, None]], axis=2))
            PU.check_attention(out.float().cpu().numpy(), want, f"all-fp8 decode step out (two_streams={two})")
            PU.check_lse(layer.lse_out.cpu().numpy(), want_lse, "all-fp8 decode step lse")
            assert M.device_status() == 0
            # the host-buffer form of the same step: same bits
            q_host = q.cpu().pin_memory()
            out_host = torch.zeros(w.B, w.Hq, w.D, dtype=torch.bfloat16).pin_memory()
            layer.step_fp8_host(q_host, torch.empty_like(q), out_host, sf8, f8, kv_start, kv_len,
                                two_streams=two, unique_tokens=int(kv_len.sum().item()))
            assert torch.equal(out_host, out.cpu())


def test_fp8_shared_rejects_what_it_does_not_serve():
    M, MoskaLayer = _mods()
    layer = MoskaLayer(4, 4, 1, 64, 8, 128, 2, 16)          # D = 64
    f8 = W.SharedStoreFp8(*(torch.zeros(1, device="cuda") for _ in range(4)))
    with pytest.raises(M.MoskaError) as e:
        layer.shared_fp8(torch.zeros(4, 4, 64, dtype=torch.bfloat16, device="cuda"), f8)
    assert e.value.status == M.ERR_UNSUPPORTED


def _dense_reference(q, sf8, C, slots, scale):
    """Oracle for dense mode over the FP8 shared store: the per-chunk partials of every row (all C
    chunks), merged over each run of ceil(C / slots) consecutive chunks."""
    B, Hq, _ = q.shape
    Hkv = sf8.k8.shape[0]
    all_chunks = np.tile(np.arange(C, dtype=np.int32), (B, Hkv, 1))
    o_c, l_c = O.shared_partials_fp8(q.cpu(), sf8.k8.cpu(), sf8.v8.cpu(), sf8.k_scale.cpu(), sf8.v_scale.cpu(),
                                     all_chunks, scale)
    run = (C + slots - 1) // slots
    o_r = np.zeros((B, Hq, slots, q.shape[2]))
    l_r = np.full((B, Hq, slots), -np.inf)
    for s in range(slots):
        c0, c1 = min(C, s * run), min(C, (s + 1) * run)
        if c1 > c0:
            o_r[:, :, s], l_r[:, :, s] = O.merge(o_c[:, :, c0:c1], l_c[:, :, c0:c1])
    return o_r, l_r


def test_fp8_shared_dense_mode_runs_of_chunks_with_different_scales():
    """Dense mode (no routing): a partial slot covers a run of chunks whose key and value scales
    differ, so the running maximum and the value scale have to carry across chunks.  Batches of one
    row tile (split over the two slots), two tiles, several items, a partial last run, G = 4 and 8."""
    M, MoskaLayer = _mods()
    for Hq, Hkv, B, C, L, slots in ((8, 2, 20, 6, 256, 3), (8, 2, 70, 5, 128, 2), (16, 2, 40, 4, 384, 4),
                                    (8, 2, 3, 7, 128, 3), (8, 2, 200, 3, 256, 1)):
        w = W.Workload("f8dense", B=B, Hq=Hq, Hkv=Hkv, D=128, C=C, L=L, k=C, unique_len=64, seed=300 + B)
        sh = W.make_shared_store(w, "cuda")
        # chunk-dependent magnitudes, so that the scales really differ from chunk to chunk
        mag = torch.linspace(0.5, 3.0, C, device="cuda").view(1, C, 1, 1)
        sh = W.SharedStore((sh.k_shared.float() * mag).to(torch.bfloat16), (sh.v_shared.float() * mag.flip(1)).to(torch.bfloat16), sh.mu)
        un = W.make_unique_store(w, "cuda")
        q = W.make_queries(w, sh, 0, "cuda")
        sf8 = W.quantize_shared_store_fp8(sh)
        layer = MoskaLayer(B, Hq, Hkv, 128, C, L, C, 64, dense=True, dense_slots=slots, n_unique_splits=2)
        layer.o_part.fill_(float("nan"))
        layer.lse_part.fill_(float("nan"))
        layer.shared_fp8(q, sf8)
        torch.cuda.synchronize()
        o_ref, l_ref = _dense_reference(q, sf8, C, slots, layer.scale)
        PU.check_lse(layer.lse_part[:, :, :slots].cpu().numpy(), l_ref, "fp8 dense lse")
        PU.check_attention(layer.o_part[:, :, :slots].cpu().numpy(), o_ref, "fp8 dense partial o")
        # the whole step, one and two streams
        dummy = torch.zeros(Hkv, 1, 128, 128, dtype=torch.bfloat16)
        o_un, l_un = O.attend_direct(q.cpu(), dummy, dummy, un.k_unique.cpu(), un.v_unique.cpu(),
                                     un.kv_start.cpu().numpy(), un.kv_len.cpu().numpy(),
                                     np.zeros((B, Hkv, 1), dtype=np.int32), layer.scale, use_shared=False)
        want, _ = O.merge(np.concatenate([o_ref, o_un[:, :, None, :]], axis=2),
                          np.concatenate([l_ref, l_un[:, :, None]], axis=2))
        for two in (False, True):
            out = layer.step_fp8shared(q, sf8, un.k_unique, un.v_unique, un.kv_start, un.kv_len, two_streams=two,
                                       unique_tokens=int(un.kv_len.sum().item()))
            torch.cuda.synchronize()
            PU.check_attention(out.float().cpu().numpy(), want, f"fp8 dense step out (two_streams={two})")
        assert M.device_status() == 0


def test_several_query_tokens_per_request_with_both_stores_in_fp8():
    """shape.q_len > 1 with the all-FP8 step: the batch rows are requests x q_len; shared attention
    treats every row as a request of its own, unique attention reads a request's codes once for all
    its tokens.  The oracle gets the batch-expanded problem (aliased kv_start, per-token context end)."""
    M, MoskaLayer = _mods()
    for Hq, Hkv, t, splits in ((8, 2, 2, 1), (4, 2, 4, 2), (8, 4, 3, 1)):
        lens_last = np.array([40, 1, 130, 77, 300, 16, 2, 0, 600, 65], dtype=np.int64)
        base = len(lens_last)
        w = W.Workload("f8multi", B=base * t, Hq=Hq, Hkv=Hkv, D=128, C=8, L=256, k=2, unique_len=0, seed=47)
        sh = W.make_shared_store(w, "cuda")
        un = W.make_unique_store(W.scaled(w, B=base, steps=0), "cuda", lens_last)
        q = W.make_queries(w, sh, 0, "cuda")
        sf8 = W.quantize_shared_store_fp8(sh)
        kv_start_dev, kv_len_dev = un.kv_start, un.kv_len
        f8 = W.quantize_unique_store_fp8(un)
        layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, int(lens_last.max()), n_unique_splits=splits,
                           fp8_unique=True, q_len=t)
        layer.build_summaries(sh.k_shared)
        out = layer.step_fp8(q, sf8, f8, kv_start_dev, kv_len_dev, two_streams=bool(t % 2))
        torch.cuda.synchronize()
        kv_start = kv_start_dev.repeat_interleave(t).cpu().numpy()
        back = np.tile(np.arange(t - 1, -1, -1), base)
        kv_len = np.maximum(0, np.repeat(lens_last, t) - back).astype(np.int32)
        o_sh, l_sh = O.shared_partials_fp8(q.cpu(), sf8.k8.cpu(), sf8.v8.cpu(), sf8.k_scale.cpu(),
                                           sf8.v_scale.cpu(), layer.topk_idx.cpu().numpy(), layer.scale)
        o_u, l_u = O.attend_unique_fp8(q.cpu(), f8.k8.cpu(), f8.v8.cpu(), f8.k_scale.cpu(), f8.v_scale.cpu(),
                                       kv_start, kv_len, layer.scale)
        want, want_lse = O.merge(np.concatenate([o_sh, o_u[:, :, None, :]], axis=2),
                                 np.concatenate([l_sh, l_u[:, :, None]], axis=2))
        PU.check_attention(out.float().cpu().numpy(), want, f"all-fp8 q_len={t} out")
        PU.check_lse(layer.lse_out.cpu().numpy(), want_lse, f"all-fp8 q_len={t} lse")
        assert M.device_status() == 0
