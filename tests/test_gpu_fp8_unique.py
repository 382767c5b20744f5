"""GPU parity of Unique KV Attention over an FP8 (E4M3) private store against the fp64 oracle, on
the same codes and scales, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2511_06010_b200 import workloads as W
from tests import parity_utils as PU

pytestmark = pytest.mark.gpu


def _run(w, lengths=None, n_unique_splits=None, sample=None):
    from paper_2511_06010_b200 import binding as M
    from paper_2511_06010_b200.engine import MoskaLayer

    sh = W.make_shared_store(W.scaled(w, C=max(2, w.k), L=128), "cuda")  # only for the query centres
    un = W.make_unique_store(w, "cuda", lengths)
    f8 = W.quantize_unique_store_fp8(un)
    q = W.make_queries(W.scaled(w, C=max(2, w.k), L=128), sh, 0, "cuda")
    max_len = int(un.kv_len.max().item()) if w.B else 1
    layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, max(2, w.k), 128, w.k, max(1, max_len),
                       n_unique_splits=n_unique_splits)
    n_sh = layer.shape.shared_slots
    layer.o_part.fill_(float("nan"))
    layer.lse_part.fill_(float("nan"))
    layer.unique_fp8(q, f8, un.kv_start, un.kv_len)
    torch.cuda.synchronize()
    rows = np.arange(w.B) if sample is None else np.asarray(sample)
    o_un = layer.o_part[rows][:, :, n_sh:].cpu().numpy()
    l_un = layer.lse_part[rows][:, :, n_sh:].cpu().numpy()
    assert not np.isnan(l_un).any() and np.isfinite(o_un).all(), "a unique slot was left unwritten"
    o_m, l_m = O.merge(o_un, l_un)
    # the oracle on the sampled requests only (their tokens compacted)
    lens = un.kv_len.cpu().numpy()[rows].astype(np.int32)
    starts = un.kv_start.cpu().numpy()[rows]
    new_start = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int64)
    sel = np.concatenate([np.arange(s, s + n) for s, n in zip(starts, lens)] + [np.zeros(0, dtype=np.int64)])
    sel_t = torch.from_numpy(sel.astype(np.int64)).to("cuda")
    pick = (lambda t: t.index_select(0, sel_t).cpu()) if len(sel) else (lambda t: t[:1].cpu())
    ref_o, ref_l = O.attend_unique_fp8(q[rows].cpu(), pick(f8.k8), pick(f8.v8), pick(f8.k_scale),
                                       pick(f8.v_scale), new_start, lens, layer.scale)
    PU.check_lse(l_m, ref_l, "fp8 unique lse")
    PU.check_attention(o_m, ref_o, "fp8 unique o")
    assert M.device_status() == 0


def test_fp8_unique_ragged_tails_and_empty_requests():
    lens = np.array([0, 1, 15, 16, 17, 63, 64, 65, 127, 129, 1000, 5, 300], dtype=np.int64)
    for Hq, Hkv in ((8, 2), (8, 1), (16, 2), (6, 2)):
        w = W.Workload("fp8", B=len(lens), Hq=Hq, Hkv=Hkv, D=128, C=4, L=128, k=2, unique_len=0, seed=7)
        _run(w, lengths=lens, n_unique_splits=3)
        _run(w, lengths=lens, n_unique_splits=1)


def test_fp8_unique_full_cfg1_sampled():
    w = W.CONFIGS[1]
    _run(w, sample=np.sort(np.random.default_rng(7).choice(w.B, size=6, replace=False)))


def test_fp8_unique_full_cfg2_sampled_with_the_default_splits():
    """Workload 2 at full size (2 M private tokens), the split count the bench uses for FP8."""
    from paper_2511_06010_b200 import binding as M

    w = W.CONFIGS[2]
    splits = M.default_unique_splits_fp8(w.B, w.Hkv, w.unique_len)
    _run(w, n_unique_splits=splits, sample=np.sort(np.random.default_rng(9).choice(w.B, size=3, replace=False)))


def _step_case(w, two_streams, lengths=None, unique_tokens=0):
    """The whole decode step with an FP8 private store against the oracle's shared partials
    (bf16 store) and FP8 unique partial, combined by the oracle's merge."""
    from paper_2511_06010_b200 import binding as M
    from paper_2511_06010_b200.engine import MoskaLayer
    from tests.test_gpu_parity import _subproblem

    sh = W.make_shared_store(w, "cuda")
    un = W.make_unique_store(w, "cuda", lengths)
    f8 = W.quantize_unique_store_fp8(un)
    q = W.make_queries(w, sh, 0, "cuda")
    max_len = int(un.kv_len.max().item())
    layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, max(1, max_len))
    layer.build_summaries(sh.k_shared)
    out = layer.step_fp8kv(q, sh.k_shared, sh.v_shared, f8, un.kv_start, un.kv_len,
                           two_streams=two_streams, unique_tokens=unique_tokens)
    torch.cuda.synchronize()
    assert M.device_status() == 0
    sample = np.arange(w.B)
    q_s, topk_s, ks, vs, _, _, st_s, len_s = _subproblem(q, layer.topk_idx, sh, un, un.kv_len, sample)
    o_sh, l_sh = O.shared_partials(q_s, ks, vs, topk_s, layer.scale)
    sel = np.concatenate([np.arange(s, s + n) for s, n in
                          zip(un.kv_start.cpu().numpy(), un.kv_len.cpu().numpy())]).astype(np.int64)
    sel_t = torch.from_numpy(sel).to("cuda")
    o_u, l_u = O.attend_unique_fp8(q_s, f8.k8.index_select(0, sel_t).cpu(), f8.v8.index_select(0, sel_t).cpu(),
                                   f8.k_scale.index_select(0, sel_t).cpu(),
                                   f8.v_scale.index_select(0, sel_t).cpu(), st_s, len_s, layer.scale)
    ref_o, ref_l = O.merge(np.concatenate([o_sh, o_u[:, :, None, :]], axis=2),
                           np.concatenate([l_sh, l_u[:, :, None]], axis=2))
    PU.check_attention(out.float().cpu().numpy(), ref_o, "fp8kv decode step out")
    PU.check_lse(layer.lse_out.cpu().numpy(), ref_l, "fp8kv decode step lse")


def test_fp8kv_decode_step_one_and_two_streams():
    lens = np.array([300, 1, 0, 1000, 64, 17, 129, 511, 2048, 77, 5, 900, 33, 640, 256, 4], dtype=np.int64)
    w = W.scaled(W.CONFIGS[1], B=16, C=16, k=4, unique_len=0)
    _step_case(w, two_streams=False, lengths=lens)
    _step_case(w, two_streams=True, lengths=lens)
    # the share of SMs branch of the schedule (long unique attention announced by the hint)
    _step_case(w, two_streams=True, lengths=lens, unique_tokens=1 << 26)


def test_fp8_unique_several_query_tokens_per_request():
    """shape.q_len > 1 with the FP8 store: one pass over a request's codes for all its query tokens;
    the oracle is given the same problem with every token as a request of its own."""
    from paper_2511_06010_b200 import binding as M
    from paper_2511_06010_b200.engine import MoskaLayer

    lens_last = np.array([40, 1, 130, 77, 300, 16, 2, 0, 1000, 65, 3], dtype=np.int64)
    base = len(lens_last)
    for Hq, Hkv, t, splits in ((8, 2, 2, 1), (8, 2, 2, 3), (4, 2, 4, 2), (6, 2, 2, 2), (4, 4, 5, 1)):
        w = W.Workload("fp8multi", B=base * t, Hq=Hq, Hkv=Hkv, D=128, C=4, L=128, k=2, unique_len=0, seed=11)
        sh = W.make_shared_store(w, "cuda")
        un = W.make_unique_store(W.scaled(w, B=base, steps=0), "cuda", lens_last)
        f8 = W.quantize_unique_store_fp8(un)
        q = W.make_queries(w, sh, 0, "cuda")
        layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, int(lens_last.max()),
                           n_unique_splits=splits, q_len=t, fp8_unique=True)
        n_sh = layer.shape.shared_slots
        layer.o_part.fill_(float("nan"))
        layer.lse_part.fill_(float("nan"))
        layer.unique_fp8(q, f8, un.kv_start, un.kv_len)
        torch.cuda.synchronize()
        o_un = layer.o_part[:, :, n_sh:].cpu().numpy()
        l_un = layer.lse_part[:, :, n_sh:].cpu().numpy()
        assert not np.isnan(l_un).any() and np.isfinite(o_un).all(), "a unique slot was left unwritten"
        o_m, l_m = O.merge(o_un, l_un)
        kv_start = un.kv_start.repeat_interleave(t).cpu().numpy()
        back = np.tile(np.arange(t - 1, -1, -1), base)
        kv_len = np.maximum(0, np.repeat(lens_last, t) - back).astype(np.int32)
        ref_o, ref_l = O.attend_unique_fp8(q.cpu(), f8.k8.cpu(), f8.v8.cpu(), f8.k_scale.cpu(),
                                           f8.v_scale.cpu(), kv_start, kv_len, layer.scale)
        PU.check_lse(l_m, ref_l, f"fp8 q_len={t} lse")
        PU.check_attention(o_m, ref_o, f"fp8 q_len={t} o")
        assert M.device_status() == 0
