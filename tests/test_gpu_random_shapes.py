"""Seeded random shapes through the whole path against the oracle: combinations of batch, group
size, chunk count and length, top-k, ragged private contexts and schedules that the hand-picked
cases of the other files do not enumerate (segments on every work list at once, pair and split
rounds of every length, dense runs of uneven length).  Every stage is compared in full by
`run_case`; D = 128 shapes also run with both KV stores in FP8."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2511_06010_b200 import workloads as W
from tests import parity_utils as PU
from tests.test_gpu_parity import run_case

pytestmark = pytest.mark.gpu


def _shapes(seed, n):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        Hkv = int(rng.choice([1, 2, 4]))
        G = int(rng.choice([1, 2, 4, 8]))
        D = 64 if i % 7 == 6 else 128
        C = int(rng.integers(1, 25))
        L = int(rng.choice([128, 256, 384, 512]))
        dense = bool(i % 5 == 4)
        k = C if dense else int(rng.integers(1, min(C, 8) + 1))
        B = int(rng.choice([1, 2, 3, 7, 17, 33, 64, 65, 100, 140]))
        if B * Hkv * G * (k * L) > 6e7:      # keeps the oracle to a second or so per case
            B = max(1, int(6e7 // (Hkv * G * k * L)))
        lens = rng.integers(0, 500, size=B).astype(np.int64)
        lens[rng.random(B) < 0.15] = 0
        out.append((W.Workload(f"rnd{seed}_{i}", B=B, Hq=Hkv * G, Hkv=Hkv, D=D, C=C, L=L, k=k, unique_len=0,
                               seed=1000 * seed + i, zipf_s=float(rng.choice([0.0, 1.1]))), lens, dense))
    return out


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_random_shapes_bf16_every_stage(seed):
    for j, (w, lens, dense) in enumerate(_shapes(seed, 12)):
        slots = None
        if dense:
            slots = max(1, min(w.C, 1 + j % 4))
        run_case(w, lengths=lens, n_unique_splits=1 + j % 3, two_streams=bool(j % 2), dense_slots=slots,
                 unique_tokens=int(lens.sum()) * (10 ** (j % 3)))


@pytest.mark.parametrize("seed", [5, 6])
def test_random_shapes_both_stores_in_fp8(seed):
    from paper_2511_06010_b200 import binding as M
    from paper_2511_06010_b200.engine import MoskaLayer

    for j, (w, lens, dense) in enumerate(_shapes(seed, 14)):
        if w.D != 128 or w.G > 8:
            continue
        sh = W.make_shared_store(w, "cuda")
        un = W.make_unique_store(w, "cuda", lens)
        q = W.make_queries(w, sh, 0, "cuda")
        sf8 = W.quantize_shared_store_fp8(sh)
        kv_start, kv_len = un.kv_start, un.kv_len
        f8 = W.quantize_unique_store_fp8(un)
        slots = max(1, min(w.C, 1 + j % 4)) if dense else None
        layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, max(1, int(lens.max())), dense=dense,
                           dense_slots=slots, n_unique_splits=1 + j % 3, fp8_unique=True)
        if not dense:
            layer.build_summaries(sh.k_shared)
        out = layer.step_fp8(q, sf8, f8, kv_start, kv_len, two_streams=bool(j % 2),
                             unique_tokens=int(lens.sum())).clone()
        torch.cuda.synchronize()
        n_sh = layer.shape.shared_slots
        if dense:
            topk = np.tile(np.arange(w.C, dtype=np.int32), (w.B, w.Hkv, 1))
        else:
            topk = layer.topk_idx.cpu().numpy()
        o_c, l_c = O.shared_partials_fp8(q.cpu(), sf8.k8.cpu(), sf8.v8.cpu(), sf8.k_scale.cpu(),
                                         sf8.v_scale.cpu(), topk, layer.scale)
        o_u, l_u = O.attend_unique_fp8(q.cpu(), f8.k8.cpu(), f8.v8.cpu(), f8.k_scale.cpu(), f8.v_scale.cpu(),
                                       kv_start.cpu().numpy(), kv_len.cpu().numpy(), layer.scale)
        want, want_lse = O.merge(np.concatenate([o_c, o_u[:, :, None, :]], axis=2),
                                 np.concatenate([l_c, l_u[:, :, None]], axis=2))
        PU.check_attention(out.float().cpu().numpy(), want, f"all-fp8 step out, {w.name}")
        PU.check_lse(layer.lse_out.cpu().numpy(), want_lse, f"all-fp8 step lse, {w.name}")
        assert torch.isfinite(layer.o_part[:, :, :n_sh]).all()
        assert M.device_status() == 0
