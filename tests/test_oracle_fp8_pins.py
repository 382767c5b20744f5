"""Pins of the FP8 part of the oracle (CPU only): the E4M3 decoder against torch's own conversion
of all 256 codes and against hand-computed values of the format, and the FP8 attention against the
bf16 oracle on stores that are exactly representable in both and against a brute-force loop."""
import math

import numpy as np
import torch

from oracle import oracle as O
from paper_2511_06010_b200 import workloads as W


def test_e4m3_decoder_matches_the_format_and_torch():
    vals = O.e4m3_values()
    # values fixed by the format: zero, smallest subnormal, largest subnormal, 1, 1.125, max 448
    assert vals[0x00] == 0.0 and vals[0x80] == 0.0 and math.copysign(1, vals[0x80]) == -1
    assert vals[0x01] == 2.0 ** -9 and vals[0x07] == 7 * 2.0 ** -9 and vals[0x08] == 2.0 ** -6
    assert vals[0x38] == 1.0 and vals[0x39] == 1.125 and vals[0x7E] == 448.0 and vals[0xFE] == -448.0
    assert np.isnan(vals[0x7F]) and np.isnan(vals[0xFF])
    # an independent library's decoder, all 256 codes
    ref = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(vals), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(vals[ok], ref[ok])


def _small(seed=0, B=3, Hq=4, Hkv=2, D=16, lens=(5, 0, 9)):
    g = torch.Generator().manual_seed(seed)
    T = int(sum(lens))
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    k = torch.randn(T, Hkv, D, generator=g).to(torch.bfloat16)
    v = torch.randn(T, Hkv, D, generator=g).to(torch.bfloat16)
    start = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int64)
    return q, k, v, start, np.asarray(lens, dtype=np.int32)


def test_fp8_attention_equals_bf16_attention_on_a_store_both_formats_hold_exactly():
    q, k, v, start, lens = _small()
    # round the store to the E4M3 grid (scale 1): every value is then exact in bf16 AND in E4M3
    k = k.float().clamp(-448, 448).to(torch.float8_e4m3fn)
    v = v.float().clamp(-448, 448).to(torch.float8_e4m3fn)
    kb, vb = k.to(torch.bfloat16), v.to(torch.bfloat16)
    assert torch.equal(kb.float(), k.float()) and torch.equal(vb.float(), v.float())
    ones = np.ones(k.shape[:2], dtype=np.float32)
    o8, l8 = O.attend_unique_fp8(q, k.view(torch.uint8), v.view(torch.uint8), ones, ones, start, lens, 0.25)
    dummy = torch.zeros(k.shape[1], 1, 128, k.shape[-1], dtype=torch.bfloat16)  # unused shared store
    ob, lb = O.attend_direct(q, dummy, dummy, kb, vb, start, lens,
                             np.zeros((q.shape[0], k.shape[1], 1), dtype=np.int32), 0.25,
                             use_shared=False)
    np.testing.assert_allclose(o8, ob, rtol=0, atol=1e-13)
    assert np.array_equal(np.isneginf(l8), np.isneginf(lb))
    np.testing.assert_allclose(l8[~np.isneginf(lb)], lb[~np.isneginf(lb)], rtol=0, atol=1e-13)


def test_fp8_attention_against_a_brute_force_loop_with_scales():
    q, k, v, start, lens = _small(seed=3)
    un = W.UniqueStore(k, v, torch.from_numpy(start), torch.from_numpy(lens), torch.from_numpy(lens.astype(np.int64)))
    f8 = W.quantize_unique_store_fp8(un)
    scale = 1.0 / math.sqrt(q.shape[-1])
    out, lse = O.attend_unique_fp8(q, f8.k8, f8.v8, f8.k_scale, f8.v_scale, start, lens, scale)
    kd = f8.k8.view(torch.float8_e4m3fn).to(torch.float64) * f8.k_scale[..., None].to(torch.float64)
    vd = f8.v8.view(torch.float8_e4m3fn).to(torch.float64) * f8.v_scale[..., None].to(torch.float64)
    B, Hq, D = q.shape
    G = Hq // k.shape[1]
    for b in range(B):
        for hq in range(Hq):
            h = hq // G
            n = int(lens[b])
            if n == 0:
                assert lse[b, hq] == -np.inf and not out[b, hq].any()
                continue
            qq = q[b, hq].to(torch.float64)
            s = torch.tensor([scale * float(qq @ kd[start[b] + t, h]) for t in range(n)], dtype=torch.float64)
            ref_lse = float(torch.logsumexp(s, 0))
            p = torch.exp(s - ref_lse)
            ref = sum(p[t] * vd[start[b] + t, h] for t in range(n))
            np.testing.assert_allclose(out[b, hq], ref.numpy(), rtol=0, atol=1e-12)
            assert abs(lse[b, hq] - ref_lse) < 1e-12
    # the quantiser really is a storage conversion: dequantised values are close to the originals
    assert float((kd.float() - k.float()).abs().max()) < 0.07 * float(k.float().abs().max())


def _small_shared(seed=5, B=3, Hq=4, Hkv=2, D=16, C=4, L=8, k=2):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ks = (torch.randn(Hkv, C, L, D, generator=g) * torch.rand(Hkv, C, 1, 1, generator=g) * 3).to(torch.bfloat16)
    vs = (torch.randn(Hkv, C, L, D, generator=g) * (0.2 + torch.rand(Hkv, C, 1, 1, generator=g))).to(torch.bfloat16)
    topk = np.stack([np.stack([np.sort(np.random.default_rng(seed + 7 * b + h).choice(C, k, replace=False))
                               for h in range(Hkv)]) for b in range(B)]).astype(np.int32)
    return q, ks, vs, topk


def test_fp8_shared_partials_equal_bf16_partials_on_a_store_both_formats_hold_exactly():
    """Codes on the E4M3 grid with per-chunk scales that are powers of two: every stored value is
    exact in bf16 too, so the FP8 staged partials must equal the bf16 oracle's (pinned elsewhere
    against brute force and the library's attention routine).  A scale applied to the wrong chunk
    or head, or a K scale used for V, changes the result."""
    q, ks, vs, topk = _small_shared()
    Hkv, C = ks.shape[:2]
    k8 = ks.float().clamp(-448, 448).to(torch.float8_e4m3fn)
    v8 = vs.float().clamp(-448, 448).to(torch.float8_e4m3fn)
    rng = np.random.default_rng(1)
    ksc = (2.0 ** rng.integers(-3, 3, size=(Hkv, C))).astype(np.float32)
    vsc = (2.0 ** rng.integers(-3, 3, size=(Hkv, C))).astype(np.float32)
    assert len(np.unique(ksc)) > 2 and not np.array_equal(ksc, vsc)
    kb = (k8.float() * torch.from_numpy(ksc)[:, :, None, None]).to(torch.bfloat16)
    vb = (v8.float() * torch.from_numpy(vsc)[:, :, None, None]).to(torch.bfloat16)
    assert torch.equal(kb.float(), k8.float() * torch.from_numpy(ksc)[:, :, None, None])
    o8, l8 = O.shared_partials_fp8(q, k8.view(torch.uint8), v8.view(torch.uint8), ksc, vsc, topk, 0.25)
    ob, lb = O.shared_partials(q, kb, vb, topk, 0.25)
    np.testing.assert_allclose(o8, ob, rtol=0, atol=1e-13)
    np.testing.assert_allclose(l8, lb, rtol=0, atol=1e-13)


def test_fp8_shared_partials_against_a_brute_force_loop_with_quantiser_scales():
    q, ks, vs, topk = _small_shared(seed=9)
    f8 = W.quantize_shared_store_fp8(W.SharedStore(ks, vs, None))
    assert f8.k_scale.shape == ks.shape[:2] and f8.k8.dtype == torch.uint8
    scale = 1.0 / math.sqrt(q.shape[-1])
    o, lse = O.shared_partials_fp8(q, f8.k8, f8.v8, f8.k_scale, f8.v_scale, topk, scale)
    kd = f8.k8.view(torch.float8_e4m3fn).to(torch.float64) * f8.k_scale[:, :, None, None].to(torch.float64)
    vd = f8.v8.view(torch.float8_e4m3fn).to(torch.float64) * f8.v_scale[:, :, None, None].to(torch.float64)
    B, Hq, D = q.shape
    G = Hq // ks.shape[0]
    L = ks.shape[2]
    for b in range(B):
        for hq in range(Hq):
            h = hq // G
            for j, c in enumerate(topk[b, h]):
                qq = q[b, hq].to(torch.float64)
                s = torch.tensor([scale * float(qq @ kd[h, c, t]) for t in range(L)], dtype=torch.float64)
                ref_lse = float(torch.logsumexp(s, 0))
                p = torch.exp(s - ref_lse)
                ref = sum(p[t] * vd[h, c, t] for t in range(L))
                np.testing.assert_allclose(o[b, hq, j], ref.numpy(), rtol=0, atol=1e-12)
                assert abs(lse[b, hq, j] - ref_lse) < 1e-12
    # the quantiser is a storage conversion: every chunk uses the full code range, values stay close
    assert int(f8.k8.view(torch.float8_e4m3fn).float().abs().amax(dim=(-1, -2)).min()) == 448
    assert float((kd.float() - ks.float()).abs().max()) < 0.07 * float(ks.float().abs().max())
