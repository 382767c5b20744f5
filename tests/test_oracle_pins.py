"""Pins of the fp64 CPU oracle against things other than itself.

Each test compares an oracle function with a brute-force restatement written here in plain
Python/numpy loops, with a closed form, with an invariant of the definition, or with an
independent library routine (torch SDPA in float64, torch.topk, numpy's stable argsort).  The
cases are chosen so that a dropped term, a wrong sign or index, a transposed operand or a wrong
tie-break fails at least one of them.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
TOL = 1e-12


def bf16(x):
    return torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)


def wide(t):
    """Exact bf16 -> float64 widening through torch (independent of the oracle's bit code)."""
    return t.to(torch.float64).numpy()


def tiny_problem(seed, B=3, Hq=4, Hkv=2, D=8, C=5, L=4, k=2, ulen=(3, 0, 6)):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ks = torch.randn(Hkv, C, L, D, generator=g).to(torch.bfloat16)
    vs = torch.randn(Hkv, C, L, D, generator=g).to(torch.bfloat16)
    lens = np.array([ulen[b % len(ulen)] for b in range(B)], dtype=np.int32)
    # leave a gap between requests so that a wrong kv_start shows
    start = np.concatenate([[0], np.cumsum(lens + 2)[:-1]]).astype(np.int64)
    T = int((lens + 2).sum())
    ku = torch.randn(T, Hkv, D, generator=g).to(torch.bfloat16)
    vu = torch.randn(T, Hkv, D, generator=g).to(torch.bfloat16)
    return dict(q=q, ks=ks, vs=vs, ku=ku, vu=vu, start=start, lens=lens,
                B=B, Hq=Hq, Hkv=Hkv, D=D, C=C, L=L, k=k, scale=1.0 / math.sqrt(D))


def brute_attention(p, topk):
    """Plain-loop softmax attention over [routed shared chunks || unique tokens] per row."""
    B, Hq, Hkv, D, L = p["B"], p["Hq"], p["Hkv"], p["D"], p["L"]
    G = Hq // Hkv
    q, ks, vs, ku, vu = (wide(p[n]) for n in ("q", "ks", "vs", "ku", "vu"))
    out = np.zeros((B, Hq, D))
    lse = np.full((B, Hq), -np.inf)
    for b in range(B):
        for hq in range(Hq):
            h = hq // G
            keys, vals = [], []
            for c in topk[b][h]:
                for t in range(L):
                    keys.append(ks[h, c, t])
                    vals.append(vs[h, c, t])
            for t in range(p["lens"][b]):
                keys.append(ku[p["start"][b] + t, h])
                vals.append(vu[p["start"][b] + t, h])
            if not keys:
                continue
            s = [p["scale"] * sum(q[b, hq, d] * kk[d] for d in range(D)) for kk in keys]
            z = sum(math.exp(x) for x in s)
            lse[b, hq] = math.log(z)
            for x, vv in zip(s, vals):
                out[b, hq] += math.exp(x) / z * vv
    return out, lse


# ---------------------------------------------------------------- summaries (closed forms, brute)
def test_summaries_identical_keys_and_cancelling_pairs():
    Hkv, C, L, D = 2, 3, 4, 8
    key = torch.randn(D).to(torch.bfloat16)
    ks = key.repeat(Hkv, C, L, 1).clone()
    # chunk (1, 2): +x / -x pairs -> mean exactly 0
    x = torch.randn(L // 2, D).to(torch.bfloat16)
    ks[1, 2, 0::2] = x
    ks[1, 2, 1::2] = -x
    s = O.chunk_summaries(ks)
    assert np.array_equal(s[0, 0], wide(key))          # mean of identical keys is that key
    assert np.array_equal(s[1, 2], np.zeros(D))
    assert s.shape == (Hkv, C, D)


def test_summaries_match_numpy_mean_and_indexing():
    g = torch.Generator().manual_seed(1)
    ks = torch.randn(2, 3, 8, 4, generator=g).to(torch.bfloat16)
    s = O.chunk_summaries(ks)
    ref = wide(ks).mean(axis=2)     # mean over the token axis only
    np.testing.assert_allclose(s, ref, rtol=0, atol=1e-15)
    # a transposed (token/dim) or head/chunk mix-up would break this spot check
    assert abs(s[1, 2, 3] - sum(float(ks[1, 2, t, 3]) for t in range(8)) / 8) < 1e-15


def test_attention_pooled_summaries_pins():
    """The second chunk embedding: softmax(scale <mean key, k_t>)-weighted mean of the keys.
    Pinned by (1) the library's attention routine with the mean key as the query and the chunk's
    keys as keys AND values, (2) plain loops, (3) scale = 0 -> the arithmetic mean, (4) identical
    keys -> that key, (5) one key far along the mean's direction takes all the weight, (6) the
    order of the tokens inside a chunk does not matter, a change of one chunk leaves the others."""
    g = torch.Generator().manual_seed(3)
    Hkv, C, L, D = 2, 3, 8, 4
    ks = torch.randn(Hkv, C, L, D, generator=g).to(torch.bfloat16)
    scale = 0.7
    s = O.chunk_summaries_attn(ks, scale)
    assert s.shape == (Hkv, C, D)
    K = ks.to(torch.float64)
    kbar = K.mean(dim=2, keepdim=True)                                  # [Hkv][C][1][D]
    ref = torch.nn.functional.scaled_dot_product_attention(kbar, K, K, scale=scale)[:, :, 0]
    np.testing.assert_allclose(s, ref.numpy(), rtol=0, atol=1e-13)
    # plain loops for one chunk: a swapped head/chunk index or a dropped max-subtraction shows
    h, c = 1, 2
    kk = wide(ks)[h, c]
    mean = [sum(kk[t][d] for t in range(L)) / L for d in range(D)]
    sc = [scale * sum(mean[d] * kk[t][d] for d in range(D)) for t in range(L)]
    z = sum(math.exp(x) for x in sc)
    brute = [sum(math.exp(sc[t]) / z * kk[t][d] for t in range(L)) for d in range(D)]
    np.testing.assert_allclose(s[h, c], brute, rtol=0, atol=1e-13)
    # scale 0: uniform weights = the mean embedding
    np.testing.assert_allclose(O.chunk_summaries_attn(ks, 0.0), O.chunk_summaries(ks), rtol=0, atol=1e-15)
    # identical keys
    key = torch.randn(D, generator=g).to(torch.bfloat16)
    same = key.repeat(1, 1, L, 1).clone()
    np.testing.assert_allclose(O.chunk_summaries_attn(same, 3.0)[0, 0], wide(key), rtol=0, atol=1e-15)
    # a dominant key: 7 keys e_0, one key 64 e_0 -> mean ~ 8.9 e_0, scores 8.9 vs 568: all weight on it
    dom = torch.zeros(1, 1, L, D)
    dom[..., 0] = 1.0
    dom[0, 0, 5, 0] = 64.0
    out = O.chunk_summaries_attn(dom.to(torch.bfloat16), 1.0)[0, 0]
    np.testing.assert_allclose(out, [64.0, 0, 0, 0], rtol=0, atol=1e-12)
    # token order inside a chunk is irrelevant; other chunks are untouched by a change in one
    perm = torch.randperm(L, generator=g)
    ks2 = ks.clone()
    ks2[0, 1] = ks[0, 1][perm]
    s2 = O.chunk_summaries_attn(ks2, scale)
    np.testing.assert_allclose(s2, s, rtol=0, atol=1e-14)
    ks3 = ks.clone()
    ks3[1, 0] = -ks[1, 0]
    s3 = O.chunk_summaries_attn(ks3, scale)
    assert np.array_equal(np.delete(s3.reshape(Hkv * C, D), 3, axis=0), np.delete(s.reshape(Hkv * C, D), 3, axis=0))
    assert not np.allclose(s3[1, 0], s[1, 0])


# ---------------------------------------------------------------- routing
def test_route_scores_and_exhaustive_topk():
    p = tiny_problem(2, B=4, Hq=6, Hkv=2, D=8, C=7, L=4, k=3)
    summ = O.chunk_summaries(p["ks"])
    idx, sc, allsc = O.route(p["q"], summ, p["k"], return_all=True)
    q = wide(p["q"]).reshape(p["B"], p["Hkv"], 3, p["D"])       # [B][Hkv][G][D]
    qbar = q.sum(axis=2)
    ref_scores = np.einsum("bhd,hcd->bhc", qbar, summ)
    np.testing.assert_allclose(allsc, ref_scores, rtol=0, atol=1e-13)
    for b in range(p["B"]):
        for h in range(p["Hkv"]):
            order = sorted(range(p["C"]), key=lambda c: (-ref_scores[b, h, c], c))[: p["k"]]
            assert list(idx[b, h]) == sorted(order)
            np.testing.assert_allclose(sc[b, h], ref_scores[b, h, sorted(order)], atol=1e-13)
    # library routine on tie-free input
    tk = torch.topk(torch.from_numpy(ref_scores), p["k"], dim=-1).indices.sort(dim=-1).values
    assert np.array_equal(idx, tk.numpy().astype(np.int32))


def test_route_ties_break_to_lower_index():
    Hkv, C, L, D, k = 1, 6, 2, 4, 3
    ks = torch.zeros(Hkv, C, L, D, dtype=torch.bfloat16)
    base = bf16([1.0, 0.5, -0.25, 2.0])
    # chunks 1, 3, 4 identical (exact tie), chunk 5 larger, chunks 0 and 2 smaller
    for c in (1, 3, 4):
        ks[0, c] = base
    ks[0, 5] = base * 2
    ks[0, 0] = -base
    ks[0, 2] = -base
    q = base.reshape(1, 1, D).clone()
    summ = O.chunk_summaries(ks)
    idx, _ = O.route(q, summ, k)
    assert list(idx[0, 0]) == [1, 3, 5]     # 5 first, then the two LOWEST of the tied 1, 3, 4
    # all-zero query: every score ties at 0 -> chunks 0..k-1
    idx0, sc0 = O.route(torch.zeros(2, 1, D, dtype=torch.bfloat16), summ, k)
    assert np.array_equal(idx0, np.tile(np.arange(k, dtype=np.int32), (2, 1, 1)))
    assert np.all(sc0 == 0)


def test_route_gqa_pooling_is_a_sum_and_G1_is_identity():
    g = torch.Generator().manual_seed(3)
    summ = torch.randn(2, 5, 8, generator=g, dtype=torch.float64).numpy()
    q = torch.randn(2, 2, 8, generator=g).to(torch.bfloat16)          # G = 1
    _, _, allsc = O.route(q, summ, 2, return_all=True)
    np.testing.assert_allclose(allsc, np.einsum("bhd,hcd->bhc", wide(q), summ), atol=1e-13)
    # G = 2 with the second head of each group zero gives the same scores as G = 1
    q2 = torch.zeros(2, 4, 8, dtype=torch.bfloat16)
    q2[:, 0::2] = q
    _, _, allsc2 = O.route(q2, summ, 2, return_all=True)
    np.testing.assert_array_equal(allsc, allsc2)


def test_route_permuting_chunks_permutes_selection():
    p = tiny_problem(4, C=6, k=2)
    summ = O.chunk_summaries(p["ks"])
    idx, _ = O.route(p["q"], summ, p["k"])
    perm = np.array([3, 0, 5, 1, 4, 2])
    summ_p = O.chunk_summaries(p["ks"][:, perm])           # new chunk i = old chunk perm[i]
    idx_p, _ = O.route(p["q"], summ_p, p["k"])
    back = np.sort(perm[idx_p], axis=-1)
    assert np.array_equal(back, idx)


# ---------------------------------------------------------------- grouping
def test_group_matches_stable_argsort_and_fast_variant():
    rng = np.random.default_rng(5)
    B, Hkv, C, k = 7, 3, 6, 3
    topk = np.stack([[np.sort(rng.choice(C, k, replace=False)) for _ in range(Hkv)]
                     for _ in range(B)]).astype(np.int32)
    off, ent = O.group_by_chunk(topk, C)
    P = B * Hkv * k
    pos = np.arange(P)
    keys = ((pos // k) % Hkv) * C + topk.reshape(-1)
    order = np.argsort(keys, kind="stable")
    assert np.array_equal(ent, order.astype(np.int32))
    counts = np.bincount(keys, minlength=Hkv * C)
    assert np.array_equal(off, np.concatenate([[0], np.cumsum(counts)]).astype(np.int32))
    off2, ent2 = O.group_by_chunk(topk, C, fast=True)
    assert np.array_equal(off, off2) and np.array_equal(ent, ent2)
    # duplicated request rows land next to each other in every segment they appear in
    topk[3] = topk[2]
    off, ent = O.group_by_chunk(topk, C)
    for key in range(Hkv * C):
        seg = list(ent[off[key]:off[key + 1]] // (Hkv * k))     # request ids
        if 2 in seg:
            assert seg[seg.index(2) + 1] == 3


# ---------------------------------------------------------------- attention: goldens, closed forms
def _read_golden(name):
    with open(os.path.join(GOLDEN, name)) as f:
        rows = [ln for ln in f if ln.strip() and not ln.startswith("#")]
    return [float(x) for x in rows[0].replace("|", " ").split()]


def _single_request(q, K, V, scale):
    """Oracle attention of one query head over an explicit unique-token list."""
    n, D = K.shape
    ks = torch.zeros(1, 1, 1, D, dtype=torch.bfloat16)
    topk = np.zeros((1, 1, 1), dtype=np.int32)
    out, lse = O.attend_direct(q.reshape(1, 1, D), ks, ks, K.reshape(n, 1, D), V.reshape(n, 1, D),
                               np.array([0]), np.array([n]), topk, scale, use_shared=False)
    return out[0, 0], lse[0, 0]


def test_golden_two_token_attention():
    o0, o1, lse_ref = _read_golden("attention_two_tokens.txt")
    out, lse = _single_request(bf16([1, 0]), bf16([[0, 0], [1, 0]]), bf16([[1, 0], [0, 1]]), 1.0)
    np.testing.assert_allclose(out, [o0, o1], atol=1e-15)
    assert abs(lse - lse_ref) < 1e-15


def test_golden_merge_two_partials():
    v = _read_golden("merge_two_partials.txt")
    lse_p = np.array([[v[0], v[1]]])
    o_p = np.array([[[v[2], v[3]], [v[4], v[5]]]])
    out, lse = O.merge(o_p, lse_p)
    np.testing.assert_allclose(out[0], [v[6], v[7]], atol=1e-15)
    assert abs(lse[0] - v[8]) < 1e-15


def test_attention_closed_forms():
    D, n = 8, 5
    g = torch.Generator().manual_seed(6)
    q = torch.randn(D, generator=g).to(torch.bfloat16)
    key = torch.randn(D, generator=g).to(torch.bfloat16)
    V = torch.randn(n, D, generator=g).to(torch.bfloat16)
    scale = 0.37
    s = scale * float(wide(q) @ wide(key))
    # all keys equal -> uniform weights
    out, lse = _single_request(q, key.repeat(n, 1), V, scale)
    np.testing.assert_allclose(out, wide(V).mean(axis=0), atol=TOL)
    assert abs(lse - (s + math.log(n))) < TOL
    # constant V -> out is that constant whatever the keys
    K = torch.randn(n, D, generator=g).to(torch.bfloat16)
    out, _ = _single_request(q, K, V[0].repeat(n, 1), scale)
    np.testing.assert_allclose(out, wide(V[0]), atol=TOL)
    # single token -> out = v, lse = s
    out, lse = _single_request(q, key.reshape(1, D), V[:1], scale)
    np.testing.assert_allclose(out, wide(V[0]), atol=TOL)
    assert abs(lse - s) < TOL
    # one dominant key -> out tends to its value
    big = (q.float() * 64).to(torch.bfloat16)
    K2 = torch.cat([big.reshape(1, D), torch.zeros(n - 1, D, dtype=torch.bfloat16)])
    out, _ = _single_request(q, K2, V, 1.0)
    np.testing.assert_allclose(out, wide(V[0]), atol=1e-9)
    # no tokens at all -> lse = -inf, out = 0, no NaN
    out, lse = _single_request(q, K[:0], V[:0], scale)
    assert lse == -np.inf and np.all(out == 0)


# ---------------------------------------------------------------- attention: brute force, SDPA
def test_direct_attention_matches_brute_force_loops():
    p = tiny_problem(7)
    summ = O.chunk_summaries(p["ks"])
    topk, _ = O.route(p["q"], summ, p["k"])
    out, lse = O.attend_direct(p["q"], p["ks"], p["vs"], p["ku"], p["vu"], p["start"], p["lens"],
                               topk, p["scale"])
    ref_out, ref_lse = brute_attention(p, topk)
    np.testing.assert_allclose(out, ref_out, atol=TOL)
    np.testing.assert_allclose(lse, ref_lse, atol=TOL)


def test_staged_partials_plus_merge_equal_direct_attention():
    p = tiny_problem(8, B=4, Hq=4, Hkv=2, D=16, C=6, L=8, k=3, ulen=(5, 0, 8, 1))
    summ = O.chunk_summaries(p["ks"])
    topk, _ = O.route(p["q"], summ, p["k"])
    direct, direct_lse = O.attend_direct(p["q"], p["ks"], p["vs"], p["ku"], p["vu"], p["start"],
                                         p["lens"], topk, p["scale"])
    o_sh, lse_sh = O.shared_partials(p["q"], p["ks"], p["vs"], topk, p["scale"])
    o_un, lse_un = O.attend_direct(p["q"], p["ks"], p["vs"], p["ku"], p["vu"], p["start"],
                                   p["lens"], topk, p["scale"], use_shared=False)
    o_all = np.concatenate([o_sh, o_un[:, :, None, :]], axis=2)
    lse_all = np.concatenate([lse_sh, lse_un[:, :, None]], axis=2)
    out, lse = O.merge(o_all, lse_all)
    np.testing.assert_allclose(out, direct, atol=TOL)
    np.testing.assert_allclose(lse, direct_lse, atol=TOL)
    # brute force agrees with both
    ref_out, ref_lse = brute_attention(p, topk)
    np.testing.assert_allclose(out, ref_out, atol=TOL)
    # merge is associative: merge(merge(first two), rest) == merge(all)
    o01, l01 = O.merge(o_all[:, :, :2], lse_all[:, :, :2])
    o_n = np.concatenate([o01[:, :, None, :], o_all[:, :, 2:]], axis=2)
    l_n = np.concatenate([l01[:, :, None], lse_all[:, :, 2:]], axis=2)
    out2, lse2 = O.merge(o_n, l_n)
    np.testing.assert_allclose(out2, out, atol=TOL)
    np.testing.assert_allclose(lse2, lse, atol=TOL)
    # and order-independent
    permuted = [3, 1, 0, 2]
    out3, _ = O.merge(o_all[:, :, permuted], lse_all[:, :, permuted])
    np.testing.assert_allclose(out3, out, atol=TOL)


def test_shared_partial_slot_is_that_chunk_alone_via_sdpa():
    p = tiny_problem(9, B=2, Hq=4, Hkv=2, D=8, C=4, L=6, k=2)
    topk = np.array([[[1, 3], [0, 2]], [[0, 1], [2, 3]]], dtype=np.int32)
    o_sh, lse_sh = O.shared_partials(p["q"], p["ks"], p["vs"], topk, p["scale"])
    G = 2
    for b in range(2):
        for hq in range(4):
            h = hq // G
            for j in range(2):
                c = topk[b, h, j]
                qq = p["q"][b, hq].double().reshape(1, 1, -1)
                kk = p["ks"][h, c].double().unsqueeze(0)
                vv = p["vs"][h, c].double().unsqueeze(0)
                ref = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, scale=p["scale"])
                np.testing.assert_allclose(o_sh[b, hq, j], ref[0, 0].numpy(), atol=TOL)
                ref_lse = torch.logsumexp(p["scale"] * (kk[0] @ qq[0, 0]), dim=0)
                assert abs(lse_sh[b, hq, j] - float(ref_lse)) < TOL


def test_k_equals_C_is_dense_attention_via_sdpa():
    p = tiny_problem(10, B=3, Hq=4, Hkv=2, D=8, C=4, L=4, k=4, ulen=(2, 5, 0))
    summ = O.chunk_summaries(p["ks"])
    topk, _ = O.route(p["q"], summ, p["k"])
    assert np.array_equal(topk, np.tile(np.arange(4, dtype=np.int32), (3, 2, 1)))
    out, lse = O.attend_direct(p["q"], p["ks"], p["vs"], p["ku"], p["vu"], p["start"], p["lens"],
                               topk, p["scale"])
    G = p["Hq"] // p["Hkv"]
    for b in range(p["B"]):
        s0, n = int(p["start"][b]), int(p["lens"][b])
        # [Hkv][S+U][D] then GQA by repeating KV heads
        K = torch.cat([p["ks"].reshape(p["Hkv"], -1, p["D"]), p["ku"][s0:s0 + n].transpose(0, 1)], 1)
        V = torch.cat([p["vs"].reshape(p["Hkv"], -1, p["D"]), p["vu"][s0:s0 + n].transpose(0, 1)], 1)
        K = K.double().repeat_interleave(G, dim=0)
        V = V.double().repeat_interleave(G, dim=0)
        qq = p["q"][b].double().unsqueeze(1)                     # [Hq][1][D]
        ref = torch.nn.functional.scaled_dot_product_attention(qq, K, V, scale=p["scale"])
        np.testing.assert_allclose(out[b], ref[:, 0].numpy(), atol=TOL)
        ref_lse = torch.logsumexp(p["scale"] * torch.einsum("hd,htd->ht", qq[:, 0], K), dim=1)
        np.testing.assert_allclose(lse[b], ref_lse.numpy(), atol=TOL)


# ---------------------------------------------------------------- invariances
def test_invariances_token_permutation_key_shift_duplicates():
    p = tiny_problem(11, B=3, Hq=4, Hkv=2, D=8, C=5, L=6, k=2, ulen=(4, 4, 4))
    summ = O.chunk_summaries(p["ks"])
    topk, _ = O.route(p["q"], summ, p["k"])
    args = (p["ku"], p["vu"], p["start"], p["lens"])
    out, lse = O.attend_direct(p["q"], p["ks"], p["vs"], *args, topk, p["scale"])
    # permute tokens inside every chunk (K and V together): summaries, routing, output unchanged
    perm = torch.tensor([4, 2, 0, 5, 1, 3])
    ks_p, vs_p = p["ks"][:, :, perm], p["vs"][:, :, perm]
    summ_p = O.chunk_summaries(ks_p)
    np.testing.assert_allclose(summ_p, summ, atol=1e-15)
    topk_p, _ = O.route(p["q"], summ_p, p["k"])
    assert np.array_equal(topk_p, topk)
    out_p, lse_p = O.attend_direct(p["q"], ks_p, vs_p, *args, topk, p["scale"])
    np.testing.assert_allclose(out_p, out, atol=TOL)
    np.testing.assert_allclose(lse_p, lse, atol=TOL)
    # permuting K but NOT V must change the result (guards against a check that cannot fail)
    out_bad, _ = O.attend_direct(p["q"], ks_p, p["vs"], *args, topk, p["scale"])
    assert np.abs(out_bad - out).max() > 1e-3
    # adding delta to every attended key: out unchanged, lse shifts by scale * <q, delta>.
    # (power-of-two data keeps q, k, k+delta exact in bf16)
    g = torch.Generator().manual_seed(12)
    qi = torch.randint(-4, 5, (1, 1, 8), generator=g).float().to(torch.bfloat16)
    K = torch.randint(-4, 5, (6, 1, 8), generator=g).float().to(torch.bfloat16)
    V = torch.randn(6, 1, 8, generator=g).to(torch.bfloat16)
    delta = torch.randint(-2, 3, (8,), generator=g).float().to(torch.bfloat16)
    z = torch.zeros(1, 1, 1, 8, dtype=torch.bfloat16)
    t0 = np.zeros((1, 1, 1), dtype=np.int32)
    a, la = O.attend_direct(qi, z, z, K, V, [0], [6], t0, 0.25, use_shared=False)
    b_, lb = O.attend_direct(qi, z, z, (K.float() + delta).to(torch.bfloat16), V, [0], [6], t0, 0.25,
                             use_shared=False)
    np.testing.assert_allclose(a, b_, atol=TOL)
    shift = 0.25 * float(wide(qi[0, 0]) @ wide(delta))
    assert abs((lb - la)[0, 0] - shift) < TOL
    # duplicated request -> identical outputs
    q2 = p["q"].clone()
    q2[2] = q2[0]
    lens2 = p["lens"].copy()
    ku2, vu2 = p["ku"].clone(), p["vu"].clone()
    s0, s2 = int(p["start"][0]), int(p["start"][2])
    ku2[s2:s2 + 4], vu2[s2:s2 + 4] = ku2[s0:s0 + 4], vu2[s0:s0 + 4]
    topk2, _ = O.route(q2, summ, p["k"])
    out2, lse2 = O.attend_direct(q2, p["ks"], p["vs"], ku2, vu2, p["start"], lens2, topk2, p["scale"])
    assert np.array_equal(out2[0], out2[2]) and np.array_equal(lse2[0], lse2[2])


def test_merge_degenerate_slots():
    o = np.array([[[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]]])
    ninf = -np.inf
    out, lse = O.merge(o, np.array([[ninf, 0.5, ninf]]))
    np.testing.assert_allclose(out[0], [3.0, 4.0], atol=0)
    assert lse[0] == 0.5
    out, lse = O.merge(o, np.array([[ninf, ninf, ninf]]))
    assert np.all(out == 0) and lse[0] == ninf
    # an empty slot may hold garbage (even NaN-free huge values) without contributing
    o[0, 0] = 1e300
    out, _ = O.merge(o, np.array([[ninf, 0.0, 0.0]]))
    np.testing.assert_allclose(out[0], [4.0, 5.0], atol=TOL)


def test_generator_structure_target_chunk_is_top1():
    """The synthetic workload makes routing checkable in kind: the chunk a query was drawn around
    must be the best-scoring one (routing quality has no other pin)."""
    from paper_2511_06010_b200 import workloads as W

    w = W.CONFIGS[0]
    sh = W.make_shared_store(w)
    q = W.make_queries(w, sh)
    summ = O.chunk_summaries(sh.k_shared)
    _, _, allsc = O.route(q, summ, w.k, return_all=True)
    tgt = W.query_targets(w)
    assert np.array_equal(allsc.argmax(axis=-1)[:, 0], tgt)
