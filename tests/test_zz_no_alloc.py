"""The allocation-free grouping entry point against the regular one.

`moska_group_by_chunk_noalloc` serves hosts that cannot hand the library a workspace (all device
memory already owned by their own pool, or no allocation allowed on their hot path): its scratch
is a fixed buffer inside the library.  It must give exactly the segments the regular call gives,
call after call, although all calls share that one buffer.  This file is collected last on
purpose, so a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

from paper_2511_06010_b200 import workloads as W


def _binding():
    from paper_2511_06010_b200 import build

    build.build()
    from paper_2511_06010_b200 import binding as M

    return M


def test_noalloc_rejects_shapes_beyond_its_buffer_on_the_host():
    """A shape whose grouping scratch exceeds the built-in buffer is refused before any launch."""
    M = _binding()
    big = M.shape(1024, 64, 8, 128, 32768, 512, 32)     # 8 * 32768 keys x 32 words: > 8 MiB
    assert M.workspace_bytes(big) > (8 << 20)
    with pytest.raises(M.MoskaError) as e:
        M.group_by_chunk_noalloc(0x1000, 0x1000, 0x1000, big, stream=0)
    assert e.value.status == M.ERR_WORKSPACE
    assert "built-in buffer" in M.last_error()


@pytest.mark.gpu
def test_noalloc_wide_bit_sets_against_the_oracle_and_allocates_nothing():
    """More than 64 requests (bit sets wider than two words take the separate counting pass) on a
    shape whose scratch nearly fills the built-in buffer, compared with the CPU oracle's grouping
    directly; the device's free memory must not move across a call."""
    from oracle import oracle as O

    M = _binding()
    rng = np.random.default_rng(5)
    B, Hq, Hkv, D, C, L, k = 300, 8, 8, 128, 12288, 128, 24
    s = M.shape(B, Hq, Hkv, D, C, L, k)
    # grouping scratch = the whole workspace minus the router's score array (C > 256)
    scratch = M.workspace_bytes(s) - (4 * B * Hkv * C + 255) // 256 * 256
    assert 0.8 * (8 << 20) < scratch <= (8 << 20), scratch
    topk = np.empty((B, Hkv, k), dtype=np.int32)
    # skewed: the low chunks are popular, so some segments hold most of the batch
    p = 1.0 / np.arange(1, C + 1) ** 1.2
    p /= p.sum()
    for b in range(B):
        for h in range(Hkv):
            topk[b, h] = np.sort(rng.choice(C, size=k, replace=False, p=p))
    t_dev = torch.from_numpy(topk).cuda()
    off = torch.full((Hkv * C + 1,), -1, dtype=torch.int32, device="cuda")
    ent = torch.full((B * Hkv * k,), -1, dtype=torch.int32, device="cuda")
    M.group_by_chunk_noalloc(t_dev, off, ent, s)          # first call on the device: set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    off.fill_(-1)
    ent.fill_(-1)
    M.group_by_chunk_noalloc(t_dev, off, ent, s)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "the allocation-free call changed the device's free memory"
    off_ref, ent_ref = O.group_by_chunk(topk, C, fast=True)
    assert np.array_equal(off.cpu().numpy(), off_ref)
    assert np.array_equal(ent.cpu().numpy(), ent_ref)
    assert M.device_status() == 0


@pytest.mark.gpu
def test_noalloc_matches_regular_grouping_on_two_calls_in_a_row():
    M = _binding()
    from paper_2511_06010_b200.engine import MoskaLayer

    dev = "cuda"
    # two different routings, the second one sparser and smaller than the first: leftovers of
    # call 1 in the shared buffer would corrupt call 2 if they were not cleared
    cases = [W.scaled(W.CONFIGS[1], B=48, C=64, k=8, unique_len=16, seed=11),
             W.scaled(W.CONFIGS[2], B=20, C=96, k=4, unique_len=16, seed=12)]
    for w in cases:
        sh = W.make_shared_store(w, dev)
        q = W.make_queries(w, sh, 0, dev)
        layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, 16)
        layer.build_summaries(sh.k_shared)
        layer.route(q)
        layer.group()                                   # regular entry point, caller workspace
        torch.cuda.synchronize()
        ref_off = layer.seg_offsets.clone()
        ref_ent = layer.seg_entries.clone()
        off = torch.full_like(ref_off, -1)
        ent = torch.full_like(ref_ent, -1)
        M.group_by_chunk_noalloc(layer.topk_idx, off, ent, layer.shape)
        torch.cuda.synchronize()
        # integer work: bit-exact, the same tolerance the other grouping tests use
        assert torch.equal(off, ref_off), f"{w.name}: seg_offsets differ"
        assert torch.equal(ent, ref_ent), f"{w.name}: seg_entries differ"
        assert int(off[-1]) == w.B * w.Hkv * w.k
        # and once more on the same input: a repeated call reproduces itself
        off2 = torch.full_like(ref_off, -1)
        ent2 = torch.full_like(ref_ent, -1)
        M.group_by_chunk_noalloc(layer.topk_idx, off2, ent2, layer.shape)
        torch.cuda.synchronize()
        assert torch.equal(off2, ref_off) and torch.equal(ent2, ref_ent)
