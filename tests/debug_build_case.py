"""Run as a script by test_gpu_debug_build.py with MOSKA_LIB pointing at the debug build of the
library (guard words behind every workspace region, capacity checks on the work lists).

1. A whole decode step against the oracle, every stage (the guard words stay intact and the debug
   checks stay silent on a correct run; the larger workspace layout changes no result).
2. A guard word overwritten from the host side is found by moska_debug_check_workspace and
   reported as ERR_CORRUPT through the device status word; the word is cleared by the read.
"""
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2511_06010_b200 import binding as M  # noqa: E402
from paper_2511_06010_b200 import workloads as W  # noqa: E402
from paper_2511_06010_b200.engine import MoskaLayer  # noqa: E402
import test_gpu_parity as T  # noqa: E402

assert M.LIB_PATH.endswith("libmoska_debug.so"), M.LIB_PATH

# 1. parity of a step whose segments land on all three work lists, few and many chunks
for w in (W.scaled(W.CONFIGS[1], B=48, C=16, k=4, unique_len=300),
          W.scaled(W.CONFIGS[2], B=24, C=320, k=6, unique_len=200)):
    rep = T.run_case(w, two_streams=True)
    assert M.device_status() == 0
print("debug build: parity ok")

# 2. guard words: intact after a step, found when overwritten
w = W.scaled(W.CONFIGS[1], B=32, C=8, k=2, unique_len=128)
sh = W.make_shared_store(w, "cuda")
q = W.make_queries(w, sh, 0, "cuda")
layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, 16)
layer.build_summaries(sh.k_shared)
layer.route(q)
layer.group()
layer.shared(q, sh.k_shared, sh.v_shared)
M.debug_check_workspace(layer.ws, layer.shape)
assert M.device_status() == 0
n = M.workspace_bytes(layer.shape)
for where in (n - 4, n - 256):          # last and first guard byte block of the last region
    saved = layer.ws[where].item()
    layer.ws[where] = saved ^ 0x5A
    M.debug_check_workspace(layer.ws, layer.shape)
    assert M.device_status() == M.ERR_CORRUPT
    assert M.device_status() == 0       # read and cleared
    layer.ws[where] = saved
    M.debug_check_workspace(layer.ws, layer.shape)
    assert M.device_status() == 0
# the grouping call re-arms the guard words and checks them itself
layer.ws[n - 4] = 0
layer.group()
assert M.device_status() == 0
# the allocation-free grouping under the debug build: its built-in buffer ends where the grouping's
# regions end, so only their guard words exist; same segments as the call with a workspace
w = W.scaled(W.CONFIGS[2], B=100, C=512, k=6, unique_len=16)
sh = W.make_shared_store(w, "cuda")
q = W.make_queries(w, sh, 0, "cuda")
layer = MoskaLayer(w.B, w.Hq, w.Hkv, w.D, w.C, w.L, w.k, 16)
layer.build_summaries(sh.k_shared)
layer.route(q)
layer.group()
off = torch.full_like(layer.seg_offsets, -1)
ent = torch.full_like(layer.seg_entries, -1)
for _ in range(2):
    M.group_by_chunk_noalloc(layer.topk_idx, off, ent, layer.shape)
    torch.cuda.synchronize()
    assert torch.equal(off, layer.seg_offsets) and torch.equal(ent, layer.seg_entries)
    assert M.device_status() == 0
print("debug build: guard words ok")
