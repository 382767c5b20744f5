"""World-size-2 gloo test of the benchmark's multi-process plumbing (CPU only)."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2511_06010_b200 import distributed as DD

    r, lr, w = DD.init("gloo")
    assert (r, lr, w) == (rank, rank, world)
    DD.barrier()
    # rank 0 is "slower": the whole-job value must use the max time and the summed units
    ms = 10.0 if rank == 0 else 4.0
    value, ms_max = DD.whole_job_throughput(64 * 5, ms)
    out[rank] = (value, ms_max, DD.kv_head_shard(8, rank, world))
    DD.finalize()


def test_two_ranks_max_time_sum_units():
    world, port = 2, _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        value, ms_max, shard = out[rank]
        assert ms_max == 10.0
        assert abs(value - (2 * 64 * 5) / 10e-3) < 1e-6
    assert out[0][2] == (0, 4) and out[1][2] == (4, 8)


def test_kv_head_shard_covers_heads_once():
    from paper_2511_06010_b200 import distributed as DD

    for Hkv in (1, 3, 8):
        for world in (1, 2, 3, 8):
            seen = []
            for rank in range(world):
                h0, h1 = DD.kv_head_shard(Hkv, rank, world)
                seen.extend(range(h0, h1))
            assert seen == list(range(Hkv))


def _disagg_worker(rank, world, port, out):
    """1 shared rank + 2 unique ranks exchanging CPU tensors: queries up, shared partials back."""
    import torch

    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2511_06010_b200 import distributed as DD
    from paper_2511_06010_b200 import disaggregated as DG

    DD.init("gloo")
    B, Hq, D = 7, 4, 8                      # 7 requests over 2 unique ranks: blocks of 4 and 3
    blocks = DG.request_blocks(B, [1, 2])
    g = torch.Generator().manual_seed(5)
    q_true = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)   # every rank can rebuild it
    if rank == 0:
        q_all = torch.zeros(B, Hq, D, dtype=torch.bfloat16)
        DG.gather_queries(q_all, blocks)
        assert torch.equal(q_all, q_true)
        # a stand-in for the shared result: any function of the row, so that misrouted rows show
        o = q_all.float() * 2.0 + 1.0
        lse = q_all.float().sum(-1)
        DG.return_shared_partials(o, lse, blocks)
        out[rank] = "ok"
    else:
        _, b0, b1 = [b for b in blocks if b[0] == rank][0]
        send = DG.send_queries(q_true[b0:b1].contiguous(), 0)
        o_in = torch.empty(b1 - b0, Hq, D)
        lse_in = torch.empty(b1 - b0, Hq)
        DG.receive_shared_partial(o_in, lse_in, 0)
        send.wait()
        assert torch.equal(o_in, q_true[b0:b1].float() * 2.0 + 1.0)
        assert torch.equal(lse_in, q_true[b0:b1].float().sum(-1))
        out[rank] = (b0, b1)
    DD.finalize()


def test_disaggregated_exchange_three_ranks():
    world, port = 3, _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_disagg_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == "ok" and out[1] == (0, 4) and out[2] == (4, 7)


def test_request_blocks_cover_requests_once():
    from paper_2511_06010_b200 import disaggregated as DG

    for n in (0, 1, 5, 64):
        for ranks in ([1], [1, 2], [3, 1, 2]):
            seen = []
            for r, b0, b1 in DG.request_blocks(n, ranks):
                seen.extend(range(b0, b1))
            assert seen == list(range(n))


def test_kv_head_shard_of_a_workload_keeps_the_request_structure():
    """A rank's share of one batch split by KV head: same requests (lengths, query targets),
    Hkv / N heads with their G query heads, its own values; uneven splits are refused."""
    import numpy as np
    import pytest

    from paper_2511_06010_b200 import workloads as W

    w = W.CONFIGS[4]
    for world in (2, 4, 8):
        for rank in range(world):
            ws = W.kv_head_shard(w, rank, world)
            assert ws.Hkv * world == w.Hkv and ws.Hq * world == w.Hq and ws.G == w.G
            assert (ws.B, ws.C, ws.L, ws.k, ws.steps) == (w.B, w.C, w.L, w.k, w.steps)
            assert np.array_equal(W.unique_lengths(ws), W.unique_lengths(w))
            assert np.array_equal(W.query_targets(ws, 3), W.query_targets(w, 3))
    small = W.scaled(W.CONFIGS[1], B=2, C=2, L=128, unique_len=4)
    a = W.make_shared_store(W.kv_head_shard(small, 0, 2)).k_shared
    b = W.make_shared_store(W.kv_head_shard(small, 1, 2)).k_shared
    assert a.shape == b.shape and not (a == b).all()
    with pytest.raises(ValueError):
        W.kv_head_shard(w, 0, 3)


def test_slice_kv_heads_is_plain_indexing():
    import torch

    from paper_2511_06010_b200 import distributed as DD

    B, Hq, Hkv, D, C, L, T = 3, 8, 4, 4, 2, 2, 5
    G = Hq // Hkv
    q = torch.arange(B * Hq * D).reshape(B, Hq, D)
    ks = torch.arange(Hkv * C * L * D).reshape(Hkv, C, L, D)
    ku = torch.arange(T * Hkv * D).reshape(T, Hkv, D)
    parts = [DD.slice_kv_heads(*DD.kv_head_shard(Hkv, r, 2), G, q, ks, ks + 1, ku, ku + 1) for r in range(2)]
    assert all(t.is_contiguous() for p in parts for t in p)
    assert torch.equal(torch.cat([p[0] for p in parts], dim=1), q)
    assert torch.equal(torch.cat([p[1] for p in parts], dim=0), ks)
    assert torch.equal(torch.cat([p[2] for p in parts], dim=0), ks + 1)
    assert torch.equal(torch.cat([p[3] for p in parts], dim=1), ku)
    assert torch.equal(torch.cat([p[4] for p in parts], dim=1), ku + 1)


class _FakeShared:
    """Stands in for the Shared-KV role: its 'shared result' is a fixed function of the query
    row, so a row delivered to the wrong owner or in the wrong order shows."""
    is_shared_rank = True

    def compute(self, q_all):
        return q_all.float() * 2.0 + 1.0, q_all.float().sum(-1)


class _FakeUnique:
    is_shared_rank = False

    def __init__(self, n, Hq, D):
        import torch

        self.o_in = torch.empty(n, Hq, D)
        self.lse_in = torch.empty(n, Hq)
        self.started = None

    def start(self, q_local, kv_len):
        self.started = (q_local.clone(), kv_len.clone())

    def finish(self):
        return self.o_in + self.lse_in[..., None]


def _disagg_step_worker(rank, world, port, out):
    """disaggregated.step() itself, three steps in a row, roles replaced by CPU stand-ins."""
    import torch

    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2511_06010_b200 import distributed as DD
    from paper_2511_06010_b200 import disaggregated as DG

    DD.init("gloo")
    B, Hq, D = 9, 4, 8
    blocks = DG.request_blocks(B, [1, 2, 3])
    results = []
    for step in range(3):
        g = torch.Generator().manual_seed(100 + step)
        q_true = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
        if rank == 0:
            q_all = torch.zeros(B, Hq, D, dtype=torch.bfloat16)
            assert DG.step(_FakeShared(), None, None, 0, blocks, q_all=q_all) is None
            assert torch.equal(q_all, q_true)
        else:
            _, b0, b1 = [b for b in blocks if b[0] == rank][0]
            role = _FakeUnique(b1 - b0, Hq, D)
            kv_len = torch.arange(b0, b1, dtype=torch.int32)
            got = DG.step(role, q_true[b0:b1].contiguous(), kv_len, 0, blocks)
            qf = q_true[b0:b1].float()
            assert torch.equal(got, qf * 2.0 + 1.0 + qf.sum(-1)[..., None])
            assert torch.equal(role.started[0], q_true[b0:b1]) and torch.equal(role.started[1], kv_len)
            results.append((b0, b1))
    out[rank] = results if rank else "ok"
    DD.finalize()


def test_disaggregated_step_function_four_ranks():
    world, port = 4, _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_disagg_step_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == "ok"
    assert out[1] == [(0, 3)] * 3 and out[2] == [(3, 6)] * 3 and out[3] == [(6, 9)] * 3
