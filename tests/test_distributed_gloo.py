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
