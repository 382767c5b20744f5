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
