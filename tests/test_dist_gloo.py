"""world_size-2 gloo test of the multi-GPU host logic (replicas only: barrier + max over ranks)."""
import os
import socket

import torch.multiprocessing as mp


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import torch.distributed as dist
    from paper_2506_13472_b200.dist import aggregate_throughput, init_from_env, max_over_ranks
    r, w, _ = init_from_env("gloo")
    assert (r, w) == (rank, world)
    dist.barrier()
    ms = 10.0 * (rank + 1)                       # rank 1 is the slow one
    out[rank] = (max_over_ranks(ms), aggregate_throughput(1000.0, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_two_ranks():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    for rank in (0, 1):
        mx, thr = out[rank]
        assert mx == 20.0
        assert abs(thr - 2 * 1000.0 / 0.020) < 1e-6
