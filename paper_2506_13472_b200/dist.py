"""Multi-GPU plumbing.  The path shards by replication only (independent replica per GPU, no
data-path collective); torch.distributed is used for the rendezvous, the barrier and the
max-over-ranks reduction of the measured time."""
import os

import torch
import torch.distributed as dist


def init_from_env(backend):
    """(rank, world_size, local_rank); initialises the process group when WORLD_SIZE > 1."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world, local


def max_over_ranks(value):
    """Largest `value` (a float, e.g. milliseconds) over all ranks; identity without a process group."""
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank, ms):
    """Whole-job throughput: units all ranks processed / the slowest rank's time (units per second)."""
    world = dist.get_world_size() if dist.is_initialized() else 1
    return world * units_per_rank / (max_over_ranks(ms) * 1e-3)
