"""One process per GPU: rendezvous from the torchrun environment, barrier and
max-over-ranks timing.  The training path itself has no collective: every rank
trains an independent replica of the workload."""
from __future__ import annotations

import datetime
import os

_state = {"on": False}


def init_from_env(backend: str):
    """Returns (rank, world_size, local_rank); a no-op outside torchrun."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world,
                                timeout=datetime.timedelta(minutes=30))
        _state["on"] = True
    return rank, world, local


def barrier():
    if _state["on"]:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(value: float) -> float:
    """The slowest rank's time: what a whole-job rate must be divided by."""
    if not _state["on"]:
        return float(value)
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def finish():
    if _state["on"]:
        import torch.distributed as dist
        dist.destroy_process_group()
        _state["on"] = False
