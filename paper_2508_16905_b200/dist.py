"""Multi-process plumbing for replicated runs (one process per GPU, no data-path collective).

The optimizer pass of one model does not shard in this library: N GPUs run N independent replicas.
The only exchange is bookkeeping: a barrier around the timed region and the max / sum of per-rank
measurements.  Works on any torch.distributed backend (nccl on GPUs, gloo in CPU tests).
"""
import os

import torch
import torch.distributed as dist


def env_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend=None):
    """Initialises the default process group from the torchrun environment when WORLD_SIZE > 1."""
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        dist.init_process_group(backend=backend or ("nccl" if torch.cuda.is_available() else "gloo"),
                                rank=rank, world_size=world)
    return rank, local_rank, world


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate(ms_local: float, units_local: float, device="cpu"):
    """Whole-job numbers of a replicated run: (max over ranks of the elapsed ms, sum over ranks of the
    units processed).  Throughput of the job = units / (ms / 1e3)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(ms_local), float(units_local)
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units_local)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def shutdown():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
