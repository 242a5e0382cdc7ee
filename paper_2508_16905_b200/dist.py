"""Multi-process plumbing (one process per GPU).

Two ways to use several GPUs.  Replicas: N GPUs run N independent copies of the pass (the benchmark's --gpus N); the
only exchange is bookkeeping, a barrier around the timed region and the max / sum of per-rank measurements.  Shards:
one model spread over the ranks by flat ranges; per step the ranks exchange one small record per layer (all-gather,
rank order) between the statistics and the update, see sharded_step.  Works on any torch.distributed backend (nccl on
GPUs, gloo in CPU tests).
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


def shard_ranges(n_total, world):
    """Cuts [0, n_total) into `world` ranges on multiples of 128 elements, as equal as that allows (the last one takes
    the rest, rounded up to the row grid the library cuts on)."""
    rows = -(-int(n_total) // 128)
    cuts = [min(rows, -(-rows * r // world)) * 128 for r in range(world + 1)]
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def gather_records(local, world=None, group=None):
    """All ranks' per-layer records in rank order: `local` is this rank's uint8 tensor of L * 40 bytes; returns a
    tensor of world * L * 40 bytes, identical on every rank.  Without a process group: the local records."""
    if not (dist.is_available() and dist.is_initialized()):
        return local.clone()
    world = world or dist.get_world_size(group)
    out = torch.empty(world * local.numel(), dtype=local.dtype, device=local.device)
    dist.all_gather_into_tensor(out, local.contiguous(), group=group)
    return out


def sharded_step(ta, h, w_local, g_local, hz_local, c_local, probe_seed, step, records=None, group=None):
    """One optimizer pass of a model spread over the ranks of `group`: local statistics, one all-gather of the
    per-layer records (40 bytes per layer and rank), decisions and local update.  `ta` is the binding module."""
    if records is None:
        records = torch.empty(h.L * ta.RECORD_BYTES, dtype=torch.uint8, device=w_local.device)
    ta.ta_shard_sweep(h, g_local, hz_local, probe_seed, step, records)
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    everyone = gather_records(records, world, group)
    ta.ta_shard_apply(h, w_local, g_local, c_local, everyone, world)
    return everyone
