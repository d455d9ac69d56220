"""Multi-GPU launch of the path: every (sequence, KV head) is independent, so ranks take independent shards
and no collective touches the data path.  `torch.distributed` is used only to line the ranks up around the
timed region and to combine their timings."""
from __future__ import annotations

import copy

import torch


def shard_spec(spec, rank: int, world: int):
    """Workload of one rank under weak scaling: same shape, its own seed (rank 0 of a single-rank job keeps
    the unsharded seed so that N = 1 reproduces the plain benchmark)."""
    out = copy.deepcopy(spec)
    if world > 1:
        out.config_id = spec.config_id * 10 + rank
    return out


def barrier(dist, device_sync=None):
    if dist is not None and dist.is_initialized():
        dist.barrier()
    if device_sync is not None:
        device_sync()


def aggregate(dist, ms_local: float, units_local: float, device="cpu"):
    """Whole-job throughput: units processed by all ranks / the slowest rank's time.
    Returns (value in units per second, max ms over ranks, total units)."""
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
    ms = float(t.item())
    units = float(u.item())
    return units / (ms * 1e-3), ms, units
