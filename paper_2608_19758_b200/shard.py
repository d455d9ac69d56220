"""Multi-GPU launch of the path: every (sequence, KV head) is independent, so ranks take independent shards
-- whole workloads of their own (weak scaling) or the KV heads of one workload (strong scaling) -- and no
collective touches the data path.  `torch.distributed` is used only to line the ranks up around the
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


def shard_spec_by_heads(spec, rank: int, world: int):
    """Workload of one rank when ONE workload is split over the ranks by KV head (strong scaling; the paper serves
    with tensor parallelism over heads, Sec. 4.1): rank r holds KV heads [r Hkv / N, (r + 1) Hkv / N) with their g
    query heads each, i.e. that head slice of q / out and of the K / V cache.  The page table, the lengths and
    every per-head quantity (seeds, FP8 scales) are those of the unsplit workload, so the rank's tensors are
    exactly the head slices of the whole (`slice_case_heads`), and its output is that slice of the whole output:
    block lists are per KV head and no step of the path looks across heads, so there is no exchange step."""
    if spec.num_kv_heads % world != 0:
        raise ValueError(f"{spec.num_kv_heads} KV heads do not split over {world} ranks")
    out = copy.deepcopy(spec)
    per = spec.num_kv_heads // world
    out.num_kv_heads = per
    out.num_q_heads = per * spec.group
    out.kv_head_offset = spec.kv_head_offset + rank * per
    return out


def slice_case_heads(case, h0: int, h1: int):
    """The KV heads [h0, h1) of a workload as a workload of its own: contiguous head slices of q, K / V cache
    and scales; page table and lengths unchanged."""
    g = case.spec.group
    spec = copy.deepcopy(case.spec)
    spec.num_kv_heads = h1 - h0
    spec.num_q_heads = (h1 - h0) * g
    spec.kv_head_offset = case.spec.kv_head_offset + h0
    cut = lambda t, a, b: None if t is None else t[a:b].contiguous()
    return type(case)(spec=spec, q=case.q[:, h0 * g:h1 * g].contiguous(),
                      k_cache=case.k_cache[:, :, h0:h1].contiguous(), v_cache=case.v_cache[:, :, h0:h1].contiguous(),
                      page_table=case.page_table, cu_seqlens_q=case.cu_seqlens_q, seqlens_k=case.seqlens_k,
                      q_scale=cut(case.q_scale, h0 * g, h1 * g), k_scale=cut(case.k_scale, h0, h1),
                      v_scale=cut(case.v_scale, h0, h1))


def gather_heads(dist, local: torch.Tensor, head_dim: int = 1):
    """Concatenates the ranks' head slices along `head_dim` (a check / result-collection helper: the path itself
    needs no collective)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local
    parts = [torch.empty_like(local) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, local.contiguous())
    return torch.cat(parts, dim=head_dim)


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
