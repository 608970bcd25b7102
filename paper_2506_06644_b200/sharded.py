"""Statistical top-k of rows sharded over the ranks of a process group (the paper's appendix on
distributed training: "global" and "local" statistical top-k).

Global form: every rank takes the moments of its part of each row, the parts' moments are
all-gathered (24 bytes per row and rank), every rank merges them into the threshold of the whole
row and selects from its own part with it -- the same active set as the unsharded operator.
Local form: no exchange, every rank runs the operator on its part with k / world_size.

`torch.distributed` is the plumbing (the all-gather); the arithmetic is passed in as three callables
so that the GPU path uses the library's kernels (`gpu_steps`) and the host logic can be exercised
on CPU ranks with any other implementation of the same three steps."""
from __future__ import annotations

from typing import Callable, NamedTuple

import torch
import torch.distributed as dist


class Steps(NamedTuple):
    moments: Callable        # (x_local [rows, n_local]) -> float64 [rows, 3] = (n, mean, M2)
    merge: Callable          # (parts float64 [world, rows, 3], k, n_total) -> float32 [rows] theta
    select: Callable         # (x_local, theta [rows]) -> whatever the caller wants back


def gather_parts(local: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather the ranks' [rows, 3] moments into [world, rows, 3], part r from rank r."""
    world = dist.get_world_size(group)
    out = torch.empty((world,) + tuple(local.shape), dtype=local.dtype, device=local.device)
    dist.all_gather(list(out.unbind(0)), local.contiguous(), group=group)      # views of one buffer: part r lands in out[r]
    return out


def global_stat_topk(x_local: torch.Tensor, k: int, n_total: int, steps: Steps, group=None):
    """Global statistical top-k: returns (theta [rows], select(x_local, theta))."""
    local = steps.moments(x_local)
    parts = gather_parts(local, group)
    counted = int(parts[:, 0, 0].sum().item()) if parts.shape[1] > 0 else n_total
    if counted != n_total:
        raise ValueError(f"the parts hold {counted} values per row, not n_total = {n_total}")
    theta = steps.merge(parts, k, n_total)
    return theta, steps.select(x_local, theta)


def local_k(k: int, world: int) -> int:
    """k' = k / m of the local form (at least one)."""
    return max(1, k // world)


def gpu_steps(ctx, fill: int, idx_cap: int) -> Steps:
    """The three steps on the library's kernels; select returns (count, idx, val) with idx local to the part."""
    from . import binding as S

    def moments(x):
        rows, n = x.shape
        out = torch.empty(rows, 3, dtype=torch.float64, device=x.device)
        S.spark_stat_moments(ctx, x, rows, n, x.stride(0), out)
        return out

    def merge(parts, k, n_total):
        world, rows, _ = parts.shape
        theta = torch.empty(rows, dtype=torch.float32, device=parts.device)
        S.spark_stat_merge(ctx, parts, world, rows, k, n_total, theta, None)
        return theta

    def select(x, theta):
        rows, n = x.shape
        count = torch.empty(rows, dtype=torch.int32, device=x.device)
        idx = torch.empty(rows, idx_cap, dtype=torch.int32, device=x.device)
        val = torch.empty(rows, idx_cap, dtype=torch.float32, device=x.device)
        S.spark_stat_select(ctx, x, rows, n, x.stride(0), theta, fill, count, idx, val, idx_cap, None)
        return count, idx, val

    return Steps(moments, merge, select)
