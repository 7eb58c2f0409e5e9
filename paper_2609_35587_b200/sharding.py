"""Multi-GPU form of the path: problems are independent, so they are partitioned across ranks
(one process per GPU) with no data-path collective; the only exchange is an all-gather of the
[P/world, k] result blocks at the end, and a MAX reduction for timing. The catalogue and the
model are replicated on every rank. Works with any torch.distributed backend (NCCL on GPUs,
gloo on CPU for the tests)."""
from __future__ import annotations

import numpy as np
import torch
import torch.distributed as dist


def partition(P: int, world: int) -> list[tuple[int, int]]:
    """Contiguous blocks of problems, sizes differing by at most one."""
    base, extra = divmod(P, world)
    out, lo = [], 0
    for r in range(world):
        hi = lo + base + (1 if r < extra else 0)
        out.append((lo, hi))
        lo = hi
    return out


def my_slice(P: int, rank: int, world: int) -> tuple[int, int]:
    return partition(P, world)[rank]


def all_gather_topk(idx: torch.Tensor, score: torch.Tensor, P: int, k: int, group=None):
    """Assemble the global [P, k] results from every rank's block (blocks may differ in size by
    one row, so each is padded to the largest before the collective)."""
    world = dist.get_world_size(group)
    parts = partition(P, world)
    rows = max(hi - lo for lo, hi in parts)
    pad_i = torch.full((rows, k), -1, dtype=torch.int32, device=idx.device)
    pad_s = torch.full((rows, k), float("-inf"), dtype=torch.float32, device=idx.device)
    pad_i[:idx.shape[0]] = idx
    pad_s[:score.shape[0]] = score
    all_i = [torch.empty_like(pad_i) for _ in range(world)]
    all_s = [torch.empty_like(pad_s) for _ in range(world)]
    dist.all_gather(all_i, pad_i, group=group)
    dist.all_gather(all_s, pad_s, group=group)
    out_i = torch.cat([all_i[r][:hi - lo] for r, (lo, hi) in enumerate(parts)])
    out_s = torch.cat([all_s[r][:hi - lo] for r, (lo, hi) in enumerate(parts)])
    return out_i, out_s


def max_over_ranks(value: float, device, group=None) -> float:
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def select_sharded(select_fn, problems: np.ndarray, k: int, device, group=None):
    """Rank this process's block of problems with `select_fn(problem_block) -> (idx, score)`
    (device tensors [rows, k]) and return the gathered global result on every rank."""
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    lo, hi = my_slice(len(problems), rank, world)
    if hi > lo:
        idx, sc = select_fn(problems[lo:hi])
    else:
        idx = torch.empty((0, k), dtype=torch.int32, device=device)
        sc = torch.empty((0, k), dtype=torch.float32, device=device)
    return all_gather_topk(idx, sc, len(problems), k, group)
