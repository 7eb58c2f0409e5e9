"""Multi-GPU form of the path: problems are independent, so they are partitioned across ranks
(one process per GPU) with no data-path collective; the only exchange is an all-gather of the
[P/world, k] result blocks at the end, and a MAX reduction for timing. The catalogue and the
model are replicated on every rank. For the single-problem call the split is by candidates
instead: every rank ranks its share of the pool, the world x k (index, score) pairs are
gathered and merged k ways (one exchange step). Works with any torch.distributed backend (NCCL
on GPUs, gloo on CPU for the tests). No peer loads, no multicast."""
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


def select_one_sharded(select_fn, merge_fn, C: int, k: int, device, group=None):
    """Candidate split of the single-problem call. `select_fn(lo, hi) -> (idx, score)` ranks the
    candidates [lo, hi) of the pool on this rank and returns its top-k ([k] tensors, POOL indices,
    -1 / -inf padding); the world x k pairs are all-gathered and `merge_fn(idx [1, world*k],
    score [1, world*k], k) -> ([1, k], [1, k])` (ks_merge_topk on a GPU) picks the k best by
    (score descending, index ascending). Every rank returns the global result."""
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    lo, hi = my_slice(C, rank, world)
    if hi > lo:
        idx, sc = select_fn(lo, hi)
        idx, sc = idx.reshape(-1)[:k].to(device), sc.reshape(-1)[:k].to(device)
    else:
        idx = torch.full((k,), -1, dtype=torch.int32, device=device)
        sc = torch.full((k,), float("-inf"), dtype=torch.float32, device=device)
    all_i = [torch.empty_like(idx) for _ in range(world)]
    all_s = [torch.empty_like(sc) for _ in range(world)]
    dist.all_gather(all_i, idx.contiguous(), group=group)
    dist.all_gather(all_s, sc.contiguous(), group=group)
    out_i, out_s = merge_fn(torch.cat(all_i).reshape(1, -1), torch.cat(all_s).reshape(1, -1), k)
    return out_i.reshape(-1), out_s.reshape(-1)
