"""Host-side logic for running the decode on several GPUs of one node.

Sequences are independent units of the method (each prompt is decoded on its own), so the batch is
split across ranks, every rank holds the full weights and runs its own steps, and no collective is
needed inside a step.  The only exchanges are at the end: responses and per-sequence counters are
gathered, and timings are reduced with MAX so that a reported time is the slowest rank's.
Works with any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np
import torch
import torch.distributed as dist


def shard_range(n_items: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous [begin, end) of rank's share; the first n_items % world ranks get one more."""
    base, extra = divmod(n_items, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def shard_prompts(prompts: np.ndarray, world: int, rank: int) -> np.ndarray:
    b, e = shard_range(len(prompts), world, rank)
    return prompts[b:e]


def gather_decodes(tokens: np.ndarray, out_len: np.ndarray, steps: np.ndarray, n_total: int, gen_len: int,
                   device="cpu"):
    """All ranks get the whole batch's responses [n_total, G], out_len and steps, in prompt order."""
    world, rank = dist.get_world_size(), dist.get_rank()
    cap = -(-n_total // world)
    buf = torch.full((cap, gen_len + 2), -1, dtype=torch.int64, device=device)
    n = len(tokens)
    if n:
        buf[:n, :gen_len] = torch.as_tensor(np.asarray(tokens), dtype=torch.int64, device=device)
        buf[:n, gen_len] = torch.as_tensor(np.asarray(out_len), dtype=torch.int64, device=device)
        buf[:n, gen_len + 1] = torch.as_tensor(np.asarray(steps), dtype=torch.int64, device=device)
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf)
    rows = []
    for r, part in enumerate(parts):
        b, e = shard_range(n_total, world, r)
        rows.append(part[: e - b].cpu().numpy())
    allr = np.concatenate(rows, axis=0)
    return allr[:, :gen_len].astype(np.int32), allr[:, gen_len].astype(np.int32), allr[:, gen_len + 1].astype(np.int32)


def reduce_timing(ms: float, counters: Sequence[float], device="cpu") -> Tuple[float, List[float]]:
    """(max over ranks of ms, sum over ranks of each counter)."""
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor(list(counters), dtype=torch.float64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return float(t[0]), [float(v) for v in c]
