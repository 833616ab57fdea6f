"""Host-side logic for running the decode on several GPUs of one node.

Sequences are independent units of the method (each prompt is decoded on its own), so the batch is
split across ranks, every rank holds the full weights and runs its own steps, and no collective is
needed inside a step.  The only exchanges are at the end: responses and per-sequence counters are
gathered, and timings are reduced with MAX so that a reported time is the slowest rank's.
Works with any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import Iterator, List, Optional, Sequence, Tuple

import numpy as np
import torch
import torch.distributed as dist


def launcher_env_present() -> bool:
    """True inside a process that a launcher (torchrun) started: RANK and WORLD_SIZE are set."""
    return "RANK" in os.environ and "WORLD_SIZE" in os.environ


def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def spawn_local_ranks(n_ranks: int, script: str, argv: Sequence[str], extra_env: Optional[dict] = None,
                      timeout: Optional[float] = None) -> int:
    """Starts `script argv...` as n_ranks processes of one node (one per GPU), the way the launcher would:
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N --master-addr 127.0.0.1 --master-port P script argv...
    Each process finds RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* in its environment.  Returns the exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n_ranks),
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), script] + list(argv)
    env = dict(os.environ)
    env.update(extra_env or {})
    return subprocess.run(cmd, env=env, timeout=timeout).returncode


def claim_chunks(store, n_chunks: int, key: str = "l2pd_next_chunk") -> Iterator[int]:
    """Over-decomposition: the batch is cut into more chunks than ranks, and a rank that has finished its chunk
    takes the next unclaimed one (sequences finish after different numbers of steps once EoTP cuts them, so a
    fixed split leaves ranks idle).  `store` is the process group's key-value store; add() is atomic, so every
    chunk index in [0, n_chunks) is yielded to exactly one rank."""
    while True:
        i = int(store.add(key, 1)) - 1
        if i >= n_chunks:
            return
        yield i


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


def gather_indexed(indices: Sequence[int], tokens: np.ndarray, out_len: np.ndarray, steps: np.ndarray, n_total: int,
                   gen_len: int, device="cpu"):
    """The same for sequences that were handed out dynamically: each rank contributes (sequence index, response,
    out_len, steps) rows for the sequences it decoded; every rank gets the whole batch in prompt order.
    Every index in [0, n_total) must have been decoded by exactly one rank."""
    world = dist.get_world_size()
    n_mine = torch.tensor([len(indices)], dtype=torch.int64, device=device)
    counts = [torch.zeros_like(n_mine) for _ in range(world)]
    dist.all_gather(counts, n_mine)
    cap = max(1, max(int(c[0]) for c in counts))
    buf = torch.full((cap, gen_len + 3), -1, dtype=torch.int64, device=device)
    n = len(indices)
    if n:
        buf[:n, 0] = torch.as_tensor(np.asarray(indices), dtype=torch.int64, device=device)
        buf[:n, 1: gen_len + 1] = torch.as_tensor(np.asarray(tokens), dtype=torch.int64, device=device)
        buf[:n, gen_len + 1] = torch.as_tensor(np.asarray(out_len), dtype=torch.int64, device=device)
        buf[:n, gen_len + 2] = torch.as_tensor(np.asarray(steps), dtype=torch.int64, device=device)
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf)
    toks = np.full((n_total, gen_len), -1, np.int32)
    lens = np.full(n_total, -1, np.int32)
    stp = np.full(n_total, -1, np.int32)
    seen = 0
    for part, c in zip(parts, counts):
        rows = part[: int(c[0])].cpu().numpy()
        for row in rows:
            i = int(row[0])
            if not (0 <= i < n_total) or lens[i] != -1:
                raise ValueError("sequence %d decoded twice or out of range" % i)
            toks[i], lens[i], stp[i] = row[1: gen_len + 1], row[gen_len + 1], row[gen_len + 2]
            seen += 1
    if seen != n_total:
        raise ValueError("%d of %d sequences were decoded" % (seen, n_total))
    return toks, lens, stp


def reduce_timing(ms: float, counters: Sequence[float], device="cpu") -> Tuple[float, List[float]]:
    """(max over ranks of ms, sum over ranks of each counter)."""
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor(list(counters), dtype=torch.float64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return float(t[0]), [float(v) for v in c]
