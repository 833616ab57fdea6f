"""Worker of tests/test_multi_rank_cpu.py: started by replicas.spawn_local_ranks as one gloo rank.
Pulls chunks of a batch from the shared queue, decodes them (the oracle stands in for the GPU decoder: the host
logic is what is under test), gathers, and rank 0 writes the result to the file named on the command line."""
import os
import sys
import time

import numpy as np
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def main():
    out_path, B, P, G, s, chunk = sys.argv[1], *map(int, sys.argv[2:7])
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    from paper_2509_25188_b200 import replicas, workloads as wl
    from tests.helpers import small_shape
    from tests.test_multi_rank_cpu import _decode_share
    prompts = wl.make_prompts(B, P, small_shape(), seed=7)
    n_chunks = -(-B // chunk)
    store = dist.distributed_c10d._get_default_store()
    idx, toks, lens, steps = [], [], [], []
    for c in replicas.claim_chunks(store, n_chunks):
        lo, hi = c * chunk, min(B, (c + 1) * chunk)
        t, l, st = _decode_share(prompts[lo:hi], G, s)
        idx += list(range(lo, hi)); toks.append(t); lens.append(l); steps.append(st)
        if rank == 0:
            time.sleep(0.3)        # a slow rank: the other one takes more chunks
    toks = np.concatenate(toks) if toks else np.zeros((0, G), np.int64)
    lens = np.concatenate(lens) if lens else np.zeros(0, np.int64)
    steps = np.concatenate(steps) if steps else np.zeros(0, np.int64)
    all_toks, all_len, all_steps = replicas.gather_indexed(idx, toks, lens, steps, B, G)
    ms, (n_mine,) = replicas.reduce_timing(10.0 + rank, [float(len(idx))])
    if rank == 0:
        np.savez(out_path, toks=all_toks, out_len=all_len, steps=all_steps, ms=ms, decoded=n_mine, world=world,
                 mine=len(idx))
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
