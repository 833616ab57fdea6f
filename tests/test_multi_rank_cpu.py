"""The N > 1 path on CPU: two gloo ranks shard a batch, decode their share (the oracle stands in for
the GPU decoder: the host logic is what is under test), gather, and must reproduce the single-process
result; timings reduce with MAX and counters with SUM."""
from __future__ import annotations

import os
import sys

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _decode_share(prompts, G, s):
    from oracle import l2pd_oracle as orc
    from paper_2509_25188_b200 import workloads as wl
    from tests.helpers import oracle_model, small_shape
    shape = small_shape()
    w = wl.make_weights(shape, seed=3, final_norm_gain=wl.spread_gain(shape), threads=1)
    m = oracle_model(shape, w, lm_head_bias=wl.make_eot_bias(shape, 3.0))
    filt = wl.make_filter(s, seed=1)
    res = orc.decode_batch(m, filt, prompts, G, orc.DecodeConfig(block_len=s), keep_trace=False)
    toks = np.stack([r.response for r in res]) if res else np.zeros((0, G), np.int64)
    return toks, np.array([r.out_len for r in res]), np.array([r.steps for r in res])


def _worker(rank, world, port, B, P, G, s, q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2509_25188_b200 import replicas, workloads as wl
    from tests.helpers import small_shape
    prompts = wl.make_prompts(B, P, small_shape(), seed=7)
    mine = replicas.shard_prompts(prompts, world, rank)
    toks, out_len, steps = _decode_share(mine, G, s)
    all_toks, all_len, all_steps = replicas.gather_decodes(toks, out_len, steps, B, G)
    ms, (tok_sum,) = replicas.reduce_timing(10.0 + rank, [float(out_len.sum())])
    if rank == 0:
        q.put((all_toks, all_len, all_steps, ms, tok_sum))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_process_batch():
    sys.path.insert(0, ROOT)
    from paper_2509_25188_b200 import replicas, workloads as wl
    from tests.helpers import small_shape
    B, P, G, s = 5, 6, 16, 4          # odd batch: ranks get 3 and 2 sequences
    assert replicas.shard_range(5, 2, 0) == (0, 3) and replicas.shard_range(5, 2, 1) == (3, 5)
    assert replicas.shard_range(2, 4, 3) == (2, 2)                       # more ranks than items
    covered = sorted(i for r in range(3) for i in range(*replicas.shard_range(7, 3, r)))
    assert covered == list(range(7))
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, B, P, G, s, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = q.get(timeout=300)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    toks, out_len, steps = _decode_share(wl.make_prompts(B, P, small_shape(), seed=7), G, s)
    assert np.array_equal(got[0], toks) and np.array_equal(got[1], out_len) and np.array_equal(got[2], steps)
    assert got[3] == 11.0                      # MAX over ranks
    assert got[4] == float(out_len.sum())      # SUM over ranks


def test_spawned_ranks_pull_chunks_from_the_queue_and_gather(tmp_path):
    """The path bench.py --gpus N takes when no launcher started it: replicas.spawn_local_ranks starts the ranks
    (here two gloo ranks on CPU), the ranks take chunks of the batch from the shared queue until none is left
    (over-decomposition: rank 0 is slowed down, so rank 1 ends up with more of them), and the gathered result
    equals the single-process decode of the whole batch."""
    sys.path.insert(0, ROOT)
    from paper_2509_25188_b200 import replicas, workloads as wl
    from tests.helpers import small_shape
    B, P, G, s, chunk = 7, 6, 16, 4, 2         # four chunks (2, 2, 2, 1 sequences) for two ranks
    out = str(tmp_path / "gathered.npz")
    rc = replicas.spawn_local_ranks(2, os.path.join(ROOT, "tests", "multi_rank_worker.py"),
                                    [out, str(B), str(P), str(G), str(s), str(chunk)],
                                    extra_env={"OMP_NUM_THREADS": "2"}, timeout=600)
    assert rc == 0
    got = np.load(out)
    toks, out_len, steps = _decode_share(wl.make_prompts(B, P, small_shape(), seed=7), G, s)
    assert np.array_equal(got["toks"], toks) and np.array_equal(got["out_len"], out_len) and np.array_equal(got["steps"], steps)
    assert int(got["world"]) == 2 and float(got["decoded"]) == B and float(got["ms"]) == 11.0
    assert 0 < int(got["mine"]) < B            # both ranks took part
