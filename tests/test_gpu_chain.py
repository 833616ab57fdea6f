"""The chained launch (output projection, RMSNorm, gate/up, down, next RMSNorm and QKV of a layer in one
persistent kernel) against the one-launch-per-projection form of the same step: both run the same tiles,
epilogues, K-slice partial sums and summation orders, so every output must agree bit for bit.  The
unchained form is the one the kernel-level and lockstep tests pin to the oracle.
"""
from __future__ import annotations

import os

import numpy as np
import pytest

from paper_2509_25188_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _device_weights(shape, seed=0):
    from paper_2509_25188_b200 import binding
    w = wl.make_weights(shape, seed=seed, final_norm_gain=wl.spread_gain(shape), threads=os.cpu_count() or 8)
    return {"tok_emb": binding.to_device(w["tok_emb"]), "lm_head": binding.to_device(w["lm_head"]),
            "final_norm": w["final_norm"],
            "layers": [{k: binding.to_device(v) for k, v in layer.items()} for layer in w["layers"]]}


def _steps(dec, prompts, G, n_steps, chain):
    dec.set_chain(int(chain))
    dec.state_reset(prompts, G)
    outs = []
    for _ in range(n_steps):
        if dec.num_active == 0:
            break
        outs.append(dec.denoise_step(want_logits=True))
    return outs, dec.tokens().copy()


@pytest.mark.parametrize("layers,B,P,G", [(3, 1, 256, 256),      # the 8B step shape: 512 rows, two row slabs per unit
                                          (2, 1, 300, 128),      # 428 rows: a ragged second slab
                                          (2, 2, 320, 192),      # two sequences, 1024 rows: two row tiles per projection
                                          (2, 3, 256, 256)])     # 1536 rows: an output projection without K slices
def test_chained_step_equals_unchained(layers, B, P, G):
    import torch
    from paper_2509_25188_b200 import binding
    shape = wl.thin(wl.LLADA_8B, layers)
    dev = _device_weights(shape)
    filt = wl.make_filter(32, 0.96, seed=0)
    prompts = wl.make_prompts(B, P, shape, seed=5)
    dec = binding.Decoder(shape, dev, filt, block_len=32, max_batch=B, max_seq=P + G,
                          lm_head_bias=wl.make_eot_bias(shape, 14.0))
    launches0 = dec.launch_count
    a, tok_a = _steps(dec, prompts, G, 3, chain=True)
    launches_chain = dec.launch_count - launches0
    b, tok_b = _steps(dec, prompts, G, 3, chain=False)
    launches_plain = dec.launch_count - launches0 - launches_chain
    dec.close()
    del dev
    torch.cuda.empty_cache()
    assert len(a) == len(b) == 3
    # the chained form really ran: far fewer launches (per layer 2 instead of 7)
    assert launches_chain < launches_plain - 3 * layers * 3
    for sa, sb in zip(a, b):
        for k in ("logits", "conf", "pred", "p", "unmask", "masks_left", "l_eff", "done", "forced"):
            assert np.array_equal(sa[k], sb[k]), "chained and unchained steps differ in %s" % k
    assert np.array_equal(tok_a, tok_b)


def test_chain_trace_records_every_phase():
    """The phase stamps: one launch for the first QKV and one per layer; opened <= finished, phases in order."""
    import torch
    from paper_2509_25188_b200 import binding
    shape = wl.thin(wl.LLADA_8B, 2)
    dev = _device_weights(shape)
    dec = binding.Decoder(shape, dev, wl.make_filter(32, 0.96, seed=0), block_len=32, max_batch=1, max_seq=512)
    prompts = wl.make_prompts(1, 256, shape, seed=5)
    dec.set_chain(1)
    dec.chain_trace_enable(True)
    dec.state_reset(prompts, 256)
    dec.denoise_step(outputs=False)
    tr = dec.chain_trace()
    dec.chain_trace_enable(False)
    dec.close()
    del dev
    torch.cuda.empty_cache()
    assert tr is not None and tr.shape[0] == 3 and tr.shape[1] == 6 and tr.shape[2] == 4
    n_phases = [1, 6, 4]                       # QKV | O norm gate/up down norm QKV | O norm gate/up down
    for launch, n in enumerate(n_phases):
        t = tr[launch, :n].astype(np.int64)
        assert (np.diff(t, axis=1) >= 0).all()   # per CTA: opened <= first ready <= last ready <= finished
        done = t[:, 3].max(axis=1)
        assert (np.diff(done) > 0).all()       # phases finish in order


@pytest.mark.parametrize("kv_cache,B,P,G", [(2, 1, 256, 256),     # dual cache: in-block steps of 32 rows
                                            (2, 8, 96, 64),       # eight sequences: 256 rows per in-block step
                                            (1, 2, 64, 64)])      # prefix cache: cached steps of 128 rows, then 64
def test_chained_cached_steps_equal_single_launches(kv_cache, B, P, G):
    """Key/value-cache configurations: steps of at most 256 rows chain with one row slab per unit and the two MMA issuers
    on alternate k-blocks.  Mode 2 runs the same tiling as single launches: every output of every step must agree bit for
    bit, across a block's first step (all rows) and the steps served from the store (including a block change)."""
    import torch
    from paper_2509_25188_b200 import binding
    shape = wl.thin(wl.LLADA_8B, 3)
    dev = _device_weights(shape)
    prompts = wl.make_prompts(B, P, shape, seed=9)
    # no filter: one commit per step, so a block has 32 steps and most of them read the store
    dec = binding.Decoder(shape, dev, None, block_len=32, max_batch=B, max_seq=P + G, kv_cache=kv_cache, use_filter=False,
                          lm_head_bias=wl.make_eot_bias(shape, 14.0))
    n_steps = 36                                   # crosses into the second block
    launches0 = dec.launch_count
    a, tok_a = _steps(dec, prompts, G, n_steps, chain=1)
    launches_chain = dec.launch_count - launches0
    b, tok_b = _steps(dec, prompts, G, n_steps, chain=2)
    launches_plain = dec.launch_count - launches0 - launches_chain
    dec.close()
    del dev
    torch.cuda.empty_cache()
    assert len(a) == len(b) >= 33
    assert launches_chain < launches_plain - len(a) * 3 * 2          # the chained form really ran on (nearly) every step
    for k_step, (sa, sb) in enumerate(zip(a, b)):
        for k in ("logits", "conf", "pred", "p", "unmask", "masks_left", "l_eff", "done", "forced"):
            assert np.array_equal(sa[k], sb[k]), "step %d: chained and single-launch steps differ in %s" % (k_step, k)
    assert np.array_equal(tok_a, tok_b)
