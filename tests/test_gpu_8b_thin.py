"""Full Learn2PD decodes at the LLaDA-8B widths (d 4096, 32 heads x 128, SwiGLU 12288, vocab
126464) with two layers, so that the oracle can follow them: the launch shapes of the decode
configurations — single sequence with an EoT bias, a batch of 16 with drop-out, and the batch of
8 with the prefix key/value cache — through the C ABI.

On every step of every sequence the decision logic (filter, threshold, fallback commit, EoTP,
block advance) is replayed in fp64 on the decoder's own confidences and must match bit for bit;
on sampled (sequence, step) pairs — the first step, the first step served from the cache, the
step after [EoT] was committed, every sixth step — the oracle's forward pass is run on the
decoder's token state and logits, confidences, ids and decisions are compared within the bf16
tolerances.
"""
from __future__ import annotations

import os

import numpy as np
import pytest

from oracle import l2pd_oracle as orc
from paper_2509_25188_b200 import workloads as wl
from tests.helpers import lockstep, oracle_model

pytestmark = pytest.mark.gpu

SHAPE = wl.thin(wl.LLADA_8B, 2)


@pytest.fixture(scope="module")
def thin8b():
    import torch
    from paper_2509_25188_b200 import binding
    w = wl.make_weights(SHAPE, seed=0, final_norm_gain=wl.spread_gain(SHAPE), threads=os.cpu_count() or 8)
    dev = {"tok_emb": binding.to_device(w["tok_emb"]), "lm_head": binding.to_device(w["lm_head"]),
           "final_norm": w["final_norm"],
           "layers": [{k: binding.to_device(v) for k, v in layer.items()} for layer in w["layers"]]}
    yield w, dev
    del dev
    torch.cuda.empty_cache()


def _run(thin8b, *, B, P, G, kv_cache, eot_bias, seed, sample, max_steps=None):
    from paper_2509_25188_b200 import binding
    w, dev = thin8b
    s = 32
    bias = wl.make_eot_bias(SHAPE, eot_bias) if eot_bias is not None else None
    m = oracle_model(SHAPE, w, lm_head_bias=bias)
    filt = wl.make_filter(s, 0.96, seed=0)
    prompts = wl.make_prompts(B, P, SHAPE, seed=seed)
    cfg = orc.DecodeConfig(block_len=s, kv_cache=bool(kv_cache), dual_cache=kv_cache == 2)
    dec = binding.Decoder(SHAPE, dev, filt, block_len=s, max_batch=B, max_seq=P + G, kv_cache=kv_cache,
                          lm_head_bias=bias)
    # spread logits (row maxima ~32): |d conf| <= 0.5 max|d logit|, and a logit error of 6e-3 of the row maximum allows 0.1
    st = lockstep(dec, m, filt, cfg, prompts, G, logit_rtol=2e-2, conf_atol=1e-3, p_margin=0.3,
                  oracle_when=sample, max_steps=max_steps)
    # The same decode through l2pd_decode: identical tokens, lengths and step counts (the path is
    # bit-reproducible: K slices are summed in a fixed order, nothing is accumulated with atomics).
    toks, out_len, steps, total = dec.decode(prompts, G)
    dec.close()
    _check_decode_invariants(st, toks, out_len, steps, total, P, G, s)
    return st, toks, out_len, steps, total


def _check_decode_invariants(st, toks, out_len, steps, total, P, G, s):
    B = toks.shape[0]
    assert total == steps.max()                       # every step runs all unfinished sequences
    agree = 0
    for i in range(B):
        n = int(out_len[i])
        assert 1 <= n <= G
        blocks_run = -(-n // s)
        assert blocks_run <= steps[i] <= blocks_run * s     # at least one step per block, at most one per mask
        if n < G:                                     # EoTP: [EoT] closes the response and fills the tail
            assert toks[i][n - 1] == SHAPE.eot_id and (toks[i][n:] == SHAPE.eot_id).all()
            assert SHAPE.eot_id not in toks[i][: n - 1]
        final = st["states"][i]
        agree += int(np.array_equal(toks[i], final.tokens[P:]) and n == final.L_eff - P)
    assert agree == B, "l2pd_decode and the step-by-step run differ in %d of %d sequences" % (B - agree, B)


def test_single_sequence_decode_with_eot_bias(thin8b):
    """Prompt 256 + generation 256, block 32, EoT logit biased so that EoTP can fire before the end."""
    seen = {"eot": False}

    def sample(i, k, state):
        # first step, every sixth step, and the first step after [EoT] has been committed
        if state.eot_pos >= 0 and not seen["eot"]:
            seen["eot"] = True
            return True
        return k == 0 or k % 6 == 5

    st, toks, out_len, steps, total = _run(thin8b, B=1, P=256, G=256, kv_cache=False, eot_bias=14.0, seed=11,
                                           sample=sample)
    assert st["oracle_steps"] >= 2 and st["replay_checked"] >= 0.9 * st["steps"]
    assert st["max_logit_rel"] < 2e-2
    assert 1 <= st["seq_steps"][0] <= 256              # never more steps than masks


def test_batch_of_16_with_drop_out(thin8b):
    """Batch 16, prompt 512 + generation 512: sequences finish at different steps and leave the batch."""
    def sample(i, k, state):
        return i == 3 and k in (0, 4)

    st, toks, out_len, steps, total = _run(thin8b, B=16, P=512, G=512, kv_cache=False, eot_bias=15.0, seed=21,
                                           sample=sample)
    assert st["oracle_steps"] >= 1
    assert st["replay_checked"] >= 0.9 * sum(st["seq_steps"])
    # drop-out: the batch shrinks before the last step unless every sequence took the same number of steps
    if len(set(st["seq_steps"])) > 1:
        taking_part = [int((np.asarray(t["done"]) >= 0).sum()) for t in st["trace"]]
        assert taking_part[0] == 16 and min(taking_part) < 16


def test_batch_of_8_prefix_cache(thin8b):
    """Batch 8, prompt 1024 + generation 1024 with the prefix key/value cache; the oracle follows
    sequence 0 with the same caching rule on the first (full) step and the first cached step."""
    def sample(i, k, state):
        return i == 0 and k in (0, 1)

    st, toks, out_len, steps, total = _run(thin8b, B=8, P=1024, G=1024, kv_cache=True, eot_bias=15.0, seed=31,
                                           sample=sample)
    assert st["oracle_steps"] == 2
    assert st["replay_checked"] >= 0.9 * sum(st["seq_steps"])


def test_dual_cache_single_sequence_and_batch(thin8b):
    """Dual cache at the 8B widths: in-block steps run 32 rows per sequence (the small-M launch shapes).
    The oracle follows the first (full) step and two stored-key steps, among them one after [EoT]."""
    seen = {"eot": False}

    def sample(i, k, state):
        if i == 0 and state.eot_pos >= 0 and not seen["eot"]:
            seen["eot"] = True
            return True
        return i == 0 and k in (0, 1, 2)

    st, toks, out_len, steps, total = _run(thin8b, B=1, P=256, G=256, kv_cache=2, eot_bias=14.0, seed=11,
                                           sample=sample)
    assert st["oracle_steps"] >= 3 and st["replay_checked"] >= 0.9 * st["steps"]
    st, toks, out_len, steps, total = _run(thin8b, B=8, P=1024, G=1024, kv_cache=2, eot_bias=15.0, seed=31,
                                           sample=lambda i, k, state: i == 0 and k in (0, 1))
    assert st["oracle_steps"] == 2
    assert st["replay_checked"] >= 0.9 * sum(st["seq_steps"])


def test_comparison_policies_at_the_8b_widths(thin8b):
    """Fixed confidence threshold and EGP (with a seeded synthetic reference: most steps take the
    fallback and write reference ids) through the full-width kernels; every decision replayed, the
    oracle's forward pass on sampled steps, and Algorithm 1's samples collected on the way."""
    from paper_2509_25188_b200 import binding
    w, dev = thin8b
    s, B, P, G = 32, 2, 96, 64
    bias = wl.make_eot_bias(SHAPE, 14.0)
    m = oracle_model(SHAPE, w, lm_head_bias=bias)
    filt = wl.make_filter(s, 0.96, seed=0)
    prompts = wl.make_prompts(B, P, SHAPE, seed=41)
    dec = binding.Decoder(SHAPE, dev, filt, block_len=s, max_batch=B, max_seq=P + G, lm_head_bias=bias)
    sample = lambda i, k, state: i == 0 and k in (0, 3)
    cfg = orc.DecodeConfig(block_len=s, rule="confidence", conf_threshold=0.6)
    dec.set_unmask_rule("confidence", conf_threshold=0.6)
    st = lockstep(dec, m, filt, cfg, prompts, G, logit_rtol=2e-2, conf_atol=1e-3, p_margin=0.3, oracle_when=sample)
    assert st["oracle_steps"] >= 1 and st["replay_checked"] >= 0.9 * sum(st["seq_steps"])
    rng = np.random.default_rng(5)
    refs = rng.integers(0, SHAPE.vocab - 2, size=(B, G))
    cfg = orc.DecodeConfig(block_len=s, rule="egp")
    dec.set_unmask_rule("egp", reference=refs)
    sink_c, sink_y = dec.set_collect(B * G)
    st = lockstep(dec, m, filt, cfg, prompts, G, logit_rtol=2e-2, conf_atol=1e-3, p_margin=0.3, oracle_when=sample, refs=refs)
    assert st["replay_checked"] == sum(st["seq_steps"])          # integer test: every step is replayed
    n = dec.collect_count
    assert n == sum(st["seq_steps"])
    for i in range(B):
        assert np.array_equal(st["states"][i].tokens[P:], refs[i])  # EGP ends in the reference
    y = sink_y[:n].cpu().numpy()
    c = sink_c[:n].cpu().numpy()
    assert set(np.unique(y)) <= {0, 1} and (c >= 0).all() and (c <= 1.0 + 1e-6).all()
    dec.close()
