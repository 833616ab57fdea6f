"""Writes tests/golden/c4_cached_steps_oracle.npz: the oracle's results for the cached denoising steps of ONE sequence of
the key/value-cache workload (prompt 1024 + generation 1024, block 32) on the LLaDA-8B-shaped model at full depth
(32 layers, bf16 weights from the seeded generator, seed 0, spread final-norm gain):

    step 1   first step of block 0: the full forward over 2048 positions (it fills the store);
    step 2p  second step under the prefix rule: rows 1024 .. 2047 against stored keys of positions 0 .. 1023;
    step 2d  second step under the dual rule: the block's 32 rows against stored prefix ++ fresh block ++ stored rest.

The decision policy is Extremely Greedy Parallel (commit where the prediction equals a reference answer), with a
reference built so that the token state entering step 2 cannot depend on bf16 rounding: at the block-0 positions whose
step-1 prediction is beyond doubt (top-2 logit gap above twice the tolerance the tests use for "sure") the reference IS
that prediction, so step 1 commits exactly those positions; everywhere else the reference is a seeded random id that is
none of the position's three best candidates, so nothing else matches.  Step 2 then finds no match and commits the most
confident masked position with its reference token; the margin by which that position wins is stored.

Calls only oracle/ and the workload generator.  Takes 10-20 minutes and ~45 GB of host memory.

    python tests/golden/make_c4_golden.py
"""
from __future__ import annotations

import copy
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import l2pd_oracle as orc  # noqa: E402
from paper_2509_25188_b200 import workloads as wl  # noqa: E402

PROMPT_SEED, REF_SEED = 101, 202


def main():
    shape, d = wl.LLADA_8B, wl.DECODES["C4"]
    P, G, s = d.prompt_len, d.gen_len, d.block_len
    t0 = time.time()
    w = wl.make_weights(shape, seed=0, final_norm_gain=wl.spread_gain(shape), threads=os.cpu_count() or 8)
    print("weights %.0f s" % (time.time() - t0), flush=True)
    prompt = wl.make_prompts(1, P, shape, seed=PROMPT_SEED)[0]
    ref = wl.make_prompts(1, G, shape, seed=REF_SEED)[0]
    filt = wl.make_filter(s, d.tau, seed=0)
    m = orc.Model(n_layers=shape.n_layers, d_model=shape.d_model, n_heads=shape.n_heads, head_dim=shape.head_dim,
                  d_ff=shape.d_ff, vocab=shape.vocab, rms_eps=shape.rms_eps, rope_theta=shape.rope_theta,
                  mask_id=shape.mask_id, eot_id=shape.eot_id, weights=w)
    vocab_cols = np.concatenate([np.arange(0, shape.vocab, 997), [shape.vocab - 2, shape.vocab - 1]])
    out = {"prompt": prompt, "ref": ref, "vocab_cols": vocab_cols, "gain": np.array(wl.spread_gain(shape))}

    def record(tag, rec, masked_before):
        masked_conf = np.sort(rec.conf[:rec.n_rows][masked_before[:rec.n_rows]])[::-1]
        out.update({tag + "_pred": rec.pred, tag + "_conf": rec.conf, tag + "_gap": rec.gap, tag + "_unmask": rec.unmask,
                    tag + "_forced": np.array(rec.forced), tag + "_logits_sample": rec.logits[:, vocab_cols],
                    tag + "_row_absmax": np.abs(rec.logits).max(-1),
                    tag + "_top2_conf": masked_conf[:2].copy()})
        print("%s: forced %s, commits %s, two best confidences %s  (%.0f s)" % (tag, rec.forced, np.where(rec.unmask)[0],
                                                                              masked_conf[:2], time.time() - t0), flush=True)

    # step 1 under the dual configuration: it stores both what the prefix rule and what the dual rule read later
    cfg_dual = orc.DecodeConfig(block_len=s, tau=d.tau, rule="egp", kv_cache=True, dual_cache=True)
    cfg_prefix = orc.DecodeConfig(block_len=s, tau=d.tau, rule="egp", kv_cache=True)
    st = orc.init_state(m, prompt, G)
    mb = st.masked[:s].copy()
    # step 1 in two halves: the forward pass (which fills the store), then the reference, then the decision
    st.steps += 1
    logits1 = orc.block_logits(m, st, cfg_dual)
    pred1, conf1, gap1 = orc.confidence_head(logits1)
    absmax1 = np.abs(logits1).max(-1)
    top3 = np.argsort(-logits1, axis=-1)[:, :3]
    for j in range(s):
        while ref[j] in top3[j]:
            ref[j] = (ref[j] + 1) % (shape.vocab - 2)
    sure = gap1 > 4 * 2e-2 * absmax1                # twice the margin beyond which the tests compare ids
    order = np.argsort(-gap1)
    assert sure[order[:4]].all(), "fewer than four block positions have a clear prediction: pick another prompt seed"
    ref[:s][sure] = pred1[sure]
    out["ref"] = ref
    print("step 1: %d of %d positions beyond doubt (smallest such gap %.2f, largest other gap %.2f)"
          % (sure.sum(), s, gap1[sure].min(), gap1[~sure].max() if (~sure).any() else 0.0), flush=True)
    record("step1", orc.decide(m, filt, st, cfg_dual, pred1, conf1, gap1, logits1, ref), mb)
    assert np.array_equal(out["step1_unmask"][:s], sure) and not bool(out["step1_forced"])
    out["tokens_after_step1"] = st.tokens.copy()
    st_prefix = copy.copy(st)
    st_prefix.tokens, st_prefix.masked = st.tokens.copy(), st.masked.copy()
    mb = st.masked[:s].copy()
    record("step2_dual", orc.denoise_step(m, filt, st, cfg_dual, keep_logits=True, ref=ref), mb)
    out["tokens_after_step2_dual"] = st.tokens.copy()
    record("step2_prefix", orc.denoise_step(m, filt, st_prefix, cfg_prefix, keep_logits=True, ref=ref), mb)
    out["tokens_after_step2_prefix"] = st_prefix.tokens.copy()
    np.savez_compressed(os.path.join(ROOT, "tests", "golden", "c4_cached_steps_oracle.npz"), **out)
    print("done %.0f s" % (time.time() - t0))


if __name__ == "__main__":
    main()
