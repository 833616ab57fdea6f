"""The key/value cache at full depth: cached denoising steps of one sequence of the cache workload (prompt 1024 +
generation 1024, block 32) on the LLaDA-8B-shaped model with all 32 layers, through the C ABI, against values the
oracle computed under the same caching rules (tests/golden/c4_cached_steps_oracle.npz, written by
tests/golden/make_c4_golden.py, which calls only the oracle).

    step 1          first step of block 0: the full forward over 2048 positions, which fills the store of every layer;
    step 2, prefix  rows 1024 .. 2047 against the stored keys / values of positions 0 .. 1023 (kv_cache_mode 1);
    step 2, dual    the block's 32 rows against stored prefix ++ fresh block ++ stored rest (kv_cache_mode 2).

A wrong layer stride, row base or sequence offset of the store that only bites beyond the second layer changes the
logits of step 2 by far more than the bf16 tolerance.  The policy is Extremely Greedy Parallel with a reference built by
the golden script so that step 1 commits exactly the block positions whose prediction is beyond doubt (there the
reference is the prediction; elsewhere it is an id outside the position's best three): the token state entering step 2
then does not depend on bf16 rounding.
Checked per step: sampled logits of the block rows within 2e-2 of the row's largest |logit|; confidences within 1e-3 of
what the rows' logit errors allow; argmax ids where the oracle's top-2 gap is clear; the committed position.
"""
from __future__ import annotations

import os

import numpy as np
import pytest

from paper_2509_25188_b200 import workloads as wl
from tests.helpers import conf_interval

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "c4_cached_steps_oracle.npz")
LOGIT_RTOL = 2e-2


@pytest.fixture(scope="module")
def c4():
    import torch
    from paper_2509_25188_b200 import binding
    shape, d = wl.LLADA_8B, wl.DECODES["C4"]
    g = np.load(GOLDEN)
    w = wl.make_weights(shape, seed=0, final_norm_gain=float(g["gain"]), threads=os.cpu_count() or 8)
    dev = {"tok_emb": binding.to_device(w["tok_emb"]), "lm_head": binding.to_device(w["lm_head"]),
           "final_norm": w["final_norm"], "layers": []}
    for layer in w["layers"]:
        dev["layers"].append({k: binding.to_device(v) for k, v in layer.items()})
        layer.clear()
    del w
    prompt = wl.make_prompts(1, d.prompt_len, shape, seed=101)
    assert np.array_equal(prompt[0], g["prompt"])
    yield shape, d, dev, g, prompt
    del dev
    torch.cuda.empty_cache()


def _compare(tag, out, g, n_rows):
    cols = g["vocab_cols"]
    absmax = g[tag + "_row_absmax"]
    logits = out["logits"][0][:n_rows].astype(np.float64)
    dl = np.abs(logits[:, cols] - g[tag + "_logits_sample"])
    err = dl / absmax[:, None]
    # the stored oracle logits are a sample of the vocabulary: a row's largest error is taken as twice the sample's
    lo, hi = conf_interval(g[tag + "_conf"], 2.0 * dl.max(axis=-1))
    gconf = out["conf"][0][:n_rows].astype(np.float64)
    excess = np.maximum(np.maximum(lo - gconf, gconf - hi), 0.0)
    print("%s: max logit error / row absmax %.3g; max confidence error %.3g (allowed by the rows' logit errors %.3g, excess %.2g)"
          % (tag, err.max(), np.abs(gconf - g[tag + "_conf"]).max(), np.maximum(hi - g[tag + "_conf"], g[tag + "_conf"] - lo).max(),
             excess.max()))
    assert err.max() <= LOGIT_RTOL, "%s: logits off by %g of the row's largest |logit|" % (tag, err.max())
    assert np.abs(np.abs(logits).max(axis=-1) / absmax - 1.0).max() <= LOGIT_RTOL
    assert excess.max() <= 1e-3
    sure = g[tag + "_gap"] > 2 * LOGIT_RTOL * absmax
    assert np.array_equal(out["pred"][0][:n_rows][sure], g[tag + "_pred"][sure])
    same = np.array_equal(out["unmask"][0].astype(bool), g[tag + "_unmask"])
    if not bool(g[tag + "_forced"]):
        # positions whose prediction equals the reference: by construction only predictions that are beyond doubt
        assert same and out["forced"][0] == 0, "%s: the committed positions differ from the oracle's" % tag
    else:
        # nothing matched: one commit, the reference token at the most confident masked position; the position must
        # agree when the two best confidences are further apart than twice what the rows' logit errors allow
        top2 = g[tag + "_top2_conf"]
        margin = 2.0 * (np.maximum(hi - g[tag + "_conf"], g[tag + "_conf"] - lo).max() + 1e-3)
        assert out["forced"][0] == 1 and out["unmask"][0].sum() == 1
        if top2[0] - top2[1] > margin:
            assert same, "%s: another position was committed although the best confidence leads by %g" % (tag, top2[0] - top2[1])
    return same


@pytest.mark.parametrize("mode,tag2", [(1, "step2_prefix"), (2, "step2_dual")])
def test_cached_steps_at_full_depth_match_oracle(c4, mode, tag2):
    from paper_2509_25188_b200 import binding
    shape, d, dev, g, prompt = c4
    P, G, s = d.prompt_len, d.gen_len, d.block_len
    dec = binding.Decoder(shape, dev, wl.make_filter(s, d.tau, seed=0), block_len=s, tau=d.tau, max_batch=1, max_seq=P + G,
                          kv_cache=mode)
    dec.set_unmask_rule("egp", reference=g["ref"][None, :])
    dec.state_reset(prompt, G)
    out1 = dec.denoise_step(want_logits=True)
    assert dec.last_step_rows == P + G                       # the block's first step: every position
    _compare("step1", out1, g, s)
    assert np.array_equal(dec.tokens()[0], g["tokens_after_step1"])
    out2 = dec.denoise_step(want_logits=True)
    assert dec.last_step_rows == (G if mode == 1 else s)     # served from the store
    _compare(tag2, out2, g, s)
    dec.close()
