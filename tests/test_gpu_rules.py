"""Comparison policies of Section 3.1 on the CUDA path (fixed confidence threshold, the vanilla
one-token-per-step limit, Extremely Greedy Parallel with a reference answer) against the oracle."""
from __future__ import annotations

import numpy as np
import pytest

from oracle import l2pd_oracle as orc
from paper_2509_25188_b200 import workloads as wl
from tests.helpers import lockstep, oracle_model

pytestmark = pytest.mark.gpu


def _b():
    from paper_2509_25188_b200 import binding
    return binding


def _setup(batch=1, seed=0):
    shape = wl.TINY
    w = wl.make_weights(shape, seed=seed, final_norm_gain=wl.spread_gain(shape))
    d = wl.DECODES["C0"]
    filt = wl.make_filter(d.block_len, d.tau, seed=0)
    dec = _b().Decoder(shape, w, filt, block_len=d.block_len, tau=d.tau, max_batch=batch,
                       max_seq=d.prompt_len + d.gen_len)
    return shape, w, d, filt, dec, oracle_model(shape, w)


def test_vanilla_limit_takes_s_steps_per_block():
    shape, w, d, filt, dec, m = _setup()
    prompts = wl.make_prompts(1, d.prompt_len, shape, seed=1)
    cfg = orc.DecodeConfig(block_len=d.block_len, rule="confidence", conf_threshold=1.0, use_eotp=False)
    want = orc.decode(m, filt, prompts[0], d.gen_len, cfg, keep_trace=False)
    dec2 = _b().Decoder(shape, w, filt, block_len=d.block_len, tau=d.tau, max_batch=1,
                        max_seq=d.prompt_len + d.gen_len, use_eotp=False)
    dec2.set_unmask_rule("confidence", conf_threshold=1.0)
    toks, out_len, steps, total = dec2.decode(prompts, d.gen_len)
    assert steps[0] == d.gen_len == want.steps            # s steps for each of the G/s blocks
    assert np.array_equal(toks[0], want.response)
    # back to the filter: fewer steps, through the same context
    dec2.set_unmask_rule("filter")
    f = orc.decode(m, filt, prompts[0], d.gen_len, orc.DecodeConfig(block_len=d.block_len, tau=d.tau, use_eotp=False),
                   keep_trace=False)
    toks, _, steps, _ = dec2.decode(prompts, d.gen_len)
    assert steps[0] == f.steps and np.array_equal(toks[0], f.response)
    dec2.close(); dec.close()


@pytest.mark.parametrize("thr", [0.5, 0.9])
def test_confidence_threshold_lockstep(thr):
    shape, w, d, filt, dec, m = _setup(batch=2)
    prompts = wl.make_prompts(2, d.prompt_len, shape, seed=3)
    cfg = orc.DecodeConfig(block_len=d.block_len, rule="confidence", conf_threshold=thr)
    dec.set_unmask_rule("confidence", conf_threshold=thr)
    st = lockstep(dec, m, filt, cfg, prompts, d.gen_len, logit_rtol=1e-4, conf_atol=1e-3, p_margin=1e-4,
                  conf_margin=1e-5)
    assert st["replay_checked"] >= st["steps"] - 2 and st["unmask_checked"] >= st["steps"] - 3
    dec.close()


def test_egp_lockstep_and_reference_reproduced():
    """Reference = the standard (one token per step) decode of the oracle, Section 3.1.  Under EGP the
    CUDA path ends in that reference, takes no more steps than it, and agrees with the oracle's EGP
    decode step by step."""
    shape, w, d, filt, dec, m = _setup(batch=2)
    prompts = wl.make_prompts(2, d.prompt_len, shape, seed=5)
    van = orc.DecodeConfig(block_len=d.block_len, use_filter=False)
    refs = np.stack([orc.decode(m, None, p, d.gen_len, van, keep_trace=False).response for p in prompts])
    cfg = orc.DecodeConfig(block_len=d.block_len, rule="egp")
    dec.set_unmask_rule("egp", reference=refs)
    st = lockstep(dec, m, filt, cfg, prompts, d.gen_len, logit_rtol=1e-4, conf_atol=1e-3, p_margin=1e-4,
                  conf_margin=1e-5, refs=refs)
    assert st["replay_checked"] == sum(st["seq_steps"])
    toks, out_len, steps, _ = dec.decode(prompts, d.gen_len)
    for i in range(2):
        want = orc.decode(m, None, prompts[i], d.gen_len, cfg, keep_trace=False, ref=refs[i])
        assert np.array_equal(toks[i], refs[i]) and np.array_equal(toks[i], want.response)
        assert steps[i] == want.steps <= d.gen_len and out_len[i] == want.out_len
    dec.close()


def test_egp_fallback_commits_reference_ids():
    """A reference the model never predicts (every id shifted by one): the steps fall back and
    write the reference id, so the decode returns the shifted reference in the oracle's step count."""
    shape, w, d, filt, dec, m = _setup()
    prompts = wl.make_prompts(1, d.prompt_len, shape, seed=5)
    van = orc.decode(m, None, prompts[0], d.gen_len, orc.DecodeConfig(block_len=d.block_len, use_filter=False),
                     keep_trace=False)
    n_special = 2                                            # the two highest ids are [EoT] and [MASK]
    ref = ((van.response + 1) % (shape.vocab - n_special)).astype(np.int64)[None]
    assert shape.eot_id >= shape.vocab - n_special and shape.mask_id >= shape.vocab - n_special
    cfg = orc.DecodeConfig(block_len=d.block_len, rule="egp")
    want = orc.decode(m, None, prompts[0], d.gen_len, cfg, keep_trace=False, ref=ref[0])
    dec.set_unmask_rule("egp", reference=ref)
    toks, _, steps, _ = dec.decode(prompts, d.gen_len)
    assert np.array_equal(toks[0], want.response) and np.array_equal(toks[0], ref[0])
    assert steps[0] == want.steps
    dec.close()


def test_rule_errors():
    b = _b()
    shape, w, d, filt, dec, m = _setup()
    prompts = wl.make_prompts(1, d.prompt_len, shape, seed=5)
    with pytest.raises(b.L2pdError) as e:
        dec.set_unmask_rule("confidence", conf_threshold=1.5)
    assert e.value.status == -1
    bad = np.full((1, d.gen_len), shape.mask_id)
    with pytest.raises(b.L2pdError) as e:
        dec.set_unmask_rule("egp", reference=bad)
    assert e.value.status == -6
    dec.set_unmask_rule("egp", reference=np.zeros((1, d.gen_len // 2), np.int64))
    with pytest.raises(b.L2pdError) as e:
        dec.state_reset(prompts, d.gen_len)                 # reference length != G
    assert e.value.status == -2
    dec.set_unmask_rule("filter")
    dec.state_reset(prompts, d.gen_len)
    dec.close()


@pytest.mark.parametrize("depth", [1, 2, 4])
def test_filter_depth_variants(depth):
    """Section 4.4: one-, two- and four-layer filters; decisions bit-exact against the oracle in lockstep."""
    shape, w, d, filt, dec, m = _setup(batch=2)
    s = d.block_len
    rng = np.random.default_rng(depth)
    base = wl.make_filter(s, d.tau, seed=depth)
    layers = [(base["w1"], base["b1"])]
    for k in range(1, depth):
        layers.append(((rng.normal(size=(s, s)) * 0.3 + np.eye(s)).astype(np.float32), (0.1 * rng.normal(size=s)).astype(np.float32)))
    if depth > 1:
        layers[-1] = (base["w2"], base["b2"])
    ofilt = {"layers": layers}
    prompts = wl.make_prompts(2, d.prompt_len, shape, seed=7)
    cfg = orc.DecodeConfig(block_len=s, tau=d.tau)
    dec.set_filter_layers(layers)
    st = lockstep(dec, m, ofilt, cfg, prompts, d.gen_len, logit_rtol=1e-4, conf_atol=1e-3, p_margin=1e-3,
                  conf_margin=1e-5, replay_margin=1e-4)
    assert st["replay_checked"] >= 0.8 * sum(st["seq_steps"])
    if depth == 2:       # the list form of the init-time filter decodes exactly like it
        toks, _, steps, _ = dec.decode(prompts, d.gen_len)
        dec.set_filter_layers([])
        dec2 = _b().Decoder(shape, w, base, block_len=s, tau=d.tau, max_batch=2, max_seq=d.prompt_len + d.gen_len)
        toks2, _, steps2, _ = dec2.decode(prompts, d.gen_len)
        assert np.array_equal(toks, toks2) and np.array_equal(steps, steps2)
        dec2.close()
    dec.close()
