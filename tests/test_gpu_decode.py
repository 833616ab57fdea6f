"""Parity of the CUDA decode path (through the C ABI) with the oracle on seeded workloads.

fp32 configurations: logits within 1e-4 relative (to the row's largest |logit|), confidence within
1e-3 absolute, committed ids / decisions / step counts / whole sequences bit-exact.
bf16 configurations: logits within 2e-2 relative, confidence within 1e-3 absolute on the
unit-gain model, ids and decisions exact wherever the oracle's top-2 gap and |p - tau| clear
those tolerances (see tests/helpers.lockstep).
"""
from __future__ import annotations

import numpy as np
import pytest

from oracle import l2pd_oracle as orc
from paper_2509_25188_b200 import workloads as wl
from tests.helpers import const_filter, find_eot_bias, lockstep, oracle_model

pytestmark = pytest.mark.gpu


def _b():
    from paper_2509_25188_b200 import binding
    return binding


def _tiny(gain=None, seed=0):
    shape = wl.TINY
    w = wl.make_weights(shape, seed=seed, final_norm_gain=wl.spread_gain(shape) if gain is None else gain)
    return shape, w


def _decoder(shape, w, filt, dshape=None, **kw):
    b = _b()
    d = dshape or wl.DECODES["C0"]
    args = dict(block_len=d.block_len, tau=d.tau, max_batch=d.batch, max_seq=d.prompt_len + d.gen_len,
                kv_cache=d.kv_cache)
    args.update(kw)
    return b.Decoder(shape, w, filt, **args)


# ----------------------------------------------------------------------------- C0: tiny fp32 model

@pytest.mark.parametrize("gain", [None, 1.0])
def test_c0_full_decode_bit_exact(gain):
    shape, w = _tiny(gain)
    d = wl.DECODES["C0"]
    filt = wl.make_filter(d.block_len, d.tau, seed=0)
    prompts = wl.make_prompts(1, d.prompt_len, shape, seed=1)
    m = oracle_model(shape, w)
    ref = orc.decode(m, filt, prompts[0], d.gen_len, orc.DecodeConfig(block_len=d.block_len, tau=d.tau))
    dec = _decoder(shape, w, filt)
    toks, out_len, steps, total = dec.decode(prompts, d.gen_len)
    assert np.array_equal(toks[0], ref.response)
    assert out_len[0] == ref.out_len and steps[0] == ref.steps == total
    dec.close()


@pytest.mark.parametrize("gain", [None, 1.0])
def test_c0_lockstep_fp32(gain):
    shape, w = _tiny(gain)
    d = wl.DECODES["C0"]
    filt = wl.make_filter(d.block_len, d.tau, seed=0)
    prompts = wl.make_prompts(1, d.prompt_len, shape, seed=1)
    m = oracle_model(shape, w)
    cfg = orc.DecodeConfig(block_len=d.block_len, tau=d.tau)
    dec = _decoder(shape, w, filt)
    st = lockstep(dec, m, filt, cfg, prompts, d.gen_len, logit_rtol=1e-4, conf_atol=1e-3, p_margin=1e-4,
                  conf_margin=1e-5 if gain is None else 1e-7)
    assert st["max_logit_rel"] < 1e-4
    assert st["replay_checked"] >= st["steps"] - 2
    if gain is None:
        assert st["unmask_checked"] >= st["steps"] - 3
        assert st["pred_checked"] > 0.9 * st["rows"]
    dec.close()


def test_decode_equals_reset_plus_step_loop():
    shape, w = _tiny()
    d = wl.DECODES["C0"]
    filt = wl.make_filter(d.block_len, d.tau, seed=1)
    prompts = wl.make_prompts(1, d.prompt_len, shape, seed=5)
    dec = _decoder(shape, w, filt)
    toks, out_len, steps, total = dec.decode(prompts, d.gen_len)
    dec.state_reset(prompts, d.gen_len)
    n = 0
    while dec.num_active > 0:
        dec.denoise_step(outputs=False)
        n += 1
    assert n == total
    assert np.array_equal(dec.tokens()[:, d.prompt_len:], toks)
    assert not dec.masked().any()
    dec.close()


def test_filter_never_and_always_step_counts():
    """'never' commits one token per step (s steps per block, the vanilla count); 'always' one step per block."""
    shape, w = _tiny()
    d = wl.DECODES["C0"]
    prompts = wl.make_prompts(1, d.prompt_len, shape, seed=2)
    m = oracle_model(shape, w)
    for bias, want in ((-50.0, d.gen_len), (50.0, d.gen_len // d.block_len)):
        filt = const_filter(d.block_len, bias)
        dec = _decoder(shape, w, filt, use_eotp=False)
        toks, out_len, steps, total = dec.decode(prompts, d.gen_len)
        ref = orc.decode(m, filt, prompts[0], d.gen_len,
                         orc.DecodeConfig(block_len=d.block_len, tau=d.tau, use_eotp=False))
        assert total == want == ref.steps
        assert np.array_equal(toks[0], ref.response)
        dec.close()
    dec = _decoder(shape, w, None, use_eotp=False)          # no filter at all: one token per step
    _, _, steps, total = dec.decode(prompts, d.gen_len)
    assert total == d.gen_len
    dec.close()


def test_eotp_mid_sequence_matches_oracle():
    shape, w = _tiny()
    d = wl.DECODES["C0"]
    filt = wl.make_filter(d.block_len, d.tau, seed=0)
    m = oracle_model(shape, w)
    cfg = orc.DecodeConfig(block_len=d.block_len, tau=d.tau)
    seed, v, ref = find_eot_bias(m, shape, filt, d.gen_len, cfg, d.prompt_len)
    prompts = wl.make_prompts(1, d.prompt_len, shape, seed=seed)
    bias = wl.make_eot_bias(shape, v)
    dec = _decoder(shape, w, filt, lm_head_bias=bias)
    toks, out_len, steps, total = dec.decode(prompts, d.gen_len)
    assert out_len[0] == ref.out_len < d.gen_len and total == ref.steps
    assert np.array_equal(toks[0], ref.response)
    assert (toks[0, out_len[0] - 1:] == shape.eot_id).all()
    st = lockstep(dec, m, filt, cfg, prompts, d.gen_len, logit_rtol=1e-4, conf_atol=1e-3, p_margin=1e-4)
    assert st["steps"] == ref.steps
    dec.close()
    # the same input without EoTP runs every block
    dec = _decoder(shape, w, filt, lm_head_bias=bias, use_eotp=False)
    _, out_len2, _, total2 = dec.decode(prompts, d.gen_len)
    assert out_len2[0] == d.gen_len and total2 > total
    dec.close()


def test_batch_is_independent_and_finished_sequences_drop_out():
    shape, w = _tiny()
    s, P, G, B = 16, 24, 48, 4
    filt = wl.make_filter(s, 0.96, seed=2)
    prompts = wl.make_prompts(B, P, shape, seed=11)
    m = oracle_model(shape, w, lm_head_bias=wl.make_eot_bias(shape, 12.0))
    cfg = orc.DecodeConfig(block_len=s)
    refs = orc.decode_batch(m, filt, prompts, G, cfg, keep_trace=False)
    b = _b()
    dec = b.Decoder(shape, w, filt, block_len=s, max_batch=B, max_seq=P + G, lm_head_bias=m.lm_head_bias)
    toks, out_len, steps, total = dec.decode(prompts, G)
    for i, r in enumerate(refs):
        assert np.array_equal(toks[i], r.response) and out_len[i] == r.out_len and steps[i] == r.steps
    assert total == max(r.steps for r in refs)
    assert len({r.steps for r in refs}) > 1          # sequences really finish at different times
    # each sequence alone gives the same row
    for i in (0, B - 1):
        t1, l1, s1, _ = dec.decode(prompts[i:i + 1], G)
        assert np.array_equal(t1[0], toks[i]) and l1[0] == out_len[i] and s1[0] == steps[i]
    st = lockstep(dec, m, filt, cfg, prompts, G, logit_rtol=1e-4, conf_atol=1e-3, p_margin=1e-4)
    assert st["seq_steps"] == [r.steps for r in refs]
    dec.close()


@pytest.mark.parametrize("mode", [1, 2])
def test_kv_cache_matches_oracle_with_the_same_rule(mode):
    """mode 1: prefix cache, 2: dual cache (Section 4.3)."""
    shape, w = _tiny()
    s, P, G, B = 16, 40, 64, 2
    filt = wl.make_filter(s, 0.96, seed=3)
    prompts = wl.make_prompts(B, P, shape, seed=21)
    m = oracle_model(shape, w)
    cfg = orc.DecodeConfig(block_len=s, kv_cache=True, dual_cache=mode == 2)
    refs = orc.decode_batch(m, filt, prompts, G, cfg, keep_trace=False)
    b = _b()
    dec = b.Decoder(shape, w, filt, block_len=s, max_batch=B, max_seq=P + G, kv_cache=mode)
    toks, out_len, steps, _ = dec.decode(prompts, G)
    for i, r in enumerate(refs):
        assert np.array_equal(toks[i], r.response) and steps[i] == r.steps
    st = lockstep(dec, m, filt, cfg, prompts, G, logit_rtol=1e-4, conf_atol=1e-3, p_margin=1e-4)
    assert st["replay_checked"] > 0
    # cached steps process only the rows from the block start on (dual cache: the block's rows)
    dec.state_reset(prompts, G)
    dec.denoise_step(outputs=False)
    assert dec.last_step_rows == B * (P + G)
    dec.denoise_step(outputs=False)
    assert dec.last_step_rows == (B * G if mode == 1 else B * s)
    dec.close()


def test_dual_cache_one_token_per_step_with_eot_cut():
    """Dual cache with the filter off (every step but a block's first reads the store) and an [EoT]
    bias that cuts the sequence in mid-block, so stored positions beyond L_eff drop out of the keys."""
    shape, w = _tiny()
    s, P, G = 16, 40, 64
    filt = const_filter(s, -50.0)
    m = oracle_model(shape, w)
    cfg = orc.DecodeConfig(block_len=s, kv_cache=True, dual_cache=True)
    seed, bias, want = find_eot_bias(m, shape, filt, G, cfg, P)
    prompts = wl.make_prompts(1, P, shape, seed=seed)
    dec = _b().Decoder(shape, w, filt, block_len=s, max_batch=1, max_seq=P + G, kv_cache=2,
                       lm_head_bias=m.lm_head_bias)
    toks, out_len, steps, _ = dec.decode(prompts, G)
    assert np.array_equal(toks[0], want.response) and steps[0] == want.steps and out_len[0] == want.out_len
    st = lockstep(dec, m, filt, cfg, prompts, G, logit_rtol=1e-4, conf_atol=1e-3, p_margin=1e-4, conf_margin=1e-6)
    assert st["replay_checked"] == st["steps"] and st["forced"] > 0
    dec.close()


def test_committed_conf_mode_one():
    shape, w = _tiny()
    d = wl.DECODES["C0"]
    filt = wl.make_filter(d.block_len, d.tau, seed=4)
    prompts = wl.make_prompts(1, d.prompt_len, shape, seed=6)
    m = oracle_model(shape, w)
    cfg = orc.DecodeConfig(block_len=d.block_len, tau=d.tau, committed_conf_mode=1)
    ref = orc.decode(m, filt, prompts[0], d.gen_len, cfg, keep_trace=False)
    dec = _decoder(shape, w, filt, committed_conf_mode=1)
    toks, _, steps, _ = dec.decode(prompts, d.gen_len)
    assert np.array_equal(toks[0], ref.response) and steps[0] == ref.steps
    dec.close()


def test_errors_come_back_as_status_codes():
    b = _b()
    shape, w = _tiny()
    filt = wl.make_filter(16)
    dec = b.Decoder(shape, w, filt, block_len=16, max_batch=2, max_seq=96)
    good = wl.make_prompts(1, 32, shape, seed=1)
    with pytest.raises(b.L2pdError) as e:
        dec.denoise_step()                          # step before reset
    assert e.value.status == -7
    with pytest.raises(b.L2pdError) as e:
        dec.state_reset(good, 60)                   # G not a multiple of the block length
    assert e.value.status == -2
    with pytest.raises(b.L2pdError) as e:
        dec.state_reset(good, 80)                   # P + G > max_seq
    assert e.value.status == -2
    with pytest.raises(b.L2pdError) as e:
        dec.state_reset(wl.make_prompts(3, 32, shape, seed=1), 64)   # B > max_batch
    assert e.value.status == -2
    bad = good.copy()
    bad[0, 5] = shape.mask_id
    with pytest.raises(b.L2pdError) as e:
        dec.state_reset(bad, 64)
    assert e.value.status == -6
    bad[0, 5] = shape.vocab + 3
    with pytest.raises(b.L2pdError) as e:
        dec.state_reset(bad, 64)
    assert e.value.status == -6
    # the context is still usable after every refusal
    toks, _, _, total = dec.decode(good, 64)
    assert total >= 4 and toks.shape == (1, 64)
    with pytest.raises(b.L2pdError) as e:
        dec.denoise_step()                          # everything already done
    assert e.value.status == -7
    dec.close()
    with pytest.raises(b.L2pdError):
        b.Decoder(shape, w, filt, block_len=65, max_batch=1, max_seq=96)


def test_device_timeout_status_maps_to_an_error_and_the_context_recovers():
    """A kernel whose bounded wait runs out leaves a code in the context's status word; the host turns it into
    L2PD_ERR_TIMEOUT, clears it, and the context stays usable.  The word is preset through the test hook: no kernel is
    made to wait."""
    b = _b()
    shape, w = _tiny()
    d = wl.DECODES["C0"]
    filt = wl.make_filter(d.block_len, d.tau, seed=0)
    prompts = wl.make_prompts(1, d.prompt_len, shape, seed=1)
    dec = _decoder(shape, w, filt)
    want, _, steps, _ = dec.decode(prompts, d.gen_len)
    dec.state_reset(prompts, d.gen_len)
    dec.debug_set_device_status(2)
    with pytest.raises(b.L2pdError) as e:
        dec.denoise_step()
    assert e.value.status == -5 and "role 2" in str(e.value)
    # the word was cleared: the same context decodes again, with the same result
    got, _, steps2, _ = dec.decode(prompts, d.gen_len)
    assert np.array_equal(got, want) and steps2[0] == steps[0]
    dec.close()


# ----------------------------------------------------------------------------- bf16 tensor-core path

def _bf16_shape(**kw):
    base = dict(n_layers=2, d_model=512, n_heads=4, head_dim=128, d_ff=1408, vocab=5000, rms_eps=1e-5,
                rope_theta=500000.0, mask_id=4999, eot_id=4998, dtype="bf16")
    base.update(kw)
    return wl.ModelShape(**base)


@pytest.mark.parametrize("spread", [False, True])
@pytest.mark.parametrize("kv_cache", [0, 1, 2])
def test_bf16_small_model_lockstep(spread, kv_cache):
    shape = _bf16_shape()
    w = wl.make_weights(shape, seed=0, final_norm_gain=wl.spread_gain(shape) if spread else 1.0)
    s, P, G, B = 32, 100, 96, 2
    filt = wl.make_filter(s, 0.96, seed=0)
    prompts = wl.make_prompts(B, P, shape, seed=31)
    m = oracle_model(shape, w, lm_head_bias=wl.make_eot_bias(shape, 6.0) if spread else None)
    cfg = orc.DecodeConfig(block_len=s, kv_cache=kv_cache > 0, dual_cache=kv_cache == 2)
    b = _b()
    dec = b.Decoder(shape, w, filt, block_len=s, max_batch=B, max_seq=P + G, kv_cache=kv_cache,
                    lm_head_bias=m.lm_head_bias)
    # confidence: 1e-3 beyond what each row's measured logit error allows (helpers.conf_interval)
    st = lockstep(dec, m, filt, cfg, prompts, G, logit_rtol=2e-2, conf_atol=1e-3,
                  p_margin=0.02 if not spread else 0.3)
    print("bf16 small model spread=%s kv_cache=%d: max logit err rel %.2e abs %.3f, max conf err %.4f (allowed by the rows' logit "
          "errors: %.4f, excess %.1e)" % (spread, kv_cache, st["max_logit_rel"], st["max_logit_abs"], st["max_conf_err"],
                                         st["max_conf_allowed"], st["max_conf_excess"]))
    assert st["max_logit_rel"] < 2e-2
    assert st["replay_checked"] >= 0.9 * sum(st["seq_steps"])
    assert st["unmask_checked"] > 0
    dec.close()


@pytest.mark.parametrize("kv_cache", [1, 2])
def test_bf16_six_layers_three_sequences_cached_lockstep(kv_cache):
    """The key/value store at depth: six layers and three sequences, so that layer strides (layers 2..5) and sequence
    strides of the store are exercised together, every step compared with the oracle run under the same caching rule;
    an [EoT] bias cuts the sequences at different places (cached steps then run on shortened inputs)."""
    shape = _bf16_shape(n_layers=6)
    w = wl.make_weights(shape, seed=2, final_norm_gain=wl.spread_gain(shape))
    s, P, G, B = 32, 72, 96, 3
    filt = wl.make_filter(s, 0.96, seed=1)
    prompts = wl.make_prompts(B, P, shape, seed=41)
    m = oracle_model(shape, w, lm_head_bias=wl.make_eot_bias(shape, 6.0))
    cfg = orc.DecodeConfig(block_len=s, kv_cache=True, dual_cache=kv_cache == 2)
    dec = _b().Decoder(shape, w, filt, block_len=s, max_batch=B, max_seq=P + G, kv_cache=kv_cache, lm_head_bias=m.lm_head_bias)
    st = lockstep(dec, m, filt, cfg, prompts, G, logit_rtol=2e-2, conf_atol=1e-3, p_margin=0.3)
    cached_steps = sum(1 for t in st["trace"]) - len({int(b) for t in st["trace"] for b in np.asarray(t["block"]) if b >= 0})
    print("six layers kv_cache=%d: %d steps (%d oracle), max logit err rel %.2e, max conf err %.4f (allowed %.4f)"
          % (kv_cache, st["steps"], st["oracle_steps"], st["max_logit_rel"], st["max_conf_err"], st["max_conf_allowed"]))
    assert st["oracle_steps"] == sum(st["seq_steps"]) and st["max_logit_rel"] < 2e-2
    assert cached_steps >= 3                      # most steps read the store
    assert st["replay_checked"] >= 0.9 * sum(st["seq_steps"])
    dec.close()
