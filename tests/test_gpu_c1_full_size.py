"""Parity at full size: one denoising step of the LLaDA-8B-shaped model (32 layers, d 4096,
vocab 126464; 256 prompt tokens + 256 masks, block 32) through the C ABI, in the launch
configuration the benchmark times, against values the oracle computed for the same seeded weights
and prompt (tests/golden/c1_step_oracle.npz, written by tests/golden/make_c1_golden.py, which
calls only the oracle).

Checked: the residual stream after layers 0, 1, 15, 31 on sampled rows / columns and its per-row
RMS on every row; sampled logits of the 32 block rows within 2e-2 of the row's largest |logit|;
confidence (Eq. 4) within 1e-3 absolute on the unit-gain model and within the bound the logit
error implies on the spread model; argmax ids (Eq. 3) exact wherever the oracle's top-2 gap
clears the logit tolerance; the unmask decision equal to the oracle's wherever |p - tau| clears
the margin, and always bit-exact against the decision logic replayed in fp64 on the decoder's
own confidences.
"""
from __future__ import annotations

import os

import numpy as np
import pytest

from oracle import l2pd_oracle as orc
from paper_2509_25188_b200 import workloads as wl
from tests.helpers import conf_interval, oracle_model

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "c1_step_oracle.npz")
LOGIT_RTOL = 2e-2


@pytest.fixture(scope="module")
def c1():
    import torch
    from paper_2509_25188_b200 import binding
    shape, d = wl.LLADA_8B, wl.DECODES["C1"]
    w = wl.make_weights(shape, seed=0, threads=os.cpu_count() or 8)
    dev = {"tok_emb": binding.to_device(w["tok_emb"]), "lm_head": binding.to_device(w["lm_head"]), "layers": []}
    for layer in w["layers"]:
        dev["layers"].append({k: binding.to_device(v) for k, v in layer.items()})
        layer.clear()
    del w
    g = np.load(GOLDEN)
    prompt = wl.make_prompts(1, d.prompt_len, shape, seed=1)
    assert np.array_equal(prompt[0], g["prompt"])
    yield shape, d, dev, g, prompt
    del dev
    torch.cuda.empty_cache()


def _step(shape, d, dev, gain, prompt, capture=False):
    import torch
    from paper_2509_25188_b200 import binding
    w = dict(dev, final_norm=np.full(shape.d_model, gain, np.float32))
    filt = wl.make_filter(d.block_len, d.tau, seed=0)
    dec = binding.Decoder(shape, w, filt, block_len=d.block_len, tau=d.tau, max_batch=1,
                          max_seq=d.prompt_len + d.gen_len)
    dec.state_reset(prompt, d.gen_len)
    cap = None
    if capture:
        cap = torch.zeros(shape.n_layers + 1, d.prompt_len + d.gen_len, shape.d_model, device="cuda")
        dec.set_capture(cap)
    out = dec.denoise_step(want_logits=True)
    dec.set_capture(None)
    rows = dec.last_step_rows
    dec.close()
    return out, cap, rows, filt


def test_c1_residual_stream_matches_oracle(c1):
    shape, d, dev, g, prompt = c1
    out, cap, rows, _ = _step(shape, d, dev, 1.0, prompt, capture=True)
    assert rows == d.prompt_len + d.gen_len
    cap = cap.cpu().numpy().astype(np.float64)
    r, c = g["resid_rows"], g["resid_cols"]
    stats = {}
    for l in (0, 1, 15, 31):
        got = cap[l + 1]
        rms_o = g["resid_rms_l%d" % l]
        rms_g = np.sqrt((got ** 2).mean(axis=-1))
        err = (got[np.ix_(r, c)] - g["resid_l%d" % l]) / rms_o[r][:, None]
        stats[l] = (np.abs(rms_g / rms_o - 1.0).max(), np.sqrt((err ** 2).mean()), np.abs(err).max())
    print("layer: (row-RMS rel err max, entry err rms / row RMS, entry err max / row RMS)", stats)
    for l, (rms_rel, e_rms, e_max) in stats.items():
        # Every activation between kernels (normed input, q/k/v, probabilities, attention output,
        # SwiGLU output) is rounded to bf16: relative error uniform in +-2^-9, 1.1e-3 rms, five or
        # six times per layer, i.e. about 5e-3 of a layer's output, added in quadrature over the
        # layers and carried by the residual stream, whose RMS grows with depth as well.  Bounds:
        # 1e-2 of the row RMS after the first two layers and 3e-2 deeper for the rms error of the
        # sample, four times that for its largest entry, 5e-3 for the RMS of each of the 512 rows.
        bound = 1e-2 if l < 2 else 3e-2
        assert rms_rel < 5e-3, "layer %d row RMS off by %g" % (l, rms_rel)
        assert e_rms < bound, "layer %d entries: rms error %g of the row RMS" % (l, e_rms)
        assert e_max < 4 * bound, "layer %d entries: largest error %g of the row RMS" % (l, e_max)


@pytest.mark.parametrize("name", ["unit", "spread"])
def test_c1_confidence_head_and_decision_match_oracle(c1, name):
    shape, d, dev, g, prompt = c1
    gain = float(g[name + "_gain"])
    out, _, _, filt = _step(shape, d, dev, gain, prompt)
    s = d.block_len
    cols = g["vocab_cols"]
    absmax = g[name + "_row_absmax"]
    logits = out["logits"][0].astype(np.float64)
    err = np.abs(logits[:, cols] - g[name + "_logits_sample"]) / absmax[:, None]
    assert err.max() <= LOGIT_RTOL, "logits off by %g of the row's largest |logit|" % err.max()
    # the row's largest |logit| itself is a property of the whole row
    assert np.abs(np.abs(logits).max(axis=-1) / absmax - 1.0).max() <= LOGIT_RTOL

    conf_o, gap_o = g[name + "_conf"], g[name + "_gap"]
    # Confidence: 1e-3 beyond the interval the row's logit error allows (helpers.conf_interval: odds of the top class move
    # by at most exp(+-2 eps)).  The stored oracle logits are a sample of the vocabulary (every 997th column), so eps of a
    # row is taken as twice the largest error among its sampled columns.
    eps_row = 2.0 * np.abs(logits[:, cols] - g[name + "_logits_sample"]).max(axis=-1)
    lo, hi = conf_interval(conf_o, eps_row)
    gconf = out["conf"][0].astype(np.float64)
    excess = np.maximum(np.maximum(lo - gconf, gconf - hi), 0.0)
    print("max logit error / row absmax: %.3g (abs %.3g); max confidence error: %.3g (allowed by the rows' logit errors: %.3g, "
          "excess %.2g)" % (err.max(), eps_row.max() / 2, np.abs(gconf - conf_o).max(), np.maximum(hi - conf_o, conf_o - lo).max(),
                           excess.max()))
    assert excess.max() <= 1e-3
    sure = gap_o > 2 * LOGIT_RTOL * absmax
    assert np.array_equal(out["pred"][0][sure], g[name + "_pred"][sure])
    if name == "spread":
        assert sure.sum() >= 8
    # the confidence the decoder reports equals Eq. 4 evaluated on its own logits
    lmax = logits.max(axis=-1, keepdims=True)
    conf_from_logits = 1.0 / np.exp(logits - lmax).sum(axis=-1)
    assert np.abs(out["conf"][0] - conf_from_logits).max() < 1e-5
    assert np.array_equal(out["pred"][0], logits.argmax(axis=-1))

    # decision logic replayed in fp64 on the decoder's own conf / pred: bit-exact
    m = oracle_model(shape, {"layers": [], "final_norm": None, "tok_emb": None, "lm_head": None})
    cfg = orc.DecodeConfig(block_len=s, tau=d.tau)
    st = orc.init_state(m, prompt[0], d.gen_len)
    st.steps += 1
    rec = orc.decide(m, filt, st, cfg, out["pred"][0].astype(np.int64), out["conf"][0].astype(np.float64))
    if np.abs(rec.p - d.tau).min() > 1e-5:
        assert np.array_equal(out["unmask"][0].astype(bool), rec.unmask)
        assert out["forced"][0] == int(rec.forced)
        assert out["masks_left"][0] == s - int(rec.unmask.sum())
        assert np.abs(out["p"][0] - rec.p).max() < 1e-4
    # the oracle's own decision wherever its filter scores are clear of the threshold
    p_margin = 0.02 if name == "unit" else 0.3
    clear = np.abs(g[name + "_p"] - d.tau) > p_margin
    if not bool(g[name + "_forced"]) and not out["forced"][0]:
        assert np.array_equal(out["unmask"][0].astype(bool)[clear], g[name + "_unmask"][clear])


@pytest.mark.parametrize("name", ["C2", "C3", "C4", "C2-dual", "C4-dual"])
def test_full_depth_decodes_replay_every_decision(c1, name):
    """The decode configurations at full depth (32 layers): single sequence with an EoT bias, batch 16
    (prompt 512 + generation 512) and batch 8 with the prefix cache (1024 + 1024); "-dual": the same
    shapes with the dual cache (in-block steps of 32 rows per sequence).  The oracle's forward
    pass is out of reach here (minutes per step and sequence); what is checked on every step of every
    sequence is the decision logic — filter, threshold, fallback, commit, EoTP, block advance — replayed
    in fp64 on the decoder's own confidences, bit for bit, and the decode invariants at the end."""
    from paper_2509_25188_b200 import binding
    from tests.helpers import lockstep
    shape, _, dev, _, _ = c1
    dual = name.endswith("-dual")
    dsh = wl.DECODES[name.split("-")[0]]
    B, P, G, s = dsh.batch, dsh.prompt_len, dsh.gen_len, dsh.block_len
    kv_mode = 2 if dual else int(dsh.kv_cache)
    bias = wl.make_eot_bias(shape, 14.0)
    w = dict(dev, final_norm=np.full(shape.d_model, wl.spread_gain(shape), np.float32))
    filt = wl.make_filter(s, dsh.tau, seed=0)
    m = oracle_model(shape, {"layers": [], "final_norm": None, "tok_emb": None, "lm_head": None}, lm_head_bias=bias)
    cfg = orc.DecodeConfig(block_len=s, tau=dsh.tau, kv_cache=kv_mode > 0, dual_cache=dual)
    prompts = wl.make_prompts(B, P, shape, seed=41)
    dec = binding.Decoder(shape, w, filt, block_len=s, tau=dsh.tau, max_batch=B, max_seq=P + G,
                          kv_cache=kv_mode, lm_head_bias=bias)
    st = lockstep(dec, m, filt, cfg, prompts, G, logit_rtol=2e-2, conf_atol=1e-3, p_margin=0.3,
                  oracle_when=lambda i, k, state: False)
    dec.close()
    assert st["oracle_steps"] == 0
    assert st["replay_checked"] >= 0.9 * sum(st["seq_steps"])
    for i in range(B):
        final = st["states"][i]
        n = final.L_eff - P
        assert final.done and 1 <= n <= G and not final.masked[:n].any()
        blocks_run = -(-n // s)
        assert blocks_run <= st["seq_steps"][i] <= blocks_run * s
        gen = final.tokens[P:]
        if n < G:
            assert gen[n - 1] == shape.eot_id and (gen[n:] == shape.eot_id).all()
    print("%s: steps per sequence %s, output lengths %s" % (name, st["seq_steps"], [st["states"][i].L_eff - P for i in range(B)]))
