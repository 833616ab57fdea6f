"""Writes tests/golden/c1_step_oracle.npz: the oracle's result for ONE denoising step of the
LLaDA-8B-shaped model (32 layers, bf16 weights from the seeded generator, seed 0) on the C1 input
(256 seeded prompt tokens + 256 masks, block 32), for the unit final-norm gain and the spread gain.
Calls only oracle/ and the workload generator.  Takes a few minutes and ~40 GB of host memory.

    python tests/golden/make_c1_golden.py
"""
from __future__ import annotations

import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import l2pd_oracle as orc  # noqa: E402
from paper_2509_25188_b200 import workloads as wl  # noqa: E402


def main():
    shape, d = wl.LLADA_8B, wl.DECODES["C1"]
    t0 = time.time()
    w = wl.make_weights(shape, seed=0, threads=os.cpu_count() or 8)
    print("weights %.0f s" % (time.time() - t0), flush=True)
    prompt = wl.make_prompts(1, d.prompt_len, shape, seed=1)[0]
    filt = wl.make_filter(d.block_len, d.tau, seed=0)
    m = orc.Model(n_layers=shape.n_layers, d_model=shape.d_model, n_heads=shape.n_heads, head_dim=shape.head_dim,
                  d_ff=shape.d_ff, vocab=shape.vocab, rms_eps=shape.rms_eps, rope_theta=shape.rope_theta,
                  mask_id=shape.mask_id, eot_id=shape.eot_id, weights=w)
    st = orc.init_state(m, prompt, d.gen_len)
    # residual stream after chosen layers, for layer-wise checks of the CUDA path
    x = orc.widen(w["tok_emb"][st.tokens])
    pos = np.arange(len(st.tokens))
    keep = {}
    rows = np.array([0, 1, 100, 255, 256, 257, 300, 511])
    cols = np.arange(0, shape.d_model, 64)
    for l, layer in enumerate(w["layers"]):
        x = orc.layer_forward(m, layer, x, pos)
        if l in (0, 1, 15, 31):
            keep["resid_l%d" % l] = x[np.ix_(rows, cols)].copy()
            keep["resid_rms_l%d" % l] = np.sqrt((x ** 2).mean(axis=-1))
        print("layer %d  %.0f s" % (l, time.time() - t0), flush=True)
    out = dict(keep, resid_rows=rows, resid_cols=cols, prompt=prompt)
    vocab_cols = np.concatenate([np.arange(0, shape.vocab, 997), [shape.vocab - 2, shape.vocab - 1]])
    cfg = orc.DecodeConfig(block_len=d.block_len, tau=d.tau)
    for name, gain in (("unit", 1.0), ("spread", wl.spread_gain(shape))):
        w["final_norm"] = np.full(shape.d_model, gain, np.float32)
        logits = orc.lm_head_logits(m, x[st.P: st.P + d.block_len])
        pred, conf, gap = orc.confidence_head(logits)
        s2 = orc.init_state(m, prompt, d.gen_len)
        rec = orc.decide(m, filt, s2, cfg, pred, conf, gap)
        out.update({name + "_pred": pred, name + "_conf": conf, name + "_gap": gap, name + "_p": rec.p,
                    name + "_unmask": rec.unmask, name + "_forced": np.array(rec.forced),
                    name + "_logits_sample": logits[:, vocab_cols], name + "_row_absmax": np.abs(logits).max(-1),
                    name + "_gain": np.array(gain)})
    out["vocab_cols"] = vocab_cols
    np.savez_compressed(os.path.join(ROOT, "tests", "golden", "c1_step_oracle.npz"), **out)
    print("done %.0f s" % (time.time() - t0))


if __name__ == "__main__":
    main()
