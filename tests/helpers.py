"""Glue between the seeded workload generator and the oracle (tests only)."""
from __future__ import annotations

import numpy as np

from oracle import l2pd_oracle as orc
from paper_2509_25188_b200 import workloads as wl


def oracle_model(shape: wl.ModelShape, weights, lm_head_bias=None) -> orc.Model:
    return orc.Model(n_layers=shape.n_layers, d_model=shape.d_model, n_heads=shape.n_heads,
                     head_dim=shape.head_dim, d_ff=shape.d_ff, vocab=shape.vocab,
                     rms_eps=shape.rms_eps, rope_theta=shape.rope_theta, mask_id=shape.mask_id,
                     eot_id=shape.eot_id, weights=weights, lm_head_bias=lm_head_bias)


def small_shape(**kw) -> wl.ModelShape:
    base = dict(n_layers=2, d_model=64, n_heads=2, head_dim=32, d_ff=96, vocab=50,
                rms_eps=1e-5, rope_theta=10000.0, mask_id=49, eot_id=48, dtype="fp32")
    base.update(kw)
    return wl.ModelShape(**base)


def const_filter(s: int, bias: float):
    """Filter whose output logit is `bias` for every position, whatever the input."""
    z = np.zeros((s, s), np.float32)
    return {"w1": z, "b1": np.zeros(s, np.float32), "w2": z.copy(),
            "b2": np.full(s, bias, np.float32)}


def identity_filter(s: int, k: float, b: float):
    """z_j = k * relu(c_j) + b, so p_j = sigmoid(k c_j + b) for c_j >= 0."""
    return {"w1": np.eye(s, dtype=np.float32), "b1": np.zeros(s, np.float32),
            "w2": (k * np.eye(s)).astype(np.float32), "b2": np.full(s, b, np.float32)}


# ------------------------------------------------------------------------------------------------
# GPU-vs-oracle lockstep (used by the -m gpu tests)

def conf_interval(conf, eps):
    """Eq. 4 under a bounded logit error: conf = p_top; if every logit of the row is off by at most eps, the odds
    p_top / (1 - p_top) change by a factor within [exp(-2 eps), exp(2 eps)] (numerator by exp(+-eps), every term of the
    rest by exp(-+eps)), and a changed argmax stays inside the same interval.  Returns (lo, hi) per row."""
    c = np.clip(np.asarray(conf, dtype=np.float64), 1e-300, 1.0)
    e = np.asarray(eps, dtype=np.float64)
    odds = c / np.maximum(1.0 - c, 1e-300)
    lo = 1.0 / (1.0 + np.exp(2 * e) / odds)
    hi = 1.0 / (1.0 + np.exp(-2 * e) / odds)
    return lo, hi

def _sync_oracle_state(st, m, toks, msk, l_eff, done, cur_block):
    st.tokens[:] = toks
    st.masked[:] = msk
    st.L_eff = int(l_eff)
    st.done = bool(done)
    st.cur_block = int(cur_block)
    gen = st.tokens[st.P: st.P + st.G]
    hits = np.where((gen == m.eot_id) & ~st.masked)[0]
    st.eot_pos = int(hits[0]) if len(hits) and st.L_eff == st.P + int(hits[0]) + 1 else -1


def lockstep(dec, m, filt, cfg, prompts, G, *, logit_rtol, conf_atol, p_margin, conf_margin=None,
             check_logits=True, max_steps=None, replay_margin=1e-5, oracle_when=None, refs=None):
    """Runs the CUDA decoder step by step; before every step the oracle is put in the decoder's
    state (teacher forcing), then both take the step and are compared:
      logits  |gpu - orc| <= logit_rtol * max|orc row|
      conf    within conf_atol of the interval the row's measured logit error allows: if every logit of the row
              moves by at most eps, the odds of the top class move by a factor in [exp(-2 eps), exp(2 eps)], i.e.
              conf_gpu lies in [sigmoid(L - 2 eps), sigmoid(L + 2 eps)] with L = logit(conf_orc) (Eq. 4; exact, not
              first order, and it also covers a changed argmax).  Where that interval is narrower than conf_atol
              (peaked or flat rows, small eps) the check is conf_atol absolute.  Without logits (check_logits off)
              it is |gpu - orc| <= conf_atol.
      pred    equal wherever the oracle's top-2 logit gap exceeds 2 * logit_rtol * max|orc row|
      unmask  equal to the oracle's wherever every |p - tau| of the block exceeds p_margin (and, on a
              forced step, the two best confidences differ by more than conf_margin, default
              2 * conf_atol); and ALWAYS equal to the oracle's decision logic replayed in fp64 on the
              decoder's own conf/pred, unless a replayed |p - tau| is within replay_margin (the
              decoder evaluates the filter in fp32).
    oracle_when(i, step_of_sequence_i, state) -> bool selects the (sequence, step) pairs on which the
    oracle's forward pass is run and compared (default: all of them); the decision replay runs on
    every step of every sequence either way, since it needs no forward pass.
    Under cfg.rule "confidence" the margins apply to |conf - conf_threshold| instead of |p - tau|;
    under "egp" (refs[i] = reference answer of sequence i) the test is an integer comparison and the
    oracle's own decision is compared where every prediction of the block is sure.
    Returns counters; asserts on any violation.
    """
    import copy

    def boundary_distance(r, blk_masked, n):
        if cfg.rule == "filter":
            return np.abs(r.p - cfg.tau)[blk_masked]
        if cfg.rule == "confidence":
            return np.abs(r.conf - cfg.conf_threshold)[blk_masked[:n]]
        return np.zeros(0)

    prompts = np.asarray(prompts)
    B, P = prompts.shape
    s = cfg.block_len
    dec.state_reset(prompts, G)
    states = [orc.init_state(m, p, G) for p in prompts]
    stat = dict(steps=0, rows=0, pred_checked=0, unmask_checked=0, replay_checked=0, forced=0,
                max_logit_rel=0.0, max_logit_abs=0.0, max_conf_err=0.0, max_conf_excess=0.0, max_conf_allowed=0.0,
                seq_steps=[0] * B, oracle_steps=0, trace=[])
    while dec.num_active > 0:
        if max_steps is not None and stat["steps"] >= max_steps:
            break
        toks, msk = dec.tokens(), dec.masked()
        active = [i for i in range(B) if not states[i].done]
        for i in active:
            assert np.array_equal(states[i].tokens, toks[i]) and np.array_equal(states[i].masked, msk[i])
        want_oracle = {i: (oracle_when is None or bool(oracle_when(i, stat["seq_steps"][i], states[i]))) for i in active}
        need_logits = check_logits and any(want_oracle.values())
        out = dec.denoise_step(want_logits=need_logits)
        stat["steps"] += 1
        stat["trace"].append({k: np.array(out[k]) for k in ("block", "masks_left", "l_eff", "done", "forced")})
        replayed = {}
        for i in active:
            st = states[i]
            pre = copy.deepcopy(st)
            blk = st.cur_block
            n = min(s, st.L_eff - (st.P + blk * s))
            stat["seq_steps"][i] += 1
            stat["rows"] += n
            assert out["block"][i] == blk
            assert (out["pred"][i, n:] == -1).all() and (out["conf"][i, n:] == 0).all()
            rec = None
            if want_oracle[i]:
                rec = orc.denoise_step(m, filt, st, cfg, keep_logits=True, ref=None if refs is None else refs[i])
                stat["oracle_steps"] += 1
                assert rec.block == blk and rec.n_rows == n
                row_max = np.abs(rec.logits).max(axis=-1)
                cerr = np.abs(out["conf"][i, :n] - rec.conf)
                stat["max_conf_err"] = max(stat["max_conf_err"], float(cerr.max()))
                step_conf_margin = conf_margin
                if check_logits:
                    eps = np.abs(out["logits"][i, :n] - rec.logits).max(axis=-1)
                    err = eps / row_max
                    stat["max_logit_rel"] = max(stat["max_logit_rel"], float(err.max()))
                    stat["max_logit_abs"] = max(stat["max_logit_abs"], float(eps.max()))
                    assert err.max() <= logit_rtol, "logits off by %g (rel) at step %d" % (err.max(), stat["steps"])
                    lo, hi = conf_interval(rec.conf, eps)
                    g = out["conf"][i, :n].astype(np.float64)
                    excess = np.maximum(np.maximum(lo - g, g - hi), 0.0)
                    stat["max_conf_excess"] = max(stat["max_conf_excess"], float(excess.max()))
                    stat["max_conf_allowed"] = max(stat["max_conf_allowed"], float(np.maximum(hi - rec.conf, rec.conf - lo).max()))
                    assert excess.max() <= conf_atol, ("confidence outside what the row's logit error allows by %g at step %d"
                                                       % (excess.max(), stat["steps"]))
                    if step_conf_margin is None:   # two confidences are told apart only beyond twice what their rows allow
                        step_conf_margin = 2 * (float(np.maximum(hi - rec.conf, rec.conf - lo).max()) + conf_atol)
                else:
                    assert cerr.max() <= conf_atol, "confidence off by %g at step %d" % (cerr.max(), stat["steps"])
                if step_conf_margin is None:
                    step_conf_margin = 2 * conf_atol
                sure = rec.gap > 2 * logit_rtol * row_max
                stat["pred_checked"] += int(sure.sum())
                assert np.array_equal(out["pred"][i, :n][sure], rec.pred[sure])

            # decision logic replayed on the decoder's own numbers
            rp = copy.deepcopy(pre)
            rp.steps += 1
            gpred = out["pred"][i, :n].astype(np.int64)
            gconf = out["conf"][i, :n].astype(np.float64)
            rrec = orc.decide(m, filt, rp, cfg, gpred, gconf, ref=None if refs is None else refs[i])
            blk_masked = pre.masked[blk * s: blk * s + s]
            near = boundary_distance(rrec, blk_masked, n)
            replay_ok = (len(near) == 0 or near.min() > replay_margin)
            if replay_ok:
                stat["replay_checked"] += 1
                assert np.array_equal(out["unmask"][i].astype(bool), rrec.unmask), "decision replay differs"
                assert out["l_eff"][i] == rp.L_eff and bool(out["done"][i]) == rp.done
                assert out["forced"][i] == int(rrec.forced)
                assert out["masks_left"][i] == int(rp.masked[blk * s: blk * s + s].sum())
                assert np.abs(out["p"][i] - rrec.p).max() < 1e-4
                replayed[i] = rp

            if rec is None:
                continue
            # the oracle's own decision, where it is clear of the margins
            near_o = boundary_distance(rec, blk_masked, n)
            clear = len(near_o) == 0 or near_o.min() > p_margin
            if cfg.rule == "egp":
                clear = bool(sure.all())
            if rec.forced:
                cm = np.sort(rec.conf[blk_masked[:n]])[::-1]
                clear = clear and (len(cm) < 2 or cm[0] - cm[1] > step_conf_margin)
            if clear:
                stat["unmask_checked"] += 1
                assert np.array_equal(out["unmask"][i].astype(bool), rec.unmask), "unmask decision differs"
                assert out["forced"][i] == int(rec.forced)
                stat["forced"] += int(rec.forced)
        toks, msk = dec.tokens(), dec.masked()
        for i, rp in replayed.items():     # the committed ids and the mask set after the step
            assert np.array_equal(rp.tokens, toks[i]) and np.array_equal(rp.masked, msk[i])
        for i in active:
            blk = out["block"][i]
            nxt = blk + 1 if (out["masks_left"][i] == 0 and not out["done"][i]) else blk
            _sync_oracle_state(states[i], m, toks[i], msk[i], out["l_eff"][i], out["done"][i], nxt)
    stat["states"] = states
    return stat


def find_eot_bias(m, shape, filt, G, cfg, prompt_len, seeds=range(3, 40), grid=None):
    """Seeded search, on the oracle only, for (prompt seed, EoT bias) whose decode stops with
    G/4 <= out_len <= 3G/4, so that EoTP fires in mid-sequence.  Returns (seed, bias, result)."""
    grid = np.arange(10.0, 24.0, 0.5) if grid is None else grid
    for seed in seeds:
        prompt = wl.make_prompts(1, prompt_len, shape, seed=seed)[0]
        for v in grid:
            m.lm_head_bias = wl.make_eot_bias(shape, float(v))
            r = orc.decode(m, filt, prompt, G, cfg, keep_trace=False)
            if G // 4 <= r.out_len <= 3 * G // 4:
                return seed, float(v), r
    raise AssertionError("no (seed, bias) on the grid stops mid-sequence")
