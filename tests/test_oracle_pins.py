"""Pins for the CPU oracle: each test ties one of its functions to something other than
itself — a value the paper prints, a closed form, an invariant, a library routine the
oracle does not call (torch CPU), or brute force with scalar loops on tiny inputs."""
from __future__ import annotations

import math
import os

import numpy as np
import pytest
import torch

from oracle import l2pd_oracle as orc
from paper_2509_25188_b200 import workloads as wl
from tests.helpers import const_filter, find_eot_bias, identity_filter, oracle_model, small_shape

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def paper_constants():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


# ----------------------------------------------------------------------------- filter

def test_filter_parameter_count_matches_paper():
    """Section 4.1: 2,112 trainable parameters at block size 32, two layers."""
    c = paper_constants()
    f = wl.make_filter(32)
    assert sum(a.size for a in f.values()) == int(c["filter_params_at_block_32"])
    assert sum(a.size for a in wl.make_filter(16).values()) == 2 * (16 * 16 + 16)
    # the oracle consumes exactly those four arrays and maps s confidences to s logits
    z = orc.filter_logits(f, np.linspace(0, 1, 32))
    assert z.shape == (32,)


def test_filter_is_two_affine_maps_with_relu_scalar_bruteforce():
    s = 5
    f = wl.make_filter(s, seed=3)
    c = np.array([0.1, 0.9, 0.5, 0.0, 1.0])
    z = orc.filter_logits(f, c)
    for j in range(s):
        acc = float(f["b2"][j])
        for h in range(s):
            pre = float(f["b1"][h])
            for i in range(s):
                pre += float(f["w1"][h, i]) * c[i]
            acc += float(f["w2"][j, h]) * max(pre, 0.0)
        assert z[j] == pytest.approx(acc, abs=1e-12)
    # a negative pre-activation must be clipped: W1 = -I gives relu(-c) = 0 -> z = b2
    g = identity_filter(s, 1.0, 0.25)
    g["w1"] = -g["w1"]
    assert np.allclose(orc.filter_logits(g, c), 0.25)


def test_sigmoid_closed_form():
    assert orc.sigmoid(np.array([0.0]))[0] == 0.5
    assert orc.sigmoid(np.array([math.log(0.96 / 0.04)]))[0] == pytest.approx(0.96, abs=1e-15)
    z = np.array([-3.0, 2.0])
    assert np.allclose(orc.sigmoid(z) + orc.sigmoid(-z), 1.0)


# ----------------------------------------------------------------------------- unmask rule

def test_unmask_rule_threshold_is_strict_and_only_masked_positions_move():
    """Algorithm 2: position j leaves the mask set iff p_j > tau."""
    tau = 0.5
    p = np.array([0.5, 0.5000001, 0.49, 0.99, 0.99])
    conf = np.array([0.9, 0.1, 0.2, 0.3, 0.4])
    masked = np.array([True, True, True, True, False])
    un, forced = orc.unmask_rule(p, conf, masked, tau)
    assert un.tolist() == [False, True, False, True, False]   # equality stays masked
    assert not forced


def test_unmask_rule_with_identity_filter_is_a_confidence_cut():
    """With W1 = I, W2 = k I the rule reduces to conf > (logit(tau) - b) / k."""
    s, k, b, tau = 8, 10.0, -4.0, 0.96
    cut = (math.log(tau / (1 - tau)) - b) / k
    conf = np.array([cut - 0.01, cut + 0.01, 0.0, 1.0, cut - 1e-6, cut + 1e-6, 0.5, 0.9])
    p = orc.sigmoid(orc.filter_logits(identity_filter(s, k, b), conf))
    un, forced = orc.unmask_rule(p, conf, np.ones(s, bool), tau)
    assert un.tolist() == (conf > cut).tolist()
    assert not forced


def test_unmask_rule_fallback_commits_highest_confidence_lowest_index():
    p = np.zeros(6)
    conf = np.array([0.2, 0.7, 0.7, 0.9, 0.1, 0.3])
    masked = np.array([True, True, True, False, True, True])
    un, forced = orc.unmask_rule(p, conf, masked, 0.96)
    assert forced and un.tolist() == [False, True, False, False, False, False]
    un, forced = orc.unmask_rule(p, conf, np.zeros(6, bool), 0.96)
    assert not forced and not un.any()


def test_lower_threshold_unmasks_a_superset_within_one_step():
    rng = np.random.default_rng(0)
    for _ in range(20):
        p, conf = rng.random(32), rng.random(32)
        masked = rng.random(32) < 0.7
        hi, f_hi = orc.unmask_rule(p, conf, masked, 0.96)
        lo, f_lo = orc.unmask_rule(p, conf, masked, 0.90)
        if not f_hi:
            assert np.all(lo[hi])


# ----------------------------------------------------------------------------- confidence head

def test_confidence_head_bruteforce_tiny_vocab():
    """Eq. 3-4 by explicit enumeration over a vocabulary of 8."""
    rng = np.random.default_rng(1)
    logits = rng.normal(size=(5, 8)) * 3
    pred, conf, gap = orc.confidence_head(logits)
    for r in range(5):
        probs = [math.exp(logits[r, v]) for v in range(8)]
        tot = sum(probs)
        probs = [x / tot for x in probs]
        best = max(range(8), key=lambda v: (probs[v], -v))
        assert pred[r] == best
        assert conf[r] == pytest.approx(probs[best], abs=1e-14)
        srt = sorted(logits[r])
        assert gap[r] == pytest.approx(srt[-1] - srt[-2], abs=1e-14)


def test_confidence_head_invariants():
    V = 37
    pred, conf, _ = orc.confidence_head(np.full((3, V), 2.5))
    assert pred.tolist() == [0, 0, 0]                      # ties -> lowest id
    assert np.allclose(conf, 1.0 / V)
    rng = np.random.default_rng(2)
    logits = rng.normal(size=(6, V)) * 4
    p1, c1, _ = orc.confidence_head(logits)
    p2, c2, _ = orc.confidence_head(logits + 123.0)        # shift invariance
    assert (p1 == p2).all() and np.allclose(c1, c2, atol=1e-13)
    assert (c1 >= 1.0 / V - 1e-15).all() and (c1 <= 1.0).all()
    one_hot = np.full((1, V), -1e4)
    one_hot[0, 11] = 0.0
    p, c, _ = orc.confidence_head(one_hot)
    assert p[0] == 11 and c[0] == pytest.approx(1.0)
    # huge logits must not overflow
    p, c, _ = orc.confidence_head(np.array([[1e4, 1e4 - math.log(3.0)]]))
    assert p[0] == 0 and c[0] == pytest.approx(0.75)


# ----------------------------------------------------------------------------- transformer pieces

def test_rmsnorm_closed_form_and_library():
    y = orc.rmsnorm(np.array([[3.0, 4.0]]), np.ones(2, np.float32), 0.0)
    assert np.allclose(y, np.array([[3.0, 4.0]]) / math.sqrt(12.5))
    rng = np.random.default_rng(3)
    x = rng.normal(size=(7, 48))
    g = rng.normal(size=48).astype(np.float32)
    want = torch.nn.functional.rms_norm(torch.from_numpy(x), (48,),
                                        torch.from_numpy(g.astype(np.float64)), 1e-5).numpy()
    assert np.allclose(orc.rmsnorm(x, g, 1e-5), want, atol=1e-13)
    y1 = orc.rmsnorm(x, np.ones(48, np.float32), 0.0)
    assert np.allclose(np.sqrt((y1 ** 2).mean(-1)), 1.0)               # unit RMS with gain 1
    assert np.allclose(orc.rmsnorm(7.5 * x, g, 0.0), orc.rmsnorm(x, g, 0.0))  # scale invariance
    # eps is inside the square root, added to the mean square
    y = orc.rmsnorm(np.array([[0.0, 0.0]]), np.ones(2, np.float32), 1e-5)
    assert np.all(y == 0.0)
    y = orc.rmsnorm(np.array([[1.0, 1.0]]), np.ones(2, np.float32), 3.0)
    assert np.allclose(y, 0.5)


def test_rope_is_complex_rotation():
    """Half-split pairing: (x_i + i x_{i+dh/2}) * exp(i * pos * theta^(-2i/dh))."""
    rng = np.random.default_rng(4)
    T, H, dh, theta = 6, 3, 8, 10000.0
    x = rng.normal(size=(T, H, dh))
    pos = np.array([0, 1, 2, 5, 17, 300])
    y = orc.rope(x, pos, theta)
    for t in range(T):
        for h in range(H):
            for i in range(dh // 2):
                z = complex(x[t, h, i], x[t, h, i + dh // 2])
                z *= complex(math.cos(pos[t] * theta ** (-2 * i / dh)),
                             math.sin(pos[t] * theta ** (-2 * i / dh)))
                assert y[t, h, i] == pytest.approx(z.real, abs=1e-12)
                assert y[t, h, i + dh // 2] == pytest.approx(z.imag, abs=1e-12)
    assert np.array_equal(y[0], x[0])                                  # position 0: identity
    assert np.allclose((y ** 2).sum(-1), (x ** 2).sum(-1))             # a rotation keeps norms
    # dh = 2: a single plane rotated by exactly `pos` radians
    y2 = orc.rope(np.array([[[1.0, 0.0]]]), np.array([2]), 500000.0)
    assert np.allclose(y2[0, 0], [math.cos(2.0), math.sin(2.0)])


def test_rope_scores_depend_only_on_relative_position():
    rng = np.random.default_rng(5)
    T, H, dh = 5, 2, 16
    q, k, v = (rng.normal(size=(T, H, dh)) for _ in range(3))
    pos = np.arange(T)
    a0 = orc.attention(orc.rope(q, pos, 1e4), orc.rope(k, pos, 1e4), v)
    a1 = orc.attention(orc.rope(q, pos + 37, 1e4), orc.rope(k, pos + 37, 1e4), v)
    assert np.allclose(a0, a1, atol=1e-12)


def test_attention_matches_library_and_scalar_loops():
    rng = np.random.default_rng(6)
    Tq, Tk, H, dh = 4, 7, 2, 8
    q = rng.normal(size=(Tq, H, dh))
    k = rng.normal(size=(Tk, H, dh))
    v = rng.normal(size=(Tk, H, dh))
    got = orc.attention(q, k, v)
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2) for a in (q, k, v))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(1, 0, 2).numpy()
    assert np.allclose(got, want, atol=1e-13)
    # scalar definition: sum_j softmax_j(q.k_j / sqrt(dh)) v_j
    for t in range(Tq):
        for h in range(H):
            sc = [sum(q[t, h, c] * k[j, h, c] for c in range(dh)) / math.sqrt(dh) for j in range(Tk)]
            w = [math.exp(x - max(sc)) for x in sc]
            for c in range(dh):
                o = sum(w[j] * v[j, h, c] for j in range(Tk)) / sum(w)
                assert got[t, h, c] == pytest.approx(o, abs=1e-12)


def test_silu_matches_library():
    x = np.linspace(-8, 8, 41)
    assert np.allclose(orc.silu(x), torch.nn.functional.silu(torch.from_numpy(x)).numpy(), atol=1e-15)
    assert orc.silu(np.array([0.0]))[0] == 0.0


def _scalar_layer(shape, layer, x, pos):
    """Textbook loops for one pre-norm block (tiny sizes only)."""
    d, H, dh, F = shape.d_model, shape.n_heads, shape.head_dim, shape.d_ff
    T = len(x)

    def norm(row, g):
        ms = sum(a * a for a in row) / len(row)
        return [a * float(gg) / math.sqrt(ms + shape.rms_eps) for a, gg in zip(row, g)]

    def lin(row, W):
        return [sum(float(W[o, i]) * row[i] for i in range(W.shape[1])) for o in range(W.shape[0])]

    def rot(vec, p):
        out = list(vec)
        for i in range(dh // 2):
            a = p * shape.rope_theta ** (-2.0 * i / dh)
            out[i] = vec[i] * math.cos(a) - vec[i + dh // 2] * math.sin(a)
            out[i + dh // 2] = vec[i + dh // 2] * math.cos(a) + vec[i] * math.sin(a)
        return out

    qs, ks, vs = [], [], []
    for t in range(T):
        qkv = lin(norm(x[t], layer["norm1"]), layer["wqkv"])
        qs.append([rot(qkv[h * dh:(h + 1) * dh], pos[t]) for h in range(H)])
        ks.append([rot(qkv[H * dh + h * dh: H * dh + (h + 1) * dh], pos[t]) for h in range(H)])
        vs.append([qkv[2 * H * dh + h * dh: 2 * H * dh + (h + 1) * dh] for h in range(H)])
    out = []
    for t in range(T):
        att = []
        for h in range(H):
            sc = [sum(a * b for a, b in zip(qs[t][h], ks[j][h])) / math.sqrt(dh) for j in range(T)]
            w = [math.exp(s_ - max(sc)) for s_ in sc]
            att += [sum(w[j] * vs[j][h][c] for j in range(T)) / sum(w) for c in range(dh)]
        x1 = [a + b for a, b in zip(x[t], lin(att, layer["wo"]))]
        n2 = norm(x1, layer["norm2"])
        gate, up = lin(n2, layer["w_gate"]), lin(n2, layer["w_up"])
        hid = [g / (1.0 + math.exp(-g)) * u for g, u in zip(gate, up)]
        out.append([a + b for a, b in zip(x1, lin(hid, layer["w_down"]))])
    return np.array(out)


def test_layer_forward_matches_textbook_loops():
    shape = small_shape(n_layers=1, d_model=12, n_heads=2, head_dim=4, d_ff=10, vocab=11)
    w = wl.make_weights(shape, seed=5, std=0.5, threads=1)
    layer = w["layers"][0]
    rng = np.random.default_rng(7)
    layer["norm1"] = rng.normal(size=12).astype(np.float32)
    layer["norm2"] = rng.normal(size=12).astype(np.float32)
    x = rng.normal(size=(5, 12))
    pos = np.array([3, 4, 5, 6, 7])
    m = oracle_model(shape, w)
    got = orc.layer_forward(m, layer, x, pos)
    want = _scalar_layer(shape, layer, x.tolist(), pos.tolist())
    assert np.allclose(got, want, atol=1e-11)


def test_layer_is_identity_on_the_residual_when_output_projections_are_zero():
    shape = small_shape(n_layers=1)
    w = wl.make_weights(shape, seed=1, threads=1)
    w["layers"][0]["wo"][:] = 0
    w["layers"][0]["w_down"][:] = 0
    m = oracle_model(shape, w)
    toks = np.array([1, 2, 3, 4])
    x = orc.forward_hidden(m, toks)
    assert np.array_equal(x, w["tok_emb"][toks].astype(np.float64))


def test_forward_is_bidirectional():
    """Changing the LAST token must change position 0 (it would not under a causal mask)."""
    shape = small_shape()
    w = wl.make_weights(shape, seed=2, std=0.3, threads=1)
    m = oracle_model(shape, w)
    a = orc.forward_hidden(m, np.array([5, 6, 7, 8, 9]))
    b = orc.forward_hidden(m, np.array([5, 6, 7, 8, 10]))
    assert np.abs(a[0] - b[0]).max() > 1e-6
    # and the first token changes the last position too
    c = orc.forward_hidden(m, np.array([4, 6, 7, 8, 9]))
    assert np.abs(a[-1] - c[-1]).max() > 1e-6


def test_lm_head_special_cases():
    shape = small_shape(n_layers=0, d_model=8, vocab=8, n_heads=1, head_dim=8, mask_id=7, eot_id=6)
    w = wl.make_weights(shape, seed=0, threads=1)
    w["lm_head"] = (2.0 * np.eye(8)).astype(np.float32)
    w["final_norm"] = np.full(8, 3.0, np.float32)
    m = oracle_model(shape, w, lm_head_bias=np.arange(8, dtype=np.float32))
    h = np.array([[1.0, -1.0, 1.0, -1.0, 1.0, -1.0, 1.0, -1.0]])
    m.rms_eps = 0.0
    assert np.allclose(orc.lm_head_logits(m, h), 6.0 * h + np.arange(8))


def test_bf16_widening_is_exact():
    bits = np.array([0x3F80, 0xBF80, 0x3C00, 0x0000, 0x4049], np.uint16)  # 1, -1, 2^-7, 0, 3.140625
    assert orc.widen(bits).tolist() == [1.0, -1.0, 2.0 ** -7, 0.0, 3.140625]
    x = np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -0.3], np.float32)   # ties go to even
    back = orc.widen(wl.f32_to_bf16_bits(x))
    assert back[0] == 1.0 and back[1] == 1.0 + 2 ** -6
    assert abs(back[2] + 0.3) < 2 ** -9 * 0.3 * 2


# ----------------------------------------------------------------------------- decode loop

def _table_predictor(table):
    """M(X) replaced by hand-built logits: table[b] is [s, V] for block b (same every step)."""
    def f(m, st, cfg):
        s = cfg.block_len
        n_rows = min(s, st.L_eff - (st.P + st.cur_block * s))
        return table[st.cur_block][:n_rows]
    return f


def _one_hot_logits(ids, V, peak=10.0):
    out = np.zeros((len(ids), V))
    out[np.arange(len(ids)), ids] = peak
    return out


def _toy_model(V=12):
    shape = small_shape(n_layers=0, vocab=V, mask_id=V - 1, eot_id=V - 2)
    return oracle_model(shape, {"layers": []})


def test_step_counts_never_and_always():
    """Filter 'never' -> one commit per step -> s steps per block (the paper's vanilla 32 at s=32);
    filter 'always' -> one step per block."""
    c = paper_constants()
    s, G, V = 32, 64, 12
    m = _toy_model(V)
    rng = np.random.default_rng(0)
    table = [_one_hot_logits(rng.integers(0, V - 2, s), V) for _ in range(G // s)]
    cfg = orc.DecodeConfig(block_len=s)
    never = orc.decode(m, const_filter(s, -50.0), [1, 2, 3], G, cfg, predictor=_table_predictor(table))
    assert never.steps == G and never.forced == G
    assert never.steps // (G // s) == int(c["vanilla_decodings_per_block_32"])
    always = orc.decode(m, const_filter(s, 50.0), [1, 2, 3], G, cfg, predictor=_table_predictor(table))
    assert always.steps == G // s and always.forced == 0
    want = np.concatenate([t.argmax(-1) for t in table])
    assert np.array_equal(never.response, want) and np.array_equal(always.response, want)
    off = orc.decode(m, const_filter(s, 50.0), [1, 2, 3], G,
                     orc.DecodeConfig(block_len=s, use_filter=False), predictor=_table_predictor(table))
    assert off.steps == G


def test_forced_commit_order_follows_confidence():
    s, V = 4, 12
    m = _toy_model(V)
    logits = np.zeros((s, V))
    for j, peak in enumerate([1.0, 4.0, 2.0, 3.0]):
        logits[j, j] = peak
    res = orc.decode(m, const_filter(s, -50.0), [0], s, orc.DecodeConfig(block_len=s),
                     predictor=_table_predictor([logits]))
    order = [int(np.where(r.unmask)[0][0]) for r in res.trace]
    assert order == [1, 3, 2, 0]


def test_eotp_truncates_and_stops_after_the_block():
    """Section 3.3 / Algorithm 3: [EoT] at generation index e -> out_len e+1, nothing after its block."""
    s, G, V, P = 8, 32, 12, 3
    m = _toy_model(V)
    ids = [np.full(s, 2), np.array([2, 2, 2, 2, 2, m.eot_id, 2, 2]), np.full(s, 3), np.full(s, 3)]
    table = [_one_hot_logits(i, V) for i in ids]
    cfg = orc.DecodeConfig(block_len=s)
    r = orc.decode(m, const_filter(s, 50.0), [1] * P, G, cfg, predictor=_table_predictor(table))
    e = s + 5
    assert r.out_len == e + 1 and r.steps == 2
    assert np.array_equal(r.response[:e], np.full(e, 2)) and (r.response[e:] == m.eot_id).all()
    r2 = orc.decode(m, const_filter(s, 50.0), [1] * P, G, orc.DecodeConfig(block_len=s, use_eotp=False),
                    predictor=_table_predictor(table))
    assert r2.steps == G // s and r2.out_len == G and (r2.response[2 * s:] == 3).all()


def test_eotp_keeps_denoising_positions_before_eot_with_shortened_input():
    """[EoT] committed at j=5 while j=2 is still masked: L_eff shrinks at once, the block
    finishes its earlier masks on the shortened sequence, later blocks never run."""
    s, G, V, P = 8, 16, 12, 4
    m = _toy_model(V)
    logits = _one_hot_logits(np.array([1, 1, 1, 1, 1, m.eot_id, 1, 1]), V, peak=8.0)
    logits[2, 1] = 0.5                      # low confidence at j=2
    pr, cf, _ = orc.confidence_head(logits)
    k, tau = 10.0, 0.96
    cut = 0.5 * (cf[2] + cf[0])
    filt = identity_filter(s, k, math.log(tau / (1 - tau)) - k * cut)
    seen = []

    def predictor(mm, st, cfg):
        n_rows = min(s, st.L_eff - (st.P + st.cur_block * s))
        seen.append((st.L_eff, n_rows))
        return logits[:n_rows]
    r = orc.decode(m, filt, [0] * P, G, orc.DecodeConfig(block_len=s), predictor=predictor)
    assert seen == [(P + G, s), (P + 6, 6)]
    assert r.steps == 2 and r.out_len == 6 and r.forced == 1
    assert r.trace[0].unmask.tolist() == [True, True, False, True, True, True, True, True]
    assert r.trace[1].filt_in[6:].tolist() == [1.0, 1.0]     # positions outside L_eff feed 1.0
    assert r.response[:6].tolist() == [1, 1, 1, 1, 1, m.eot_id]


def test_earliest_eot_wins():
    s, V = 8, 12
    m = _toy_model(V)
    logits = _one_hot_logits(np.array([1, 1, m.eot_id, 1, 1, m.eot_id, 1, 1]), V)
    r = orc.decode(m, const_filter(s, 50.0), [0], s, orc.DecodeConfig(block_len=s),
                   predictor=_table_predictor([logits]))
    assert r.out_len == 3 and (r.response[3:] == m.eot_id).all()


def test_committed_conf_mode_one_feeds_ones():
    s, V = 4, 12
    m = _toy_model(V)
    logits = _one_hot_logits(np.array([1, 2, 3, 4]), V, peak=1.0)
    cfg = orc.DecodeConfig(block_len=s, committed_conf_mode=1)
    r = orc.decode(m, const_filter(s, -50.0), [0], s, cfg, predictor=_table_predictor([logits]))
    assert r.trace[1].filt_in[0] == 1.0 and r.trace[0].filt_in[0] < 1.0
    r0 = orc.decode(m, const_filter(s, -50.0), [0], s, orc.DecodeConfig(block_len=s),
                    predictor=_table_predictor([logits]))
    assert r0.trace[1].filt_in[0] == r0.trace[0].filt_in[0]


def test_generation_length_must_be_a_multiple_of_block():
    with pytest.raises(ValueError):
        orc.decode(_toy_model(), const_filter(8, 0.0), [0], 12, orc.DecodeConfig(block_len=8))


def test_steps_are_bounded_on_a_real_tiny_model():
    shape = small_shape()
    w = wl.make_weights(shape, seed=3, final_norm_gain=wl.spread_gain(shape), threads=1)
    m = oracle_model(shape, w)
    s, G = 4, 16
    filt = wl.make_filter(s, seed=1)
    prompts = wl.make_prompts(2, 6, shape, seed=1)
    for p in prompts:
        r = orc.decode(m, filt, p, G, orc.DecodeConfig(block_len=s, use_eotp=False))
        assert G // s <= r.steps <= G
        assert len(r.response) == G


# ----------------------------------------------------------------------------- prefix cache

def _cache_models(n_layers):
    shape = small_shape(n_layers=n_layers)
    w = wl.make_weights(shape, seed=4, std=0.2, final_norm_gain=wl.spread_gain(shape), threads=1)
    return shape, oracle_model(shape, w)


def test_prefix_cache_is_exact_for_one_layer():
    """With one layer the prefix K/V depend only on the prefix embeddings, so the cached
    decode equals the uncached one."""
    shape, m = _cache_models(1)
    s, G = 4, 12
    filt = const_filter(s, -50.0)                             # one commit per step: most steps read the store
    p = wl.make_prompts(1, 5, shape, seed=3)[0]
    a = orc.decode(m, filt, p, G, orc.DecodeConfig(block_len=s), keep_logits=True)
    b = orc.decode(m, filt, p, G, orc.DecodeConfig(block_len=s, kv_cache=True), keep_logits=True)
    assert a.steps == b.steps > G // s and np.array_equal(a.response, b.response)
    for ra, rb in zip(a.trace, b.trace):
        assert np.allclose(ra.logits, rb.logits, atol=1e-10)


def test_prefix_cache_first_step_of_each_block_is_the_full_forward():
    shape, m = _cache_models(2)
    s, G = 4, 12
    filt = const_filter(s, -50.0)
    p = wl.make_prompts(1, 5, shape, seed=4)[0]
    st = orc.init_state(m, p, G)
    cfg_c = orc.DecodeConfig(block_len=s, kv_cache=True)
    cfg_u = orc.DecodeConfig(block_len=s)
    differs = False
    while not st.done:
        first = st.cache_block != st.cur_block
        S_b = st.P + st.cur_block * s
        full = orc.lm_head_logits(m, orc.forward_hidden(m, st.tokens[: st.L_eff])[S_b: S_b + s])
        rec = orc.denoise_step(m, filt, st, cfg_c, keep_logits=True)
        if first:
            assert np.allclose(rec.logits, full[: rec.n_rows], atol=1e-10)
        elif np.abs(rec.logits - full[: rec.n_rows]).max() > 1e-8:
            differs = True                       # stale prefix K/V: an approximation for NL > 1
    assert differs
    del cfg_u


def test_dual_cache_is_exact_for_one_layer_and_uses_block_rows_only():
    """One layer: K/V of a position depend on its own token alone, so reading the positions before
    AND after the block from the store changes nothing as long as their tokens are unchanged
    (they are: only the current block's positions are committed, and those rows are fresh)."""
    shape, m = _cache_models(1)
    s, G = 4, 12
    filt = const_filter(s, -50.0)
    p = wl.make_prompts(1, 5, shape, seed=3)[0]
    a = orc.decode(m, filt, p, G, orc.DecodeConfig(block_len=s), keep_logits=True)
    b = orc.decode(m, filt, p, G, orc.DecodeConfig(block_len=s, kv_cache=True, dual_cache=True), keep_logits=True)
    assert a.steps == b.steps and np.array_equal(a.response, b.response)
    assert a.steps > G // s                                   # some steps did read the store
    for ra, rb in zip(a.trace, b.trace):
        assert np.allclose(ra.logits, rb.logits, atol=1e-10)


def test_dual_cache_two_layers_brute_force_and_eotp():
    """Two layers: a later step of a block equals a by-hand evaluation in which layer 2's keys and
    values outside the block are the ones of the block's first step (stale), inside it fresh; the
    first step of each block is the full forward.  Runs with an [EoT] bias so the sequence is cut."""
    shape, m = _cache_models(2)
    s, G = 4, 12
    filt = const_filter(s, -50.0)
    cfg = orc.DecodeConfig(block_len=s, kv_cache=True, dual_cache=True)
    seed, bias, _ = find_eot_bias(m, shape, filt, G, cfg, 5, grid=np.arange(5.0, 120.0, 5.0))
    m.lm_head_bias = wl.make_eot_bias(shape, bias)
    p = wl.make_prompts(1, 5, shape, seed=seed)[0]
    st = orc.init_state(m, p, G)
    H, dh = m.n_heads, m.head_dim
    layers = m.weights["layers"]
    stale = None
    later = 0
    while not st.done:
        first = st.cache_block != st.cur_block
        S_b = st.P + st.cur_block * s
        L = st.L_eff
        n = min(s, L - S_b)
        # by hand: layer 1 over every position (its K/V do not depend on other tokens' state)
        x0 = orc.widen(m.weights["tok_emb"][st.tokens[:L]])
        pos = np.arange(L)
        kv1 = []
        x1 = orc.layer_forward(m, layers[0], x0, pos, kv_out=kv1)
        if first:
            kv2 = []
            x2 = orc.layer_forward(m, layers[1], x1, pos, kv_out=kv2)
            stale = (x0.copy(), kv1[0], kv2[0])
            want = orc.lm_head_logits(m, x2[S_b: S_b + n])
        else:
            later += 1
            x0_old, (k1o, v1o), (k2o, v2o) = stale
            blk = slice(S_b, S_b + n)
            # layer 1 on the block rows: keys of the other positions from the first step
            k1 = np.concatenate([k1o[:S_b], kv1[0][0][blk], k1o[S_b + n: L]])
            v1 = np.concatenate([v1o[:S_b], kv1[0][1][blk], v1o[S_b + n: L]])

            def block_layer(layer, xin, k_all, v_all):
                nn = orc.rmsnorm(xin, layer["norm1"], m.rms_eps)
                q = orc.rope(orc.linear(nn, layer["wqkv"])[:, : H * dh].reshape(n, H, dh), pos[blk], m.rope_theta)
                xo = xin + orc.linear(orc.attention(q, k_all, v_all).reshape(n, H * dh), layer["wo"])
                nn = orc.rmsnorm(xo, layer["norm2"], m.rms_eps)
                return xo + orc.linear(orc.silu(orc.linear(nn, layer["w_gate"])) * orc.linear(nn, layer["w_up"]), layer["w_down"])

            xb1 = block_layer(layers[0], x0[blk], k1, v1)
            nn = orc.rmsnorm(xb1, layers[1]["norm1"], m.rms_eps)
            qkv = orc.linear(nn, layers[1]["wqkv"])
            kf = orc.rope(qkv[:, H * dh: 2 * H * dh].reshape(n, H, dh), pos[blk], m.rope_theta)
            vf = qkv[:, 2 * H * dh:].reshape(n, H, dh)
            k2 = np.concatenate([k2o[:S_b], kf, k2o[S_b + n: L]])
            v2 = np.concatenate([v2o[:S_b], vf, v2o[S_b + n: L]])
            xb2 = block_layer(layers[1], xb1, k2, v2)
            want = orc.lm_head_logits(m, xb2)
        rec = orc.denoise_step(m, filt, st, cfg, keep_logits=True)
        assert rec.n_rows == n and np.allclose(rec.logits, want, atol=1e-9)
    assert later >= 2 and 0 <= st.eot_pos < G - 1            # cut before the end


def test_prefix_cache_two_layers_later_steps_by_hand_with_eotp():
    """Two layers, prefix rule: a later step of a block equals a by-hand evaluation of the rows from the
    block start to L_eff in which the keys and values of the positions BEFORE the block are those the
    block's first step stored, layer by layer (layer 1's equal the fresh ones, layer 2's are stale: they
    were computed when the block was still all masks), and the keys and values of the rows from the block
    start on are fresh.  An [EoT] bias cuts the sequence, so some later steps run on a shortened input."""
    shape, m = _cache_models(2)
    s, G = 4, 12
    filt = const_filter(s, -50.0)
    cfg = orc.DecodeConfig(block_len=s, kv_cache=True)
    seed, bias, _ = find_eot_bias(m, shape, filt, G, cfg, 5, grid=np.arange(5.0, 120.0, 5.0))
    m.lm_head_bias = wl.make_eot_bias(shape, bias)
    p = wl.make_prompts(1, 5, shape, seed=seed)[0]
    st = orc.init_state(m, p, G)
    H, dh = m.n_heads, m.head_dim
    layers = m.weights["layers"]
    stored = None
    later = shortened = stale_seen = 0
    while not st.done:
        first = st.cache_block != st.cur_block
        S_b = st.P + st.cur_block * s
        L = st.L_eff
        n = min(s, L - S_b)
        pos = np.arange(L)
        x0 = orc.widen(m.weights["tok_emb"][st.tokens[:L]])
        if first:
            kv1, kv2 = [], []
            x1 = orc.layer_forward(m, layers[0], x0, pos, kv_out=kv1)
            x2 = orc.layer_forward(m, layers[1], x1, pos, kv_out=kv2)
            stored = [(kv1[0][0][:S_b], kv1[0][1][:S_b]), (kv2[0][0][:S_b], kv2[0][1][:S_b])]
            stored_len = L
            want = orc.lm_head_logits(m, x2[S_b: S_b + n])
        else:
            later += 1
            shortened += int(L < stored_len)
            rows = slice(S_b, L)
            xr = x0[rows]
            for li, layer in enumerate(layers):
                nn = orc.rmsnorm(xr, layer["norm1"], m.rms_eps)
                qkv = orc.linear(nn, layer["wqkv"])
                T = L - S_b
                q = orc.rope(qkv[:, : H * dh].reshape(T, H, dh), pos[rows], m.rope_theta)
                kf = orc.rope(qkv[:, H * dh: 2 * H * dh].reshape(T, H, dh), pos[rows], m.rope_theta)
                vf = qkv[:, 2 * H * dh:].reshape(T, H, dh)
                k_all = np.concatenate([stored[li][0], kf])
                v_all = np.concatenate([stored[li][1], vf])
                xo = xr + orc.linear(orc.attention(q, k_all, v_all).reshape(T, H * dh), layer["wo"])
                nn = orc.rmsnorm(xo, layer["norm2"], m.rms_eps)
                xr = xo + orc.linear(orc.silu(orc.linear(nn, layer["w_gate"])) * orc.linear(nn, layer["w_up"]), layer["w_down"])
            want = orc.lm_head_logits(m, xr[:n])
            # layer 2's stored prefix keys really are stale: they differ from what a full forward gives now
            kv_now = []
            orc.forward_hidden(m, st.tokens[:L], kv_out=kv_now)
            assert np.allclose(kv_now[0][0][:S_b], stored[0][0], atol=1e-12)      # layer 1: token-only, never stale
            stale_seen += int(np.abs(kv_now[1][0][:S_b] - stored[1][0]).max() > 1e-8)
        rec = orc.denoise_step(m, filt, st, cfg, keep_logits=True)
        assert rec.n_rows == n and np.allclose(rec.logits, want, atol=1e-9)
    assert later >= 2 and stale_seen >= 1 and 0 <= st.eot_pos < G - 1


# ----------------------------------------------------------------------------- planted mistakes

def test_planted_mistakes_are_caught(monkeypatch):
    """A pin is only worth something if a plausible slip trips it."""
    rng = np.random.default_rng(8)
    q, k, v = (rng.normal(size=(4, 1, 8)) for _ in range(3))
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2) for a in (q, k, v))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(1, 0, 2).numpy()

    def causal_attention(q, k, v):
        out = np.empty_like(q)
        for t in range(len(q)):
            out[t:t + 1] = orc.attention(q[t:t + 1], k[:t + 1], v[:t + 1])
        return out
    assert not np.allclose(causal_attention(q, k, v), want, atol=1e-6)

    def rope_wrong_sign(x, pos, theta):
        return orc.rope(x, -pos, theta)
    x = rng.normal(size=(2, 1, 4))
    z = complex(x[1, 0, 0], x[1, 0, 2]) * complex(math.cos(1.0), math.sin(1.0))
    assert abs(rope_wrong_sign(x, np.array([0, 1]), 1e4)[1, 0, 0] - z.real) > 1e-3
    assert abs(orc.rope(x, np.array([0, 1]), 1e4)[1, 0, 0] - z.real) < 1e-12

    # a non-strict threshold would commit position 0 without the fallback
    p = np.array([0.5, 0.9])
    un, forced = orc.unmask_rule(p, p, np.ones(2, bool), 0.5)
    assert un.tolist() == [False, True] and not forced


def test_linear_is_x_times_w_transposed():
    rng = np.random.default_rng(9)
    x = rng.normal(size=(3, 5))
    w = rng.normal(size=(4, 5)).astype(np.float32)
    y = orc.linear(x, w)
    assert y.shape == (3, 4)
    for t in range(3):
        for o in range(4):
            assert y[t, o] == pytest.approx(sum(x[t, i] * float(w[o, i]) for i in range(5)), abs=1e-13)
    assert np.array_equal(orc.linear(x, np.eye(5, dtype=np.float32)), x)


# ----------------------------------------------------------------------------- comparison policies

def test_confidence_rule_closed_form_and_vanilla_limit():
    """Fixed-threshold policy on one-hot logits: conf = e^a / (e^a + V - 1) in closed form, so which
    positions pass 0.9 is known by hand; with the threshold at 1 nothing passes and the decode takes
    s steps per block (Section 3.1's vanilla count), ending in the same tokens."""
    s, V = 8, 12
    m = _toy_model(V)
    peaks = np.array([6.0, 1.0, 5.0, 2.0, 7.0, 0.5, 4.0, 3.0])
    ids = np.array([3, 1, 4, 1, 5, 9, 2, 6])
    logits = np.zeros((s, V))
    logits[np.arange(s), ids] = peaks
    conf = np.exp(peaks) / (np.exp(peaks) + V - 1)
    first = conf > 0.9
    assert first.sum() == 3                                   # peaks 6, 5, 7 (4 gives 0.832)
    cfg = orc.DecodeConfig(block_len=s, rule="confidence", conf_threshold=0.9)
    r = orc.decode(m, const_filter(s, 50.0), [0], s, cfg, predictor=_table_predictor([logits]))
    assert np.array_equal(r.trace[0].unmask, first) and not r.trace[0].forced
    assert (r.trace[0].p == 0).all()                          # the filter takes no part
    # afterwards nothing passes: one forced commit per step, highest confidence first
    rest = [int(np.where(t.unmask)[0][0]) for t in r.trace[1:]]
    assert rest == [6, 7, 3, 1, 5] and all(t.forced for t in r.trace[1:])
    assert r.steps == 1 + 5 and np.array_equal(r.response, ids)
    van = orc.decode(m, None, [0], s, orc.DecodeConfig(block_len=s, rule="confidence", conf_threshold=1.0),
                     predictor=_table_predictor([logits]))
    assert van.steps == s and van.forced == s and np.array_equal(van.response, ids)
    off = orc.decode(m, None, [0], s, orc.DecodeConfig(block_len=s, use_filter=False),
                     predictor=_table_predictor([logits]))
    assert [np.where(t.unmask)[0][0] for t in van.trace] == [np.where(t.unmask)[0][0] for t in off.trace]


def _chain_predictor(ref, V, wrong):
    """Predicts the reference at block position j only once position j-1 of the block is committed
    (position 0 at once); elsewhere it predicts `wrong`."""
    def f(m, st, cfg):
        s = cfg.block_len
        g0 = st.cur_block * s
        ids = np.full(s, wrong)
        for j in range(s):
            if j == 0 or not st.masked[g0 + j - 1]:
                ids[j] = ref[g0 + j]
        return _one_hot_logits(ids, V)
    return f


def test_egp_unmasks_on_first_match_and_reproduces_the_reference():
    """Section 3.1: a position is committed at the first step whose prediction equals the reference,
    never earlier and never later; the response is the reference."""
    s, G, V = 4, 8, 12
    m = _toy_model(V)
    ref = np.array([1, 2, 3, 4, 5, 6, 7, 8])
    cfg = orc.DecodeConfig(block_len=s, rule="egp")
    # (a) every prediction right at once: one step per block
    table = [_one_hot_logits(ref[b * s:(b + 1) * s], V) for b in range(G // s)]
    r = orc.decode(m, None, [0], G, cfg, predictor=_table_predictor(table), ref=ref)
    assert r.steps == G // s and r.forced == 0 and np.array_equal(r.response, ref)
    # (b) a prediction turns right only after its left neighbour is committed: step k of a block
    #     commits position k alone, no fallback is needed, the labels are Algorithm 1's
    r = orc.decode(m, None, [0], G, cfg, predictor=_chain_predictor(ref, V, wrong=0), ref=ref)
    assert r.steps == G and r.forced == 0 and np.array_equal(r.response, ref)
    for k, t in enumerate(r.trace):
        want = np.zeros(s, bool)
        want[k % s] = True
        assert np.array_equal(t.unmask, want)
        labels = orc.egp_labels(t.pred, ref[t.block * s:(t.block + 1) * s])
        assert np.array_equal(labels[k % s:], want[k % s:])   # right of k: still wrong
        assert labels[:k % s + 1].all()                        # committed positions stay right
    with pytest.raises(ValueError):
        orc.decode(m, None, [0], G, cfg, predictor=_table_predictor(table))


def test_egp_fallback_commits_the_reference_token():
    """Where the model never predicts the reference, the loop still ends and still returns the
    reference: each such step commits the most confident masked position with its reference token."""
    s, V = 4, 12
    m = _toy_model(V)
    ref = np.array([1, 2, 3, 4])
    ids = np.array([1, 9, 3, 9])                 # positions 1 and 3 never match
    logits = np.zeros((s, V))
    logits[np.arange(s), ids] = [5.0, 2.0, 5.0, 3.0]
    r = orc.decode(m, None, [0], s, orc.DecodeConfig(block_len=s, rule="egp"),
                   predictor=_table_predictor([logits]), ref=ref)
    assert np.array_equal(r.trace[0].unmask, [True, False, True, False]) and not r.trace[0].forced
    assert [int(np.where(t.unmask)[0][0]) for t in r.trace[1:]] == [3, 1]
    assert r.steps == 3 and r.forced == 2 and np.array_equal(r.response, ref)


def test_egp_with_the_models_own_answer_as_reference_skips_repeats():
    """Section 3.1 defines the reference as the answer of the standard decode; under EGP with that
    reference the small transformer needs no more steps than the standard decode and every
    step's commits are exactly the masked positions where pred == reference."""
    shape = small_shape()
    w = wl.make_weights(shape, seed=5)
    m = oracle_model(shape, w)
    s, G = 8, 16
    prompt = wl.make_prompts(1, 6, shape, seed=1)[0]
    van = orc.decode(m, None, prompt, G, orc.DecodeConfig(block_len=s, use_filter=False, use_eotp=False))
    egp = orc.decode(m, None, prompt, G, orc.DecodeConfig(block_len=s, rule="egp", use_eotp=False),
                     ref=van.response)
    assert egp.steps <= van.steps and np.array_equal(egp.response, van.response)
    masked = np.ones(G, bool)
    for t in egp.trace:
        blk = slice(t.block * s, (t.block + 1) * s)
        if not t.forced:
            assert np.array_equal(t.unmask, masked[blk] & orc.egp_labels(t.pred, van.response[blk]))
        masked[blk] &= ~t.unmask
    assert not masked.any()


# ----------------------------------------------------------------------------- filter training (Algorithm 1)

def _train_data(s=8, n=40, seed=0):
    rng = np.random.default_rng(seed)
    C = rng.uniform(0.0, 1.0, size=(n, s))
    Y = (C + 0.15 * rng.normal(size=(n, s)) > 0.6).astype(np.float64)      # high confidence -> mostly "unmask"
    return C, Y


def test_bce_at_zero_logits_is_log_two_and_matches_the_definition():
    """Eq. 5/6: with p = 1/2 everywhere the loss is ln 2 = 0.693 (the paper's curve starts at 0.68);
    the overflow-free form equals the printed definition where that one is finite."""
    y = np.array([[0.0, 1.0, 1.0, 0.0]])
    assert abs(orc.bce_with_logits(np.zeros((1, 4)), y) - math.log(2.0)) < 1e-15
    z = np.array([[-3.0, 0.5, 2.0, 7.0]])
    p = 1.0 / (1.0 + np.exp(-z))
    want = -np.mean(y * np.log(p) + (1 - y) * np.log(1 - p))
    assert abs(orc.bce_with_logits(z, y) - want) < 1e-12
    assert np.isfinite(orc.bce_with_logits(np.array([[800.0, -800.0]]), np.array([[0.0, 1.0]])))


def test_filter_gradients_match_central_differences():
    s = 6
    C, Y = _train_data(s, 12, seed=1)
    filt = {k: v.astype(np.float64) for k, v in wl.make_filter(s, seed=5).items()}
    loss, g = orc.filter_loss_and_grads(filt, C, Y)
    eps = 1e-6
    rng = np.random.default_rng(2)
    for k in ("w1", "b1", "w2", "b2"):
        for _ in range(6):
            idx = tuple(rng.integers(0, n) for n in filt[k].shape)
            up = {a: b.copy() for a, b in filt.items()}
            dn = {a: b.copy() for a, b in filt.items()}
            up[k][idx] += eps
            dn[k][idx] -= eps
            num = (orc.filter_loss_and_grads(up, C, Y)[0] - orc.filter_loss_and_grads(dn, C, Y)[0]) / (2 * eps)
            assert abs(num - g[k][idx]) < 1e-7, (k, idx, num, g[k][idx])


@pytest.mark.parametrize("batch_size", [0, 16])
def test_training_matches_torch_adamw(batch_size):
    """The same network, loss and optimiser built from torch's CPU library (nn.Linear,
    binary_cross_entropy_with_logits, optim.AdamW) in fp64: parameters and loss curve agree."""
    s = 8
    C, Y = _train_data(s, 40, seed=3)
    f0 = wl.make_filter(s, seed=7)
    epochs = 25
    filt, losses = orc.train_filter(f0, C, Y, epochs, lr=1e-2, weight_decay=0.05, batch_size=batch_size)
    l1, l2 = torch.nn.Linear(s, s).double(), torch.nn.Linear(s, s).double()
    with torch.no_grad():
        l1.weight.copy_(torch.from_numpy(f0["w1"].astype(np.float64))); l1.bias.copy_(torch.from_numpy(f0["b1"].astype(np.float64)))
        l2.weight.copy_(torch.from_numpy(f0["w2"].astype(np.float64))); l2.bias.copy_(torch.from_numpy(f0["b2"].astype(np.float64)))
    opt = torch.optim.AdamW(list(l1.parameters()) + list(l2.parameters()), lr=1e-2, betas=(0.9, 0.999), eps=1e-8,
                            weight_decay=0.05)
    tc, ty = torch.from_numpy(C), torch.from_numpy(Y)
    bs = len(C) if batch_size == 0 else batch_size
    ref_losses = []
    for _ in range(epochs):
        for lo in range(0, len(C), bs):
            opt.zero_grad()
            z = l2(torch.relu(l1(tc[lo: lo + bs])))
            loss = torch.nn.functional.binary_cross_entropy_with_logits(z, ty[lo: lo + bs])
            loss.backward()
            opt.step()
            ref_losses.append(float(loss.detach()))
    assert np.allclose(losses, ref_losses, rtol=0, atol=1e-10)
    assert np.allclose(filt["w1"], l1.weight.detach().numpy(), atol=1e-9)
    assert np.allclose(filt["b1"], l1.bias.detach().numpy(), atol=1e-9)
    assert np.allclose(filt["w2"], l2.weight.detach().numpy(), atol=1e-9)
    assert np.allclose(filt["b2"], l2.bias.detach().numpy(), atol=1e-9)
    assert losses[-1] < losses[0]


def test_first_adamw_step_moves_every_parameter_by_lr():
    """Closed form: at t = 1 the bias-corrected ratio m_hat / sqrt(v_hat) is sign(g), so without
    weight decay each parameter with a non-zero gradient moves by lr (up to eps)."""
    p = np.array([0.5, -0.25, 2.0])
    g = np.array([0.3, -4.0, 1e-3])
    q, m, v = orc.adamw_step(p, g, np.zeros(3), np.zeros(3), 1, 1e-3, 0.9, 0.999, 1e-8, 0.0)
    assert np.allclose(q, p - 1e-3 * np.sign(g), atol=1e-7)
    q2, _, _ = orc.adamw_step(p, g, np.zeros(3), np.zeros(3), 1, 1e-3, 0.9, 0.999, 1e-8, 0.1)
    assert np.allclose(q2 - q, -1e-3 * 0.1 * p, atol=1e-12)     # decay is decoupled from the gradient


def test_egp_samples_are_algorithm_one_targets():
    """Stage 1: the samples of an EGP decode are the filter inputs of its steps and pred == ref."""
    s, G, V = 4, 8, 12
    m = _toy_model(V)
    ref = np.array([1, 2, 3, 4, 5, 6, 7, 8])
    r = orc.decode(m, None, [0], G, orc.DecodeConfig(block_len=s, rule="egp"),
                   predictor=_chain_predictor(ref, V, wrong=0), ref=ref)
    C, Y = orc.egp_samples(r.trace, ref, s)
    assert C.shape == Y.shape == (G, s)
    for k in range(G):
        want = np.zeros(s)
        want[: k % s + 1] = 1.0                    # committed positions and the one that just turned right
        assert np.array_equal(Y[k], want)
        assert np.array_equal(C[k], r.trace[k].filt_in)
    # the trained filter separates the two groups of this toy: its loss falls well below ln 2
    f0 = wl.make_filter(s, seed=1)
    _, losses = orc.train_filter(f0, C, Y, 300, lr=1e-2)
    assert losses[0] > 0.3 and losses[-1] < 0.6 * losses[0]


# ----------------------------------------------------------------------------- filter depth (Section 4.4)

def test_filter_depth_variants():
    """One layer is an affine map; the two-entry list equals the named two-layer filter; four layers
    equal torch's Sequential of Linear / ReLU in fp64."""
    s = 6
    rng = np.random.default_rng(3)
    c = rng.uniform(size=s)
    f2 = wl.make_filter(s, seed=2)
    two = {"layers": [(f2["w1"], f2["b1"]), (f2["w2"], f2["b2"])]}
    assert np.allclose(orc.filter_logits(two, c), orc.filter_logits(f2, c), atol=0)
    one = {"layers": [(f2["w1"], f2["b1"])]}
    assert np.allclose(orc.filter_logits(one, c), f2["w1"].astype(np.float64) @ c + f2["b1"], atol=1e-15)
    ws = [(rng.normal(size=(s, s)), rng.normal(size=s)) for _ in range(4)]
    mods = []
    for k, (w, b) in enumerate(ws):
        lin = torch.nn.Linear(s, s).double()
        with torch.no_grad():
            lin.weight.copy_(torch.from_numpy(w)); lin.bias.copy_(torch.from_numpy(b))
        mods += ([torch.nn.ReLU()] if k else []) + [lin]
    want = torch.nn.Sequential(*mods)(torch.from_numpy(c)).detach().numpy()
    assert np.allclose(orc.filter_logits({"layers": ws}, c), want, atol=1e-12)
    # parameter counts of the three depths at s = 32: 1,056 / 2,112 (the printed count) / 4,224
    assert [k * (32 * 32 + 32) for k in (1, 2, 4)] == [1056, int(paper_constants()["filter_params_at_block_32"]), 4224]


@pytest.mark.parametrize("depth", [1, 2, 4])
def test_depth_variant_training_matches_torch_and_the_two_layer_form(depth):
    """Backpropagation through 1, 2 and 4 layers against torch autograd + optim.AdamW in fp64; at depth 2 the
    list form also reproduces train_filter."""
    s = 6
    C, Y = _train_data(s, 30, seed=11)
    rng = np.random.default_rng(depth)
    layers0 = [((rng.normal(size=(s, s)) * 0.5).astype(np.float32), (0.1 * rng.normal(size=s)).astype(np.float32))
               for _ in range(depth)]
    epochs = 20
    got, losses = orc.train_filter_layers(layers0, C, Y, epochs, lr=1e-2, weight_decay=0.02, batch_size=16)
    mods = []
    lins = []
    for k, (w, b) in enumerate(layers0):
        lin = torch.nn.Linear(s, s).double()
        with torch.no_grad():
            lin.weight.copy_(torch.from_numpy(w.astype(np.float64))); lin.bias.copy_(torch.from_numpy(b.astype(np.float64)))
        lins.append(lin)
        mods += ([torch.nn.ReLU()] if k else []) + [lin]
    net = torch.nn.Sequential(*mods)
    opt = torch.optim.AdamW(net.parameters(), lr=1e-2, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.02)
    tc, ty = torch.from_numpy(C), torch.from_numpy(Y)
    ref_losses = []
    for _ in range(epochs):
        for lo in range(0, len(C), 16):
            opt.zero_grad()
            loss = torch.nn.functional.binary_cross_entropy_with_logits(net(tc[lo: lo + 16]), ty[lo: lo + 16])
            loss.backward()
            opt.step()
            ref_losses.append(float(loss.detach()))
    assert np.allclose(losses, ref_losses, rtol=0, atol=1e-10)
    for (w, b), lin in zip(got, lins):
        assert np.allclose(w, lin.weight.detach().numpy(), atol=1e-9) and np.allclose(b, lin.bias.detach().numpy(), atol=1e-9)
    if depth == 2:
        f0 = {"w1": layers0[0][0], "b1": layers0[0][1], "w2": layers0[1][0], "b2": layers0[1][1]}
        two, l2 = orc.train_filter(f0, C, Y, epochs, lr=1e-2, weight_decay=0.02, batch_size=16)
        assert np.allclose(l2, losses, atol=1e-12) and np.allclose(two["w2"], got[1][0], atol=1e-12)
