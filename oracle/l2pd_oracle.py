"""CPU oracle for Learn2PD decoding: plain numpy, fp64, slow and direct.

TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA path is compared
with; it is imported by the tests, by the smoke check and by the benchmark's CPU
baseline leg, never by the product.  It shares no code with the CUDA path and
imports nothing from it: inputs arrive as numpy arrays.

What it follows
---------------
* Decode loop: the paper's inference procedure (Algorithm 2) with the
  end-of-text break of the updated procedure (Algorithm 3): for each prompt,
  X = prompt ++ [MASK]^G; blocks of s positions left to right; inside a block
  repeat  conf, pre = M(X); p = sigmoid(f_theta(conf)); unmask where p > tau
  until the block has no masked position.
* Greedy prediction and confidence: Eq. 3 (argmax over the vocabulary) and
  Eq. 4 (model probability of that argmax).
* Filter f_theta: Section 3.2 / Section 4.1: a two-layer MLP over the block's s
  confidences; 2*(s*s+s) parameters (2,112 at s = 32); sigmoid on its output.
* EoTP: Section 3.3: when [EoT] is unmasked, later positions are discarded and
  the shortened sequence is the next step's input.
* The mask predictor M is not defined in the paper.  It is a LLaDA-style
  bidirectional transformer: pre-norm residual blocks with RMSNorm, rotary
  position embedding on q and k (half-split pairing), multi-head attention with
  NO causal mask, SwiGLU MLP, final RMSNorm and an untied LM head.

All arithmetic is fp64 on the stored weight values (bf16 bit patterns or fp32
are widened exactly); nothing is rounded between stages.  Matrix products use
numpy's matmul as a library step; there is no tiling, fusion or reordering.

Readings of the paper that no printed value pins ("parity unpinned" for these
choices; the arithmetic of every function below is pinned by tests):
  * RoPE pairing (i, i + dh/2) and angle pos * theta^(-2i/dh);
  * ReLU as the filter's hidden activation;
  * the filter sees the model's recomputed confidence at block positions that
    are already committed (mode 0) — or 1.0 there (mode 1);
  * progress fallback: if no masked position passes the threshold the masked
    position with the highest confidence is committed;
  * EoTP truncates at the committing step and decoding continues until the
    masked positions before [EoT] in the current block are done.
  * KV caches (Section 4.3 names a prefix cache and a dual cache and gives no rule):
    the first step of a block is a full forward pass that stores K (rotated) and V
    per layer; the block's other steps recompute rows from the block start to the
    end of the sequence against stored prefix ++ fresh keys (prefix cache), or only
    the block's own rows against stored prefix ++ fresh block ++ stored positions
    after the block (dual cache).  Stored entries go stale as tokens are committed:
    both are approximations for more than one layer and exact for one.

Comparison policies (the strategies the paper measures Learn2PD against; same loop,
another test inside it), selected by DecodeConfig.rule:
  * "confidence": a masked position is committed when its confidence (Eq. 4)
    exceeds a fixed threshold (the confidence-threshold parallel decoding the
    related-work section cites); with the threshold at 1 nothing passes and the
    fallback commits one position per step, i.e. low-confidence remasking with one
    token per step, the paper's vanilla decoding (Section 3.1: s steps per block);
  * "egp": Extremely Greedy Parallel, Section 3.1: unmask position j if and only
    if the prediction equals the reference answer r_j (Algorithm 1's test).
    Unpinned reading: when no masked position of the block matches, the masked
    position with the highest confidence is committed WITH ITS REFERENCE TOKEN, so
    that the loop ends and the response equals the reference, as the section says
    of the oracle.  egp_labels() gives Algorithm 1's targets y_j for a step.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np


# ----------------------------------------------------------------------------
# storage -> fp64

def widen(w: np.ndarray) -> np.ndarray:
    """Exact widening of stored values to fp64 (uint16 arrays are bf16 bit patterns)."""
    if w.dtype == np.uint16:
        return (w.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return w.astype(np.float64)


@dataclass
class Model:
    """Architecture constants plus stored weights (layout as documented in forward_hidden)."""
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    rms_eps: float
    rope_theta: float
    mask_id: int
    eot_id: int
    weights: Dict[str, object]
    lm_head_bias: Optional[np.ndarray] = None  # [V] added to the logits, or None


# ----------------------------------------------------------------------------
# transformer pieces (the mask predictor M)

def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """y = x * g / sqrt(mean(x^2) + eps), row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x * widen(gain) / np.sqrt(ms + eps)


def linear(x: np.ndarray, w: np.ndarray) -> np.ndarray:
    """y = x W^T for a weight stored [out, in] (library matmul on the widened values)."""
    return x @ widen(w).T


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding on x[T, H, dh] at integer positions pos[T].

    Pair (i, i + dh/2), i < dh/2, is rotated by the angle pos * theta^(-2i/dh).
    """
    dh = x.shape[-1]
    half = dh // 2
    i = np.arange(half, dtype=np.float64)
    ang = pos.astype(np.float64)[:, None] * theta ** (-2.0 * i / dh)[None, :]  # [T, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    """Bidirectional multi-head attention: softmax(q k^T / sqrt(dh)) v per head, no mask.

    q[Tq, H, dh], k[Tk, H, dh], v[Tk, H, dh] -> [Tq, H, dh].
    """
    dh = q.shape[-1]
    out = np.empty_like(q)
    for h in range(q.shape[1]):
        sc = q[:, h, :] @ k[:, h, :].T / np.sqrt(dh)
        sc = sc - sc.max(axis=-1, keepdims=True)
        w = np.exp(sc)
        w = w / w.sum(axis=-1, keepdims=True)
        out[:, h, :] = w @ v[:, h, :]
    return out


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def layer_forward(m: Model, layer: Dict[str, np.ndarray], x: np.ndarray, pos: np.ndarray,
                  k_prefix: Optional[np.ndarray] = None, v_prefix: Optional[np.ndarray] = None,
                  kv_out: Optional[list] = None,
                  k_suffix: Optional[np.ndarray] = None, v_suffix: Optional[np.ndarray] = None) -> np.ndarray:
    """One pre-norm block on rows x[T, d] at positions pos[T].

    k_prefix / v_prefix [Tp, H, dh] (k already rotated) are put before this
    call's keys and values (prefix-cache rule), k_suffix / v_suffix [Ts, H, dh]
    after them (dual-cache rule).  kv_out, if a list, receives (k_rotated, v) of
    this call's rows.
    """
    H, dh = m.n_heads, m.head_dim
    T = x.shape[0]
    n = rmsnorm(x, layer["norm1"], m.rms_eps)
    qkv = linear(n, layer["wqkv"])                     # [T, 3*H*dh]: q rows, then k, then v
    q = qkv[:, : H * dh].reshape(T, H, dh)
    k = qkv[:, H * dh: 2 * H * dh].reshape(T, H, dh)
    v = qkv[:, 2 * H * dh:].reshape(T, H, dh)
    q = rope(q, pos, m.rope_theta)
    k = rope(k, pos, m.rope_theta)
    if kv_out is not None:
        kv_out.append((k, v))
    if k_prefix is not None:
        k = np.concatenate([k_prefix, k], axis=0)
        v = np.concatenate([v_prefix, v], axis=0)
    if k_suffix is not None:
        k = np.concatenate([k, k_suffix], axis=0)
        v = np.concatenate([v, v_suffix], axis=0)
    a = attention(q, k, v).reshape(T, H * dh)
    x = x + linear(a, layer["wo"])
    n = rmsnorm(x, layer["norm2"], m.rms_eps)
    h = silu(linear(n, layer["w_gate"])) * linear(n, layer["w_up"])
    return x + linear(h, layer["w_down"])


def forward_hidden(m: Model, tokens: np.ndarray, pos0: int = 0,
                   prefix_kv: Optional[list] = None, kv_out: Optional[list] = None,
                   suffix_kv: Optional[list] = None) -> np.ndarray:
    """Residual stream after the last layer for `tokens` placed at positions pos0...

    Weights: tok_emb[V,d], layers[l]{wqkv[3Hdh,d], wo[d,Hdh], w_gate[F,d], w_up[F,d],
    w_down[d,F], norm1[d], norm2[d]}, final_norm[d], lm_head[V,d]; all [out, in].
    prefix_kv[l] = (k, v) of earlier positions for layer l, or None; suffix_kv[l] the
    same for later positions.
    kv_out, if a list, receives one (k, v) per layer for this call's rows.
    """
    w = m.weights
    x = widen(w["tok_emb"][np.asarray(tokens, dtype=np.int64)])
    pos = pos0 + np.arange(len(tokens))
    for l, layer in enumerate(w["layers"]):
        kp, vp = (prefix_kv[l] if prefix_kv is not None else (None, None))
        ks, vs = (suffix_kv[l] if suffix_kv is not None else (None, None))
        x = layer_forward(m, layer, x, pos, kp, vp, kv_out, ks, vs)
    return x


def lm_head_logits(m: Model, hidden_rows: np.ndarray) -> np.ndarray:
    """Final RMSNorm then the LM head (+ optional bias) on the given rows -> [R, V]."""
    n = rmsnorm(hidden_rows, m.weights["final_norm"], m.rms_eps)
    logits = linear(n, m.weights["lm_head"])
    if m.lm_head_bias is not None:
        logits = logits + widen(m.lm_head_bias)[None, :]
    return logits


# ----------------------------------------------------------------------------
# confidence head, filter, unmasking rule, EoTP

def confidence_head(logits: np.ndarray):
    """Eq. 3: pred = argmax_v logits (lowest id on ties); Eq. 4: conf = softmax prob of pred.

    Also returns the gap between the two largest logits of each row.
    """
    pred = np.argmax(logits, axis=-1)
    top = np.take_along_axis(logits, pred[:, None], axis=-1)[:, 0]
    lse = top + np.log(np.sum(np.exp(logits - top[:, None]), axis=-1))
    conf = np.exp(top - lse)
    if logits.shape[1] > 1:
        part = np.partition(logits, -2, axis=-1)
        gap = part[:, -1] - part[:, -2]
    else:
        gap = np.full(len(pred), np.inf)
    return pred.astype(np.int64), conf, gap


def filter_logits(filt: Dict[str, np.ndarray], conf_block: np.ndarray) -> np.ndarray:
    """f_theta: z = W2 relu(W1 c + b1) + b2 on the block's s confidences (Section 3.2).

    The depth study of Section 4.4 (one, two and four layers) uses filt["layers"], a list of
    (W, b) pairs of Linear(s, s) layers with ReLU between consecutive layers and none after the last.
    """
    if "layers" in filt:
        h = conf_block
        for k, (w, b) in enumerate(filt["layers"]):
            if k > 0:
                h = np.maximum(h, 0.0)
            h = widen(w) @ h + widen(b)
        return h
    h = widen(filt["w1"]) @ conf_block + widen(filt["b1"])
    h = np.maximum(h, 0.0)
    return widen(filt["w2"]) @ h + widen(filt["b2"])


def sigmoid(z: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-z))


def unmask_rule(p: np.ndarray, conf: np.ndarray, masked: np.ndarray, tau: float):
    """Algorithm 2, the `if` inside the while loop: a masked position j leaves the
    mask set when p_j > tau (strict).  If none does, the masked position with the
    highest confidence is committed (lowest index on ties) so the loop advances.

    Returns (unmask[s] bool, forced bool).  `masked` marks positions that may be committed.
    """
    unmask = masked & (p > tau)
    forced = False
    if masked.any() and not unmask.any():
        cand = np.where(masked)[0]
        j = cand[np.argmax(conf[cand])]
        unmask[j] = True
        forced = True
    return unmask, forced


def confidence_rule(conf: np.ndarray, masked: np.ndarray, threshold: float):
    """Fixed-threshold policy: commit masked positions whose confidence exceeds the threshold
    (strict); same progress fallback as unmask_rule."""
    return unmask_rule(conf, conf, masked, threshold)


def egp_labels(pred: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """Algorithm 1: y_j = 1 where the prediction equals the reference token, else 0."""
    return np.asarray(pred) == np.asarray(ref)


def egp_rule(pred: np.ndarray, ref: np.ndarray, conf: np.ndarray, masked: np.ndarray):
    """Section 3.1 (EGP): unmask j iff pred_j == r_j.  Returns (unmask, forced); on a forced step the
    caller commits the reference token at the chosen position (see the module header)."""
    unmask = masked & egp_labels(pred, ref)
    forced = False
    if masked.any() and not unmask.any():
        cand = np.where(masked)[0]
        unmask[cand[np.argmax(conf[cand])]] = True
        forced = True
    return unmask, forced


@dataclass
class DecodeConfig:
    block_len: int
    tau: float = 0.96
    rule: str = "filter"         # "filter" (Learn2PD, Algorithm 2), "confidence", "egp"
    conf_threshold: float = 0.9  # rule "confidence"
    use_filter: bool = True      # False: nothing passes the threshold (one token per step)
    use_eotp: bool = True
    kv_cache: bool = False       # block-level prefix cache
    dual_cache: bool = False     # with kv_cache: the positions after the block are cached as well
    committed_conf_mode: int = 0  # 0: model confidence at committed positions, 1: 1.0 there


@dataclass
class SeqState:
    tokens: np.ndarray           # [P + G]
    masked: np.ndarray           # [G] bool: still in some block's mask set
    P: int
    G: int
    L_eff: int
    cur_block: int = 0
    done: bool = False
    steps: int = 0
    forced: int = 0
    eot_pos: int = -1            # generation index of the earliest committed [EoT], -1 if none
    prefix_kv: Optional[list] = None     # prefix cache of the current block
    all_kv: Optional[list] = None        # dual cache: K, V of every position at the block's first step
    cache_block: int = -1                # block the cache was filled for


@dataclass
class StepRecord:
    block: int
    L_eff_in: int
    n_rows: int
    pred: np.ndarray
    conf: np.ndarray
    gap: np.ndarray
    filt_in: np.ndarray
    p: np.ndarray
    unmask: np.ndarray
    forced: bool
    logits: Optional[np.ndarray] = None


def init_state(m: Model, prompt: Sequence[int], G: int) -> SeqState:
    """Algorithm 2: X <- concat(prompt, [MASK]^G); every generation position is masked."""
    prompt = np.asarray(prompt, dtype=np.int64)
    P = len(prompt)
    tokens = np.concatenate([prompt, np.full(G, m.mask_id, dtype=np.int64)])
    return SeqState(tokens=tokens, masked=np.ones(G, dtype=bool), P=P, G=G, L_eff=P + G)


def block_logits(m: Model, st: SeqState, cfg: DecodeConfig) -> np.ndarray:
    """conf, pre = M(X): logits of the current block's rows that are inside L_eff."""
    s = cfg.block_len
    S_b = st.P + st.cur_block * s
    n_rows = min(s, st.L_eff - S_b)
    if not cfg.kv_cache:
        x = forward_hidden(m, st.tokens[: st.L_eff])
        return lm_head_logits(m, x[S_b: S_b + n_rows])
    if st.cache_block != st.cur_block:
        # first step of the block: full forward; keep K (rotated) and V of positions [0, S_b)
        kv: list = []
        x = forward_hidden(m, st.tokens[: st.L_eff], kv_out=kv)
        st.prefix_kv = [(k[:S_b].copy(), v[:S_b].copy()) for (k, v) in kv]
        st.all_kv = kv if cfg.dual_cache else None
        st.cache_block = st.cur_block
        return lm_head_logits(m, x[S_b: S_b + n_rows])
    if cfg.dual_cache:
        # later steps, dual cache: only the block's rows; keys = cached prefix ++ fresh block rows ++
        # cached positions after the block (those still inside L_eff)
        end = S_b + n_rows
        suffix = [(k[end: st.L_eff], v[end: st.L_eff]) for (k, v) in st.all_kv]
        x = forward_hidden(m, st.tokens[S_b: end], pos0=S_b, prefix_kv=st.prefix_kv, suffix_kv=suffix)
        return lm_head_logits(m, x)
    # later steps of the block: only rows [S_b, L_eff), keys = cached prefix ++ fresh rows
    x = forward_hidden(m, st.tokens[S_b: st.L_eff], pos0=S_b, prefix_kv=st.prefix_kv)
    return lm_head_logits(m, x[:n_rows])


def decide(m: Model, filt: Dict[str, np.ndarray], st: SeqState, cfg: DecodeConfig,
           pred: np.ndarray, conf: np.ndarray, gap: Optional[np.ndarray] = None,
           logits: Optional[np.ndarray] = None, ref: Optional[np.ndarray] = None) -> StepRecord:
    """Everything after M(X) in one step: filter, threshold, in-place commit, EoTP, block advance.

    pred/conf hold the n_rows block positions that are inside L_eff, in position order.
    """
    s = cfg.block_len
    b = st.cur_block
    g0 = b * s                                  # generation index of the block's first position
    n_rows = len(pred)
    L_eff_in = st.L_eff

    # filter input: s confidences in position order; positions outside L_eff count as finished
    c = np.ones(s, dtype=np.float64)
    c[:n_rows] = conf
    blk_masked = st.masked[g0: g0 + s].copy()
    if cfg.committed_conf_mode == 1:
        c[~blk_masked] = 1.0
    conf_full = np.zeros(s, dtype=np.float64)
    conf_full[:n_rows] = conf

    if cfg.use_filter and cfg.rule == "filter":
        p = sigmoid(filter_logits(filt, c))
    else:
        p = np.zeros(s, dtype=np.float64)
    commit = np.full(s, -1, dtype=np.int64)     # token written at each committed position
    commit[:n_rows] = pred
    if cfg.rule == "filter":
        unmask, forced = unmask_rule(p, conf_full, blk_masked, cfg.tau)
    elif cfg.rule == "confidence":
        unmask, forced = confidence_rule(conf_full, blk_masked, cfg.conf_threshold)
    elif cfg.rule == "egp":
        r_blk = np.asarray(ref, dtype=np.int64)[g0: g0 + s]
        pred_full = np.full(s, -1, dtype=np.int64)
        pred_full[:n_rows] = pred
        unmask, forced = egp_rule(pred_full, r_blk, conf_full, blk_masked)
        if forced:
            commit = np.where(unmask, r_blk, commit)
    else:
        raise ValueError("unknown rule %r" % (cfg.rule,))

    for j in np.where(unmask)[0]:
        st.masked[g0 + j] = False
        st.tokens[st.P + g0 + j] = commit[j]
    st.forced += int(forced)

    # EoTP: earliest committed [EoT] in the generation region cuts the sequence there
    if cfg.use_eotp:
        gen = st.tokens[st.P: st.P + st.G]
        hits = np.where((gen == m.eot_id) & ~st.masked)[0]
        if len(hits):
            e = int(hits[0])
            st.eot_pos = e
            st.L_eff = st.P + e + 1
            st.masked[e + 1:] = False
            st.tokens[st.P + e + 1: st.P + st.G] = m.eot_id

    if not st.masked[g0: g0 + s].any():
        if st.eot_pos >= 0 or b + 1 == st.G // s:
            st.done = True
        else:
            st.cur_block = b + 1

    return StepRecord(block=b, L_eff_in=L_eff_in, n_rows=n_rows, pred=pred.copy(), conf=conf.copy(),
                      gap=None if gap is None else gap.copy(), filt_in=c, p=p, unmask=unmask,
                      forced=forced, logits=logits)


def denoise_step(m: Model, filt: Dict[str, np.ndarray], st: SeqState, cfg: DecodeConfig,
                 keep_logits: bool = False, predictor=None, ref: Optional[np.ndarray] = None) -> StepRecord:
    """One iteration of the while loop of Algorithm 2 for one sequence.

    predictor(m, st, cfg) -> logits[n_rows, V] replaces the transformer when given
    (tests drive the decision logic with hand-built logits through it).
    """
    assert not st.done
    st.steps += 1
    logits = (predictor or block_logits)(m, st, cfg)
    pred, conf, gap = confidence_head(logits)
    return decide(m, filt, st, cfg, pred, conf, gap, logits if keep_logits else None, ref)


@dataclass
class DecodeResult:
    response: np.ndarray   # [G]; positions after [EoT] hold eot_id
    out_len: int           # tokens up to and including [EoT], or G
    steps: int             # number of M(X) evaluations
    forced: int
    trace: List[StepRecord] = field(default_factory=list)


def decode(m: Model, filt: Dict[str, np.ndarray], prompt: Sequence[int], G: int,
           cfg: DecodeConfig, keep_trace: bool = True, keep_logits: bool = False,
           predictor=None, ref: Optional[np.ndarray] = None) -> DecodeResult:
    """Algorithm 2 with Algorithm 3's end-of-text break, for one prompt.  `ref` [G]: the reference
    answer of rule "egp" (Algorithm 1's decode, without the filter update)."""
    if cfg.rule == "egp" and (ref is None or len(ref) != G):
        raise ValueError("rule 'egp' needs a reference answer of G tokens")
    if G % cfg.block_len != 0:
        raise ValueError("generation length must be a multiple of the block length")
    st = init_state(m, prompt, G)
    trace = []
    while not st.done:
        rec = denoise_step(m, filt, st, cfg, keep_logits, predictor, ref)
        if keep_trace:
            trace.append(rec)
    out_len = st.eot_pos + 1 if st.eot_pos >= 0 else G
    return DecodeResult(response=st.tokens[st.P: st.P + G].copy(), out_len=out_len,
                        steps=st.steps, forced=st.forced, trace=trace)


def decode_batch(m: Model, filt: Dict[str, np.ndarray], prompts: np.ndarray, G: int,
                 cfg: DecodeConfig, **kw) -> List[DecodeResult]:
    """Sequences are independent: each prompt is decoded on its own."""
    return [decode(m, filt, p, G, cfg, **kw) for p in prompts]


# ----------------------------------------------------------------------------
# Filter training (Algorithm 1, Eq. 5-6, Section 4.1)
#
# Stage 1 collects, under the EGP policy, one sample per decoding step: the filter's input
# (the block's s confidences, as decide() feeds them) and Algorithm 1's targets y_j.  Stage 2
# minimises the mean binary cross-entropy between sigmoid(f_theta(conf)) and y with AdamW.
# Readings (the paper gives the optimiser, the learning rate 0.001 and the epoch count only):
#   * the loss of a batch is the mean over its samples and all s positions (Eq. 6 with
#     m = samples * s);
#   * AdamW as published (Loshchilov & Hutter): decoupled weight decay, bias-corrected moments;
#     beta1 0.9, beta2 0.999, eps 1e-8, weight decay 0.01 unless given;
#   * an epoch visits the samples in the given order in consecutive batches (batch_size 0 = one
#     batch holding every sample); the caller shuffles, if it wants to, before the call.

def egp_samples(trace: List[StepRecord], ref: np.ndarray, s: int):
    """Stage 1 for one decoded sequence: (C[n, s], Y[n, s]) from the steps of an EGP decode.
    Positions cut off by EoTP carry pred = -1 and therefore the target 0."""
    C = np.stack([t.filt_in for t in trace]).astype(np.float64)
    Y = np.zeros((len(trace), s), dtype=np.float64)
    for n, t in enumerate(trace):
        pred = np.full(s, -1, dtype=np.int64)
        pred[: t.n_rows] = t.pred
        Y[n] = egp_labels(pred, np.asarray(ref)[t.block * s: (t.block + 1) * s])
    return C, Y


def bce_with_logits(z: np.ndarray, y: np.ndarray) -> float:
    """Eq. 6: -mean[y log sigmoid(z) + (1 - y) log(1 - sigmoid(z))], in the overflow-free form
    max(z, 0) - z y + log(1 + exp(-|z|))."""
    return float(np.mean(np.maximum(z, 0.0) - z * y + np.log1p(np.exp(-np.abs(z)))))


def filter_layers_loss_and_grads(layers, C: np.ndarray, Y: np.ndarray):
    """The same for the depth variants of Section 4.4: layers = [(W, b), ...], ReLU between consecutive
    layers.  Returns (loss, [(dW, db), ...])."""
    acts = [C]                                   # input of layer k
    pres = []
    x = C
    for k, (w, b) in enumerate(layers):
        if k > 0:
            x = np.maximum(x, 0.0)
            acts.append(x)
        x = x @ widen(w).T + widen(b)
        pres.append(x)
    z = x
    loss = bce_with_logits(z, Y)
    delta = (sigmoid(z) - Y) / z.size            # d loss / d (output of the last layer)
    grads = [None] * len(layers)
    for k in range(len(layers) - 1, -1, -1):
        grads[k] = (delta.T @ acts[k], delta.sum(axis=0))
        if k > 0:
            delta = (delta @ widen(layers[k][0])) * (pres[k - 1] > 0.0)
    return loss, grads


def train_filter_layers(layers0, C: np.ndarray, Y: np.ndarray, epochs: int, lr: float = 1e-3, beta1: float = 0.9,
                        beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.01, batch_size: int = 0):
    """train_filter for a filter given as a list of (W, b) layers; returns (layers, losses)."""
    layers = [(widen(w).copy(), widen(b).copy()) for (w, b) in layers0]
    mom = [(np.zeros_like(w), np.zeros_like(b)) for (w, b) in layers]
    var = [(np.zeros_like(w), np.zeros_like(b)) for (w, b) in layers]
    N = len(C)
    bs = N if batch_size <= 0 else batch_size
    losses = []
    t = 0
    for _ in range(epochs):
        for lo in range(0, N, bs):
            loss, g = filter_layers_loss_and_grads(layers, C[lo: lo + bs], Y[lo: lo + bs])
            losses.append(loss)
            t += 1
            for k in range(len(layers)):
                new = []
                for q in range(2):
                    p, m, v = adamw_step(layers[k][q], g[k][q], mom[k][q], var[k][q], t, lr, beta1, beta2, eps, weight_decay)
                    new.append((p, m, v))
                layers[k] = (new[0][0], new[1][0])
                mom[k] = (new[0][1], new[1][1])
                var[k] = (new[0][2], new[1][2])
    return layers, np.asarray(losses)


def filter_loss_and_grads(filt: Dict[str, np.ndarray], C: np.ndarray, Y: np.ndarray):
    """Loss of Eq. 6 over the batch (C[n, s], Y[n, s]) and its gradient w.r.t. w1, b1, w2, b2."""
    w1, b1, w2, b2 = (widen(filt[k]) for k in ("w1", "b1", "w2", "b2"))
    pre = C @ w1.T + b1                       # [n, s]
    h = np.maximum(pre, 0.0)
    z = h @ w2.T + b2
    loss = bce_with_logits(z, Y)
    dz = (sigmoid(z) - Y) / z.size            # d loss / d z
    g = {"w2": dz.T @ h, "b2": dz.sum(axis=0)}
    dh = dz @ w2
    dpre = dh * (pre > 0.0)
    g["w1"] = dpre.T @ C
    g["b1"] = dpre.sum(axis=0)
    return loss, g


def adamw_step(param: np.ndarray, grad: np.ndarray, m: np.ndarray, v: np.ndarray, t: int,
               lr: float, beta1: float, beta2: float, eps: float, weight_decay: float):
    """One AdamW update, step count t >= 1; returns (param, m, v)."""
    param = param * (1.0 - lr * weight_decay)
    m = beta1 * m + (1.0 - beta1) * grad
    v = beta2 * v + (1.0 - beta2) * grad * grad
    m_hat = m / (1.0 - beta1 ** t)
    v_hat = v / (1.0 - beta2 ** t)
    return param - lr * m_hat / (np.sqrt(v_hat) + eps), m, v


def train_filter(filt0: Dict[str, np.ndarray], C: np.ndarray, Y: np.ndarray, epochs: int,
                 lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                 weight_decay: float = 0.01, batch_size: int = 0):
    """Stage 2 of Algorithm 1.  Returns (filter, losses): the trained parameters (fp64) and the
    loss of every update's batch, measured before the update."""
    names = ("w1", "b1", "w2", "b2")
    filt = {k: widen(filt0[k]).copy() for k in names}
    mom = {k: np.zeros_like(filt[k]) for k in names}
    var = {k: np.zeros_like(filt[k]) for k in names}
    N = len(C)
    bs = N if batch_size <= 0 else batch_size
    losses = []
    t = 0
    for _ in range(epochs):
        for lo in range(0, N, bs):
            loss, g = filter_loss_and_grads(filt, C[lo: lo + bs], Y[lo: lo + bs])
            losses.append(loss)
            t += 1
            for k in names:
                filt[k], mom[k], var[k] = adamw_step(filt[k], g[k], mom[k], var[k], t, lr, beta1, beta2, eps,
                                                     weight_decay)
    return filt, np.asarray(losses)
