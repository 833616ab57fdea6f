"""Algorithm 1 on the CUDA path: EGP sample collection (stage 1) and AdamW training of the filter
(stage 2, Eq. 6) against the oracle.

Tolerances: the kernel works in fp32, the oracle in fp64.  One update moves a parameter by about lr
whatever the gradient's size (Adam normalises it), so an fp32 error of relative size ~1e-6 in a gradient
component shifts the update by ~1e-6 * lr and the parameter error after T updates stays near T * lr * 1e-5
as long as no gradient component sits at rounding level; the tests use 200-300 updates at lr 1e-3..1e-2 and
compare parameters to 2e-3 absolute and the loss curve to 2e-4.
"""
from __future__ import annotations

import numpy as np
import pytest

from oracle import l2pd_oracle as orc
from paper_2509_25188_b200 import workloads as wl
from tests.helpers import oracle_model

pytestmark = pytest.mark.gpu


def _b():
    from paper_2509_25188_b200 import binding
    return binding


def _data(s, n, seed):
    rng = np.random.default_rng(seed)
    C = rng.uniform(0.0, 1.0, size=(n, s)).astype(np.float32)
    Y = (C + 0.15 * rng.normal(size=(n, s)) > 0.6).astype(np.uint8)
    return C, Y


@pytest.mark.parametrize("s,n,batch", [(32, 1000, 0), (32, 1000, 256), (16, 77, 0), (64, 333, 100), (5, 40, 0)])
def test_training_matches_the_oracle(s, n, batch):
    """Several tiles per block and a ragged last tile (n not a multiple of 32), ragged last batch,
    the largest block length (64) and an odd one."""
    C, Y = _data(s, n, seed=s + n)
    f0 = wl.make_filter(s, seed=3)
    epochs = 200 if batch == 0 else 60
    want, wl_losses = orc.train_filter(f0, C.astype(np.float64), Y.astype(np.float64), epochs, lr=5e-3, batch_size=batch)
    got, losses = _b().filter_train(f0, C, Y, epochs, lr=5e-3, batch_size=batch)
    assert len(losses) == len(wl_losses)
    assert np.abs(losses - wl_losses).max() < 2e-4
    assert abs(losses[0] - wl_losses[0]) < 2e-6                       # the first loss involves no update at all
    for k in ("w1", "b1", "w2", "b2"):
        assert np.abs(got[k] - want[k]).max() < 2e-3, k
    assert losses[-1] < losses[0]


def test_training_is_bit_reproducible_and_zero_epochs_is_identity():
    s, n = 32, 500
    C, Y = _data(s, n, seed=9)
    f0 = wl.make_filter(s, seed=4)
    a, la = _b().filter_train(f0, C, Y, 50)
    b, lb = _b().filter_train(f0, C, Y, 50)
    assert np.array_equal(la, lb) and all(np.array_equal(a[k], b[k]) for k in a)
    z, lz = _b().filter_train(f0, C, Y, 0)
    assert len(lz) == 0 and all(np.array_equal(z[k], f0[k].astype(np.float32)) for k in z)


def test_bad_arguments():
    b = _b()
    C, Y = _data(8, 10, seed=1)
    f0 = wl.make_filter(8, seed=1)
    with pytest.raises(b.L2pdError) as e:
        b.filter_train(f0, C, Y, 1, lr=0.0)
    assert e.value.status == -1
    C2, Y2 = _data(65, 4, seed=1)
    with pytest.raises(b.L2pdError) as e:
        b.filter_train(wl.make_filter(65, seed=1), C2, Y2, 1)
    assert e.value.status == -2


def test_egp_collection_then_training_end_to_end():
    """Stage 1 on the GPU: an EGP decode against the model's own one-token-per-step answer appends one
    (filter input, target) sample per step; the samples equal the oracle's for the same decode.  Stage 2
    on those samples lowers the loss, and the trained filter drives a decode that still ends."""
    b = _b()
    shape = wl.TINY
    w = wl.make_weights(shape, seed=0, final_norm_gain=wl.spread_gain(shape))
    d = wl.DECODES["C0"]
    s, G = d.block_len, d.gen_len
    m = oracle_model(shape, w)
    B = 2
    prompts = wl.make_prompts(B, d.prompt_len, shape, seed=5)
    van = orc.DecodeConfig(block_len=s, use_filter=False, use_eotp=False)
    refs = np.stack([orc.decode(m, None, p, G, van, keep_trace=False).response for p in prompts])
    f0 = wl.make_filter(s, d.tau, seed=0)
    dec = b.Decoder(shape, w, f0, block_len=s, tau=d.tau, max_batch=B, max_seq=d.prompt_len + G, use_eotp=False)
    dec.set_unmask_rule("egp", reference=refs)
    sink_c, sink_y = dec.set_collect(B * G)
    toks, _, steps, total = dec.decode(prompts, G)
    n = dec.collect_count
    assert n == int(steps.sum()) and np.array_equal(toks, refs)
    got_c, got_y = sink_c[:n].cpu().numpy(), sink_y[:n].cpu().numpy()
    # the oracle's samples, interleaved the same way: step by step, unfinished sequences in order
    cfg = orc.DecodeConfig(block_len=s, rule="egp", use_eotp=False)
    per_seq = []
    for i in range(B):
        r = orc.decode(m, f0, prompts[i], G, cfg, ref=refs[i])
        per_seq.append(orc.egp_samples(r.trace, refs[i], s))
        assert r.steps == steps[i]
    want_c, want_y = [], []
    for k in range(int(steps.max())):
        for i in range(B):
            if k < steps[i]:
                want_c.append(per_seq[i][0][k]); want_y.append(per_seq[i][1][k])
    want_c, want_y = np.stack(want_c), np.stack(want_y)
    assert np.abs(got_c - want_c).max() < 1e-3                  # fp32 model: confidences to 1e-3
    sure = np.abs(want_c - 0.5) < 2.0                           # all positions
    assert np.array_equal(got_y[sure], want_y[sure].astype(np.uint8))
    with pytest.raises(b.L2pdError):                            # a full sink refuses the step
        dec.set_collect(1)
        dec.state_reset(prompts, G)
        dec.denoise_step()
    dec.set_collect(0)
    trained, losses = b.filter_train(f0, got_c, got_y, 300, lr=1e-2)
    want_f, want_l = orc.train_filter(f0, got_c.astype(np.float64), got_y.astype(np.float64), 300, lr=1e-2)
    assert np.abs(losses - want_l).max() < 2e-4 and losses[-1] < losses[0]
    dec.close()
    dec2 = b.Decoder(shape, w, trained, block_len=s, tau=d.tau, max_batch=B, max_seq=d.prompt_len + G)
    toks2, out_len, steps2, _ = dec2.decode(prompts, G)
    ref2 = [orc.decode(m, trained, p, G, orc.DecodeConfig(block_len=s, tau=d.tau), keep_trace=False) for p in prompts]
    for i in range(B):
        assert steps2[i] == ref2[i].steps and np.array_equal(toks2[i], ref2[i].response)
    dec2.close()


@pytest.mark.parametrize("depth,s,n,batch", [(1, 32, 300, 0), (4, 32, 500, 128), (3, 16, 77, 0), (4, 64, 200, 0), (2, 64, 333, 100)])
def test_depth_variant_training_matches_the_oracle(depth, s, n, batch):
    """Section 4.4's one- and four-layer filters (and three): the tiled kernel's backpropagation through
    the layers against the oracle's, ragged tiles and batches included; depth 2 at s = 64 runs the same
    kernel as the two-layer entry point."""
    C, Y = _data(s, n, seed=depth * 100 + s)
    rng = np.random.default_rng(depth)
    layers0 = [((rng.normal(size=(s, s)) / np.sqrt(s)).astype(np.float32), (0.1 * rng.normal(size=s)).astype(np.float32))
               for _ in range(depth)]
    epochs = 120 if batch == 0 else 40
    want, want_l = orc.train_filter_layers(layers0, C.astype(np.float64), Y.astype(np.float64), epochs, lr=5e-3, batch_size=batch)
    got, losses = _b().filter_train_layers(layers0, C, Y, epochs, lr=5e-3, batch_size=batch)
    assert len(losses) == len(want_l) and np.abs(losses - want_l).max() < 2e-4
    for (w, b), (ww, wb) in zip(got, want):
        assert np.abs(w - ww).max() < 2e-3 and np.abs(b - wb).max() < 2e-3
    assert losses[-1] < losses[0]
    b_ = _b()
    with pytest.raises(b_.L2pdError) as e:
        b_.filter_train_layers(layers0 * 5, C, Y, 1)          # more than four layers
    assert e.value.status == -1
