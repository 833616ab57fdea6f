"""Kernel-level parity, through the C ABI, against the oracle's functions on the same seeded inputs.

Tolerances (bf16 inputs, fp32 accumulation, one rounding of the output to bf16):
a product of K terms of magnitude ~|a||w| accumulated in fp32 is exact to ~K*2^-24 relative to
sum|a||w|; the bf16 store adds 2^-9 relative.  The checks below use
|gpu - oracle| <= 2^-8 * |oracle| + 2e-3 * row_scale, row_scale = rms of the oracle's row.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

from oracle import l2pd_oracle as orc
from paper_2509_25188_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _b():
    from paper_2509_25188_b200 import binding
    return binding


def _bf16(seed, stream, shape, std):
    return wl.make_activations(seed, stream, shape, std, "bf16")


def _close_bf16(got, want, extra=0.0):
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    scale = np.sqrt((want ** 2).mean(axis=-1, keepdims=True)) + 1e-30
    tol = 2.0 ** -8 * np.abs(want) + (2e-3 + extra) * scale
    bad = np.abs(got - want) > tol
    assert not bad.any(), "max err %g at %s (want %g)" % (
        np.abs(got - want).max(), np.argwhere(bad)[0], want[tuple(np.argwhere(bad)[0])])


GEMM_SHAPES = [
    (128, 256, 64, 0),      # single tile, one k-block
    (200, 320, 192, 0),     # ragged M, several tiles
    (512, 1024, 512, 0),
    (77, 136, 72, 64),      # ragged everything: N tail inside a tile, K tail inside a k-block
    (300, 528, 1032, 176),  # odd tile width (multiple of 16), K tail
    (1, 64, 64, 0),
    (640, 2048, 256, 112),  # many tiles per CTA: accumulator double-buffering, ring wrap-around
    (512, 1024, 512, 2000),  # pair of SMs per 256-row tile (cta_group::2), automatic width
    (300, 528, 1032, 2176),  # pair: ragged M (second half-tile partly empty), N and K tails
    (640, 2048, 256, 2112),  # pair: several tiles per pair
    (129, 256, 128, 2256),   # pair: second CTA holds a single live row
    (4000, 4608, 320, 0),    # many row tiles: automatic plan
    (512, 1056, 512, 202176),  # two 256-row slabs per unit (accumulators not double-buffered), one unit per pair
    (300, 528, 1032, 202176),  # two slabs: the second one mostly empty, N and K tails
    (1100, 2048, 256, 202128), # two slabs: several units per pair, ragged last row tile
    (512, 12288, 320, 202256), # two slabs, full-width accumulators (all 512 tensor-memory columns)
    (32, 1024, 4096, 1000096),  # few rows: the two MMA issuers take alternate k-blocks (two accumulators added in the epilogue)
    (100, 528, 1032, 1001176),  # the same with an odd number of k-blocks, N and K tails
    (128, 512, 320, 1000256),   # the same with both accumulators 256 columns wide
    (32, 1024, 4096, 2000096),  # alternation switched off: one issuer
    (32, 12288, 4096, 0),       # the QKV projection of a 32-row step, automatic plan
    (256, 2048, 1032, 1002240), # alternate k-blocks on a pair of SMs (one 256-row slab), K tail
    (200, 12288, 4096, 0),      # QKV at 200 rows, automatic plan
    (64, 8192, 320, 1001032),   # alternate k-blocks with several units per CTA (the accumulators are reused unit after unit)
]


@pytest.mark.parametrize("M,N,K,tile_n", GEMM_SHAPES)
def test_gemm_bf16_store(M, N, K, tile_n):
    b = _b()
    A = _bf16(1, 0, (M, K), 1.0)
    W = _bf16(1, 1, (N, K), 0.05)
    got = b.gemm_bf16(b.to_device(A), b.to_device(W), tile_n).float().cpu().numpy()
    want = orc.linear(orc.widen(A), W)
    _close_bf16(got, want)


RESIDUAL_SHAPES = GEMM_SHAPES[:5] + [
    (512, 1024, 2048, 22128),   # pair + K split in two: slices add into X with reductions
    (300, 528, 4104, 31064),    # single CTA, three K slices, K tail in the last slice
    (512, 512, 12288, 0),       # automatic plan for a narrow, deep projection
    (512, 4096, 1024, 2240),    # pair, width 240
    (512, 4096, 4096, 232176),  # two slabs + three K slices
    (400, 1024, 12288, 222176), # two slabs + two K slices, ragged rows
    (32, 4096, 4096, 1041112),  # few rows: four K slices, alternate k-blocks inside each
    (64, 528, 4104, 1031064),   # three slices, the last one shorter, K tail
    (100, 512, 192, 1031064),   # slices of a single k-block: the second issuer has nothing to add
    (32, 4096, 12288, 0),       # the down projection of a 32-row step, automatic plan
    (256, 4096, 12288, 1042240), # pair, four K slices, alternate k-blocks
    (256, 4096, 12288, 0),
]


@pytest.mark.parametrize("M,N,K,tile_n", RESIDUAL_SHAPES)
def test_gemm_bf16_residual(M, N, K, tile_n):
    b = _b()
    A = _bf16(2, 0, (M, K), 1.0)
    W = _bf16(2, 1, (N, K), 0.05)
    X = wl.make_activations(2, 2, (M, N), 1.0, "fp32")
    Xd = b.to_device(X.copy())
    b.gemm_bf16_residual(b.to_device(A), b.to_device(W), Xd, tile_n)
    want = X.astype(np.float64) + orc.linear(orc.widen(A), W)
    got = Xd.cpu().numpy()
    assert np.allclose(got, want, rtol=1e-5, atol=1e-4 * np.sqrt(K))


@pytest.mark.parametrize("M,F,K,tile_n", [(128, 128, 64, 0), (200, 336, 192, 0), (512, 1408, 512, 224),
                                          (77, 136, 72, 64), (640, 2048, 256, 96), (512, 1408, 512, 2224),
                                          (200, 336, 192, 2064), (1000, 2048, 256, 2256),
                                          (512, 1408, 512, 202160), (300, 2048, 256, 202256),
                                          (512, 1408, 512, 202176), (200, 336, 192, 1176), (130, 1408, 128, 2144),
                                          (512, 24576, 256, 0), (32, 1408, 4096, 1000176), (90, 336, 192, 1000064),
                                          (32, 12288, 4096, 0), (256, 1408, 4096, 1002176), (256, 12288, 4096, 0),
                                          (32, 8192, 192, 1001064)])
def test_gemm_bf16_swiglu(M, F, K, tile_n):
    b = _b()
    A = _bf16(3, 0, (M, K), 1.0)
    Wg = _bf16(3, 1, (F, K), 0.08)
    Wu = _bf16(3, 2, (F, K), 0.08)
    got = b.gemm_bf16_swiglu(b.to_device(A), b.to_device(Wg), b.to_device(Wu), tile_n).float().cpu().numpy()
    a = orc.widen(A)
    want = orc.silu(orc.linear(a, Wg)) * orc.linear(a, Wu)
    _close_bf16(got, want)


@pytest.mark.parametrize("R,V,K,with_bias", [(32, 4096, 256, False), (16, 5000, 136, True), (200, 1000, 512, True),
                                             (1, 70, 64, False), (32, 20000, 1024, True)])
def test_lm_head_fused_confidence(R, V, K, with_bias):
    """Eq. 3-4: argmax and softmax probability of the argmax, reduced without storing logits."""
    b = _b()
    A = _bf16(4, 0, (R, K), 1.0)
    W = _bf16(4, 1, (V, K), 0.3)
    bias = wl.make_activations(4, 2, (V,), 1.0, "fp32") if with_bias else None
    pred, conf, logits = b.lm_head_bf16(b.to_device(A), b.to_device(W),
                                        b.to_device(bias) if with_bias else None, want_logits=True)
    ref = orc.linear(orc.widen(A), W)
    if with_bias:
        ref = ref + bias.astype(np.float64)[None, :]
    rp, rc, gap = orc.confidence_head(ref)
    got_logits = logits.cpu().numpy()
    assert np.abs(got_logits - ref).max() <= 1e-4 * np.abs(ref).max() + 1e-5 * np.sqrt(K)
    pred, conf = pred.cpu().numpy(), conf.cpu().numpy()
    sure = gap > 1e-3 * np.abs(ref).max()
    assert sure.mean() > 0.5
    assert np.array_equal(pred[sure], rp[sure])
    assert np.abs(conf - rc)[sure].max() < 1e-3
    # the fused reduction must agree with the logits the same kernel wrote
    p2, c2, _ = orc.confidence_head(got_logits.astype(np.float64))
    assert np.array_equal(pred, p2)
    assert np.abs(conf - c2).max() < 1e-5
    # without the debug buffer the result is the same
    pred3, conf3, _ = b.lm_head_bf16(b.to_device(A), b.to_device(W), b.to_device(bias) if with_bias else None)
    assert np.array_equal(pred3.cpu().numpy(), pred) and np.array_equal(conf3.cpu().numpy(), conf)


def test_lm_head_ties_pick_lowest_id():
    b = _b()
    R, V, K = 4, 600, 64
    A = np.zeros((R, K), np.float32)
    A[:, 0] = 1.0
    W = np.zeros((V, K), np.float32)
    W[[7, 300, 599], 0] = 2.0          # three equal maxima, in different vocabulary tiles
    pred, conf, _ = b.lm_head_bf16(b.to_device(wl.f32_to_bf16_bits(A)), b.to_device(wl.f32_to_bf16_bits(W)))
    rp, rc, _ = orc.confidence_head(orc.linear(A.astype(np.float64), W))
    assert pred.cpu().numpy().tolist() == [7] * R == rp.tolist()
    assert np.abs(conf.cpu().numpy() - rc).max() < 1e-6


# impl 0 = tensor-memory (tcgen05) kernel for head size 128, 1 = warp-level (mma.sync) kernel
@pytest.mark.parametrize("Tq,Tk,H,dh,impl", [(64, 64, 2, 128, 0), (100, 100, 3, 128, 0), (37, 200, 2, 64, 0),
                                             (512, 512, 4, 128, 0), (5, 1, 1, 64, 0), (130, 1030, 2, 128, 0),
                                             (1, 1, 1, 128, 0), (129, 128, 1, 128, 0), (128, 129, 2, 128, 0),
                                             (300, 257, 3, 128, 0), (256, 2048, 2, 128, 0),
                                             (64, 64, 2, 128, 1), (130, 1030, 2, 128, 1), (512, 512, 4, 128, 1)])
def test_attention_bidirectional(Tq, Tk, H, dh, impl):
    b = _b()
    q = _bf16(5, 0, (Tq, H * dh), 1.0)
    k = _bf16(5, 1, (Tk, H * dh), 1.0)
    v = _bf16(5, 2, (Tk, H * dh), 1.0)
    got = b.attention_bf16(b.to_device(q), b.to_device(k), b.to_device(v), H, dh, impl).float().cpu().numpy()
    want = orc.attention(orc.widen(q).reshape(Tq, H, dh), orc.widen(k).reshape(Tk, H, dh),
                         orc.widen(v).reshape(Tk, H, dh)).reshape(Tq, H * dh)
    # probabilities are rounded to bf16 before the second product: 2^-9 relative on each weight
    assert np.abs(got - want).max() < 2e-2
    assert np.sqrt(((got - want) ** 2).mean()) < 4e-3


@pytest.mark.parametrize("impl", [0, 1])
def test_attention_scores_that_grow_along_the_keys(impl):
    """Later keys score far higher than earlier ones for some query rows and not for others, so the
    running row maximum jumps by many powers of two between key tiles in part of each warp only:
    exercises the rescaling of the partial output (for the tensor-memory kernel, the lazy one)."""
    b = _b()
    Tq, Tk, H, dh = 200, 640, 2, 128
    rng = np.random.default_rng(7)
    q = np.abs(rng.standard_normal((Tq, H * dh))).astype(np.float32)
    q[::3] *= 0.01                                   # every third row: nearly flat scores
    k = np.abs(rng.standard_normal((Tk, H * dh))).astype(np.float32)
    k *= (0.05 + 2.0 * np.arange(Tk)[:, None] / Tk)  # key norm grows with the key index
    v = rng.standard_normal((Tk, H * dh)).astype(np.float32)
    qb, kb, vb = (wl.f32_to_bf16_bits(a) for a in (q, k, v))
    got = b.attention_bf16(b.to_device(qb), b.to_device(kb), b.to_device(vb), H, dh, impl).float().cpu().numpy()
    want = orc.attention(orc.widen(qb).reshape(Tq, H, dh), orc.widen(kb).reshape(Tk, H, dh),
                         orc.widen(vb).reshape(Tk, H, dh)).reshape(Tq, H * dh)
    assert np.abs(got - want).max() < 3e-2
    assert np.sqrt(((got - want) ** 2).mean()) < 6e-3


def test_shape_errors_are_reported_not_launched():
    b = _b()
    A = b.to_device(_bf16(6, 0, (16, 64), 1.0))
    W = b.to_device(_bf16(6, 1, (64, 64), 1.0))
    with pytest.raises(b.L2pdError) as e:
        b.gemm_bf16(A, W, tile_n=40)          # not a multiple of 16
    assert e.value.status == -2
    with pytest.raises(b.L2pdError):
        b.gemm_bf16(A[:, :60], W[:, :60])      # K not a multiple of 8
