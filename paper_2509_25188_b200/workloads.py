"""Seeded synthetic workloads for Learn2PD decoding.

This module only draws random numbers and lays them out as arrays.  It holds
none of the method's arithmetic (no norm, attention, softmax, filter or
unmasking code) so that the CPU oracle and the CUDA path can both be fed from
it without sharing any computation.  numpy only; no torch, no CUDA.

Every tensor is drawn from its own Philox stream keyed by (seed, tensor id), so
tensors can be generated in any order or in parallel and are identical on every
machine with the same numpy.

The paper evaluates LLaDA-8B-Instruct (block size 32, generation length 256 or
1024) on public benchmarks; neither the weights, the trained filter nor the
datasets are available here, so random-init models of the same shapes and
uniform-random prompts stand in for them.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np


@dataclass(frozen=True)
class ModelShape:
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
    dtype: str  # "fp32" or "bf16": storage type of matrices and embedding

    @property
    def n_params(self) -> int:
        d, f, v = self.d_model, self.d_ff, self.vocab
        return self.n_layers * (4 * d * d + 3 * d * f) + 2 * v * d


@dataclass(frozen=True)
class DecodeShape:
    batch: int
    prompt_len: int
    gen_len: int
    block_len: int
    tau: float = 0.96
    kv_cache: bool = False


# Tiny fp32 model: the full decode finishes in seconds on the CPU.
TINY = ModelShape(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ff=688, vocab=4096,
                  rms_eps=1e-5, rope_theta=10000.0, mask_id=4095, eot_id=4094, dtype="fp32")
# LLaDA-8B-shaped model, bf16 storage.
LLADA_8B = ModelShape(n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ff=12288,
                      vocab=126464, rms_eps=1e-5, rope_theta=500000.0,
                      mask_id=126463, eot_id=126462, dtype="bf16")

MODELS = {"tiny": TINY, "llada8b": LLADA_8B}

DECODES = {
    "C0": DecodeShape(batch=1, prompt_len=32, gen_len=64, block_len=16),
    "C1": DecodeShape(batch=1, prompt_len=256, gen_len=256, block_len=32),
    "C2": DecodeShape(batch=1, prompt_len=256, gen_len=256, block_len=32),
    "C3": DecodeShape(batch=16, prompt_len=512, gen_len=512, block_len=32),
    "C4": DecodeShape(batch=8, prompt_len=1024, gen_len=1024, block_len=32, kv_cache=True),
}


def thin(shape: ModelShape, n_layers: int) -> ModelShape:
    """Same widths, fewer layers (used where a full-depth oracle run is too slow)."""
    return replace(shape, n_layers=n_layers)


def spread_gain(shape: ModelShape) -> float:
    """Final-norm gain that makes logits of a random-init model wide enough for
    confidences to cover (0, 1): target logit std = 1.5 * sqrt(2 ln V), while a
    unit-RMS hidden row times N(0, 0.02^2) weights has std 0.02 * sqrt(d)."""
    return 1.5 * math.sqrt(2.0 * math.log(shape.vocab)) / (0.02 * math.sqrt(shape.d_model))


# ----------------------------------------------------------------------------
# number formats (storage conversion only)

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# random streams

def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream)]))


def _normal(seed: int, stream: int, shape, std: float, dtype: str) -> np.ndarray:
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16 if dtype == "bf16" else np.float32)
    g = _rng(seed, stream)
    chunk = 1 << 24
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        v = g.standard_normal(e - s, dtype=np.float32) * np.float32(std)
        out[s:e] = f32_to_bf16_bits(v) if dtype == "bf16" else v
    return out.reshape(shape)


_PER_LAYER = ("wqkv", "wo", "w_gate", "w_up", "w_down")


def make_weights(shape: ModelShape, seed: int = 0, final_norm_gain: float = 1.0,
                 std: float = 0.02, threads: int = 8) -> Dict[str, object]:
    """Random-init weights, every matrix i.i.d. N(0, std^2), stored row-major [out, in].

    Returns {"tok_emb": [V,d], "lm_head": [V,d], "final_norm": [d] f32,
             "layers": [{"wqkv": [3d,d], "wo": [d,d], "w_gate": [F,d], "w_up": [F,d],
                         "w_down": [d,F], "norm1": [d] f32, "norm2": [d] f32}, ...]}
    Matrices are float32 arrays (dtype "fp32") or uint16 bf16 bit patterns ("bf16").
    Norm gains are 1 except final_norm, which is the constant final_norm_gain.
    """
    d, f, v = shape.d_model, shape.d_ff, shape.vocab
    hd = shape.n_heads * shape.head_dim
    dims = {"wqkv": (3 * hd, d), "wo": (d, hd), "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f)}
    jobs = [("tok_emb", None, 0, (v, d)), ("lm_head", None, 1, (v, d))]
    for l in range(shape.n_layers):
        for k, name in enumerate(_PER_LAYER):
            jobs.append((name, l, 16 + l * 8 + k, dims[name]))

    def run(job):
        name, l, stream, shp = job
        return name, l, _normal(seed, stream, shp, std, shape.dtype)

    if threads > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            results = list(ex.map(run, jobs))
    else:
        results = [run(j) for j in jobs]

    layers = [dict(norm1=np.ones(d, np.float32), norm2=np.ones(d, np.float32))
              for _ in range(shape.n_layers)]
    out: Dict[str, object] = {"layers": layers,
                              "final_norm": np.full(d, final_norm_gain, np.float32)}
    for name, l, arr in results:
        if l is None:
            out[name] = arr
        else:
            layers[l][name] = arr
    return out


def make_filter(block_len: int, tau: float = 0.96, seed: int = 0, gain: float = 12.0,
                pivot: float = 0.3, mix: float = 0.5) -> Dict[str, np.ndarray]:
    """Seeded two-layer filter MLP, Linear(s,s)+b -> act -> Linear(s,s)+b, fp32.

    A trained filter is not available, so this one is built to behave like one:
    a noisy identity in both layers, so that position j's output rises with its own
    confidence and is perturbed by its neighbours':
      W1 = I + N(0, mix^2/s),  b1 ~ N(0, 0.02^2),
      W2 = gain * (I + N(0, mix^2/s)),  b2 = ln(tau/(1-tau)) - gain*pivot + N(0, 0.5^2),
    i.e. p_j crosses tau near conf_j = pivot, with seeded position-to-position variation.
    """
    s = block_len
    g = _rng(seed, 7)
    eye = np.eye(s)
    w1 = (eye + g.standard_normal((s, s)) * (mix / math.sqrt(s))).astype(np.float32)
    b1 = (g.standard_normal(s) * 0.02).astype(np.float32)
    w2 = (gain * (eye + g.standard_normal((s, s)) * (mix / math.sqrt(s)))).astype(np.float32)
    b2 = (math.log(tau / (1.0 - tau)) - gain * pivot + 0.5 * g.standard_normal(s)).astype(np.float32)
    return {"w1": w1, "b1": b1, "w2": w2, "b2": b2}


def make_prompts(batch: int, prompt_len: int, shape: ModelShape, seed: int = 1) -> np.ndarray:
    """Uniform ids in [0, min(mask_id, eot_id)): neither special id appears. Row i uses seed+i."""
    hi = min(shape.mask_id, shape.eot_id)
    rows = [_rng(seed + i, 3).integers(0, hi, size=prompt_len, dtype=np.int64) for i in range(batch)]
    return np.stack(rows).astype(np.int32)


def make_eot_bias(shape: ModelShape, value: float) -> np.ndarray:
    """LM-head bias that is zero except at eot_id (lets a workload place [EoT] mid-sequence)."""
    b = np.zeros(shape.vocab, np.float32)
    b[shape.eot_id] = value
    return b


def make_activations(seed: int, stream: int, shape, std: float = 1.0, dtype: str = "fp32") -> np.ndarray:
    """Generic N(0, std^2) tensor for kernel-level tests."""
    return _normal(seed, 1000 + stream, shape, std, dtype)
