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
