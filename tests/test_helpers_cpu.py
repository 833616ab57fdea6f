"""The bound the GPU tests hold confidences to, checked by brute force (no GPU): perturbing every logit of a row by at
most eps keeps the softmax probability of the (possibly changed) argmax inside helpers.conf_interval."""
from __future__ import annotations

import numpy as np

from oracle import l2pd_oracle as orc
from tests.helpers import conf_interval


def test_conf_interval_holds_under_any_bounded_logit_error():
    rng = np.random.default_rng(0)
    tight = 0.0
    for _ in range(3000):
        V = int(rng.integers(2, 40))
        logits = rng.normal(size=(1, V)) * rng.uniform(0.05, 8.0)
        eps = float(rng.uniform(0.0, 0.5))
        _, c0, _ = orc.confidence_head(logits)
        lo, hi = conf_interval(c0, np.array([eps]))
        for trial in range(4):
            d = rng.uniform(-eps, eps, size=(1, V))
            if trial == 0:                      # the extreme case: top up, everything else down
                d = np.full((1, V), -eps)
                d[0, logits.argmax()] = eps
            _, c1, _ = orc.confidence_head(logits + d)
            assert lo[0] - 1e-12 <= c1[0] <= hi[0] + 1e-12
            tight = max(tight, float((c1[0] - c0[0]) / max(hi[0] - c0[0], 1e-300)))
    assert tight > 0.999                        # the bound is attained, not loose


def test_conf_interval_limits():
    lo, hi = conf_interval(np.array([0.5, 1.0, 1e-4]), np.array([0.0, 0.3, 0.1]))
    assert lo[0] == hi[0] == 0.5                # no logit error: no room
    assert lo[1] == hi[1] == 1.0                # a certain row stays certain
    assert np.isclose(hi[2], 1e-4 * np.exp(0.2), rtol=1e-3) and np.isclose(lo[2], 1e-4 * np.exp(-0.2), rtol=1e-3)
