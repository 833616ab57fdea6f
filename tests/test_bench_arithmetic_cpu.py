"""The bench's roofline arithmetic, counted by hand for the 8B-shaped step (no GPU): a dropped projection, a wrong
factor of two or a swapped peak would move the reported fractions without any kernel changing."""
from __future__ import annotations

import math

import bench
from paper_2509_25188_b200 import workloads as wl


def test_step_work_of_the_8b_step_counted_term_by_term():
    sh = wl.LLADA_8B
    T, L, R = 512, 512, 32
    w = bench.step_work(sh, T, L, R)
    d, F, V, NL, hd = 4096, 12288, 126464, 32, 32 * 128
    per_layer = (2 * T * d * 3 * hd        # QKV
                 + 2 * T * hd * d          # output projection
                 + 2 * T * d * 2 * F       # gate and up
                 + 2 * T * F * d           # down
                 + 2 * T * L * hd * 2)     # scores and probability-weighted values
    assert w["flops"] == NL * per_layer + 2 * R * d * V
    assert math.isclose(w["flops"], 7.3174e12, rel_tol=1e-4)
    n_weights = NL * (3 * hd * d + hd * d + 3 * d * F) + V * d          # bf16: the embedding table is only gathered from
    assert w["weight_bytes"] == 2 * n_weights
    assert math.isclose(w["weight_bytes"], 14.99e9, rel_tol=1e-3)


def test_roofline_takes_the_slower_of_flops_and_bytes_for_both_peak_figures():
    pk = {"hbm_gbs": 6525.2, "bf16_tflops": 1657.2, "bf16_tflops_sustained": 1383.3}
    w = bench.step_work(wl.LLADA_8B, 512, 512, 32)
    t_burst, t_sust, t_bytes, bound = bench.roofline_ms(w, pk)
    assert bound == "tensor"
    assert math.isclose(t_burst, w["flops"] / 1657.2e12 * 1e3) and math.isclose(t_burst, 4.4155, rel_tol=1e-3)
    assert math.isclose(t_sust, 5.2898, rel_tol=1e-3)
    assert math.isclose(t_bytes, (w["weight_bytes"] + w["act_bytes"]) / 6525.2e9 * 1e3)
    # a step of 32 rows against stored keys is bound by its bytes: the weights and the store read once
    kv = 2.0 * 2 * 32 * 512 * 4096
    w32 = bench.step_work(wl.LLADA_8B, 32, 512, 32, kv)
    t_burst32, t_sust32, t_bytes32, bound32 = bench.roofline_ms(w32, pk)
    assert bound32 == "hbm" and t_burst32 == t_sust32 == t_bytes32
    assert math.isclose(t_bytes32, (w32["weight_bytes"] + w32["act_bytes"] + kv) / 6525.2e9 * 1e3)
    assert 2.3 < t_bytes32 < 2.45
