"""The allocation-free LM-head entry point against the ordinary one.

Some callers of this library cannot call cudaMalloc when they need a result: their device memory is
owned by an arena set up at start, or is fully committed to weights and caches.  For them the
library keeps the LM head's per-tile reduction records in a fixed array of its own.  This test calls
that entry point through the C ABI twice in a row, on different inputs, and checks both results
against l2pd_lm_head_bf16 (same kernels, caller-provided scratch): predictions identical,
confidences within the 1e-6 the kernel tests use for identical arithmetic — and against the CPU
oracle's Eq. 3-4 on the same inputs, with the checks the LM-head kernel test applies (ids where the
top-2 logit gap is clear, confidences to 1e-3).  It is collected last so that a run stopping at the
first failure has already run everything else; it also passes alone.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

from oracle import l2pd_oracle as orc
from paper_2509_25188_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _host_case(seed, R, V, K, with_bias):
    A = wl.make_activations(seed, 0, (R, K), 1.0, "bf16")
    W = wl.make_activations(seed, 1, (V, K), 0.3, "bf16")
    bias = wl.make_activations(seed, 2, (V,), 1.0, "fp32") if with_bias else None
    return A, W, bias


def _case(b, seed, R, V, K, with_bias):
    A, W, bias = _host_case(seed, R, V, K, with_bias)
    return b.to_device(A), b.to_device(W), (b.to_device(bias) if with_bias else None)


def test_static_scratch_entry_point_matches_twice_in_a_row():
    from paper_2509_25188_b200 import binding as b
    pred = torch.empty(128, dtype=torch.int32, device="cuda")
    conf = torch.empty(128, dtype=torch.float32, device="cuda")
    for call, (seed, R, V, K, with_bias) in enumerate([(11, 32, 20000, 512, True), (12, 100, 5000, 136, False)]):
        A, W, bias = _case(b, seed, R, V, K, with_bias)
        want_pred, want_conf, _ = b.lm_head_bf16(A, W, bias)
        torch.cuda.synchronize()
        before = torch.cuda.mem_get_info()[0]
        pred.fill_(-7)
        conf.fill_(-1.0)
        b.lm_head_bf16_static(A, W, bias, pred, conf)
        torch.cuda.synchronize()
        after = torch.cuda.mem_get_info()[0]
        assert np.array_equal(pred[:R].cpu().numpy(), want_pred.cpu().numpy()), "call %d" % call
        assert np.abs(conf[:R].cpu().numpy() - want_conf.cpu().numpy()).max() <= 1e-6, "call %d" % call
        assert (pred[R:] == -7).all() and (conf[R:] == -1.0).all()      # nothing written past R rows
        # the oracle on the same bytes: Eq. 3 where the top-2 gap is clear, Eq. 4 to 1e-3
        hA, hW, hbias = _host_case(seed, R, V, K, with_bias)
        ref = orc.linear(orc.widen(hA), hW)
        if with_bias:
            ref = ref + hbias.astype(np.float64)[None, :]
        rp, rc, gap = orc.confidence_head(ref)
        sure = gap > 1e-3 * np.abs(ref).max()
        assert sure.mean() > 0.5
        assert np.array_equal(pred[:R].cpu().numpy()[sure], rp[sure]), "call %d: ids differ from the oracle" % call
        assert np.abs(conf[:R].cpu().numpy() - rc)[sure].max() < 1e-3, "call %d: confidences differ from the oracle" % call
        if call > 0:
            assert after == before      # once the kernels are loaded, a call takes no device memory


def test_static_scratch_entry_point_refuses_sizes_beyond_its_array():
    from paper_2509_25188_b200 import binding as b
    A, W, bias = _case(b, 13, 129, 256, 64, False)
    pred = torch.empty(129, dtype=torch.int32, device="cuda")
    conf = torch.empty(129, dtype=torch.float32, device="cuda")
    with pytest.raises(b.L2pdError) as e:
        b.lm_head_bf16_static(A, W, None, pred, conf)       # R > 128
    assert e.value.status == -2
    # V beyond the limit is refused from the sizes alone (the pointers are never touched)
    st = b.lib.l2pd_lm_head_bf16_static(None, A.data_ptr(), W.data_ptr(), None, 32, 131073, 64,
                                        pred.data_ptr(), conf.data_ptr(), 1)
    assert st == -2
