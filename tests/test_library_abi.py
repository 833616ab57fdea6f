"""The C-ABI library builds, loads without a GPU and exports every symbol include/l2pd.h declares."""
from __future__ import annotations

import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "l2pd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(l2pd_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2509_25188_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert "l2pd_init" in names and "l2pd_denoise_step" in names and "l2pd_decode" in names
    for n in names:
        assert hasattr(lib, n), "%s is declared in l2pd.h but not exported" % n


def test_binding_lists_the_same_symbols():
    from paper_2509_25188_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_null_arguments_are_refused_without_a_gpu():
    from paper_2509_25188_b200 import binding
    assert binding.lib.l2pd_init(None, None, 0, None) == -1
    assert binding.lib.l2pd_num_active(None) == 0
    assert binding.lib.l2pd_last_error(None) == b""
    binding.lib.l2pd_destroy(None)
    assert binding.lib.l2pd_lm_head_scratch_elems(32, 126464) == 3 * 1976 * 128


def test_struct_layouts_match_the_header():
    from paper_2509_25188_b200 import binding
    assert ctypes.sizeof(binding.Config) == 19 * 4
    assert ctypes.sizeof(binding.Weights) == 15 * 8
    assert ctypes.sizeof(binding.StepOut) == 10 * 8
