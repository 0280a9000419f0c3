"""The C-ABI library builds, loads and exports every symbol that include/abs.h declares
(no compute calls: this runs without a GPU)."""
import ctypes
import os
import re

import pytest

import paper_2406_13936_b200 as pkg
from paper_2406_13936_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "abs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"^\s*(?:const\s+char\s*\*|int)\s+(\w+)\s*\(", text, flags=re.M)))


def test_header_declares_the_hot_path_calls():
    names = _declared_functions()
    for required in ("abs_test_stats", "abs_next_batch", "local_sgd_step", "local_adamw_step", "replica_average"):
        assert required in names


def test_library_builds_and_exports_every_declared_symbol():
    path = pkg.build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    for name in _declared_functions():
        assert hasattr(lib, name), "missing export %s" % name


def test_binding_covers_every_declared_symbol():
    declared = set(_declared_functions())
    bound = set(binding.EXPORTS) | {"abs_last_error", "abs_noalloc_last_error"}
    assert declared <= bound, declared - bound


def test_struct_sizes_match_the_header():
    assert ctypes.sizeof(binding.Stats) == 56
    assert ctypes.sizeof(binding.TestCfg) == 56
    assert ctypes.sizeof(binding.AdamWCfg) == 32
    assert ctypes.sizeof(binding.RoundCtl) == 32
    assert ctypes.sizeof(binding.RoundOpts) == 24


def test_create_fails_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(pkg.AbsError, match="no CPU fallback|CUDA"):
        pkg.Context(0)
