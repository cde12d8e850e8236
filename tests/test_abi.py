"""The C-ABI library loads on a machine without a GPU and exports every declared entry point."""
import ctypes as C
import os
import re

import pytest

from paper_2508_17624_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "expertweave.h")).read()
    declared = set(re.findall(r"\b(ew_[a-z_]+)\s*\(", header))
    declared -= {"ew_pool_t", "ew_status_t"}
    assert {"ew_pool_create", "ew_load_adapter", "ew_unload_adapter", "ew_moe_forward", "ew_reroute"} <= declared
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(binding.EXPORTS)


def test_status_strings(lib):
    for i, name in enumerate(binding.STATUS_NAMES):
        assert lib.ew_status_str(i).decode() == name


def test_argument_errors_without_a_gpu(lib):
    assert lib.ew_pool_create(None, None) == 1
    h = C.c_void_p()
    bad = binding.EwConfig(-1, 1, 250, 128, 16, 1, 2, 2, 3, 64, 0, 1.0, 0, 0, 0, 0, 0)   # H not a multiple of 64
    assert lib.ew_pool_create(C.byref(bad), C.byref(h)) == 1
    bad = binding.EwConfig(-1, 1, 256, 128, 16, 1, 17, 2, 3, 64, 0, 1.0, 0, 0, 0, 0, 0)  # k > M
    assert lib.ew_pool_create(C.byref(bad), C.byref(h)) == 1
    pool = binding.Pool(device=-1, hidden=256, inter=128, num_experts=16, num_shared=1, top_k=2, max_adapters=2,
                        e_max=3, max_tokens=64)
    # an accounting-only pool refuses compute calls loudly instead of falling back to anything
    assert lib.ew_moe_forward(pool._h, 0, None, None, 4, None, None) == 9
    assert lib.ew_reroute(pool._h, 0, None, None, 4, None, None, None) == 9
    assert lib.ew_moe_forward(pool._h, 3, None, None, 4, None, None) == 1
    assert lib.ew_unload_adapter(pool._h, 0) == 4
    assert lib.ew_unload_adapter(pool._h, 7) == 1
    pool.destroy()
