"""Host-side checks of the C-ABI library: it loads, exports what the header declares, and
validates arguments before touching a device (no compute calls here)."""
import ctypes as C
import os
import re

import pytest

from paper_2503_00979_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "mkv.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(mkv_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_sizes_match_the_header(lib):
    # int x12, pointer, size_t / 7 pointers, 2 x int32, int64
    assert C.sizeof(binding.mkv_params) == 12 * 4 + 8 + 8 + 4 * 4 + 8
    assert C.sizeof(binding.mkv_view) == 7 * 8 + 2 * 4 + 8 + 8


def test_defaults(lib):
    p = binding.mkv_default_params()
    assert (p.fusion, p.dtype, p.evict_interval, p.kernel, p.splits, p.workspace) == (0, 0, 1, 0, 0, None)


@pytest.mark.parametrize("field,value", [("layers", 0), ("batch", -1), ("n_kv_heads", 3), ("head_dim", 96), ("C", 0),
                                         ("R", 0), ("fusion", 2), ("dtype", 5), ("n_q_heads", 17 * 8)])
def test_invalid_parameters_are_rejected_before_any_device_use(lib, field, value):
    p = binding.mkv_default_params()
    p.layers, p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim, p.C, p.R = 1, 1, 8, 2, 64, 16, 4
    assert binding.mkv_workspace_bytes(p) > 0
    setattr(p, field, value)
    assert binding.mkv_workspace_bytes(p) == 0
    st, h = binding.mkv_create_ex(p)
    assert st == binding.INVALID_ARG and h is None


def test_workspace_size_accounts_for_the_cache(lib):
    p = binding.mkv_default_params()
    p.layers, p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim, p.C, p.R = 32, 1, 32, 8, 128, 2000, 32
    n = binding.mkv_workspace_bytes(p)
    kv = 2 * 256 * 2032 * 128 * 2
    assert kv < n < 1.25 * kv


def test_null_handles(lib):
    assert lib.mkv_create_ex(None, None) == binding.INVALID_ARG
    assert lib.mkv_decode_step(None, None, None, None, None, None) == binding.INVALID_ARG
    assert lib.mkv_prefill(None, None, None, None, 1, None) == binding.INVALID_ARG
    assert lib.mkv_cache_view(None, 0, None) == binding.INVALID_ARG
    assert lib.mkv_sync(None, None) == binding.INVALID_ARG
    assert binding.mkv_last_error(None) == ""
    assert binding.mkv_launch_count(None) == 0
    lib.mkv_destroy(None)


def test_no_device_means_an_error_not_a_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    st, h = binding.mkv_create(1, 1, 8, 2, 64, 16, 4, 0)
    assert st == binding.CUDA and h is None


def test_coarse_grained_eviction_adds_its_interval_to_the_capacity(lib):
    # evict_interval T > 1: the cache holds up to C + R + T tokens (the scoring step appends before it drops)
    p = binding.mkv_default_params()
    p.layers, p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim, p.C, p.R = 2, 1, 8, 2, 128, 1000, 32
    base = binding.mkv_workspace_bytes(p)
    p.evict_interval = 8
    grown = binding.mkv_workspace_bytes(p)
    units, row = 2 * 1 * 2, 128 * 2
    assert grown - base >= 2 * units * 8 * row          # at least K and V rows of the 8 extra slots
    p.evict_interval = 65                               # beyond what one compaction handles
    assert binding.mkv_workspace_bytes(p) == 0
