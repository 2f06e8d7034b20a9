"""The C-ABI library loads and exports every symbol include/benes.h declares;
host-side argument checks and sizing helpers (no GPU work is launched)."""
import ctypes
import os
import re

import pytest

from paper_1912_04050_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared():
    src = open(os.path.join(ROOT, "include", "benes.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(benes_[a-z_0-9]+)\s*\(", src)))


def test_header_symbols_are_exported_and_bound(lib):
    names = _declared()
    assert "benes_route" in names and "benes_apply" in names and len(names) >= 12
    raw = ctypes.CDLL(binding.LIB_PATH)
    for name in names:
        assert hasattr(raw, name), name
        assert name in binding.SYMBOLS, "binding lacks %s" % name
    assert sorted(binding.SYMBOLS) == names


def test_checked_build_has_the_same_abi():
    path = build.build(debug=True)
    raw = ctypes.CDLL(path)
    for name in _declared():
        assert hasattr(raw, name), name
    assert raw.benes_debug_build() == 1
    assert ctypes.CDLL(binding.LIB_PATH).benes_debug_build() == 0


def test_sizing_helpers(lib):
    assert lib.benes_switch_words(10, 1) == 19 * 16
    assert lib.benes_switch_words(8, 16384) == 16384 * 15 * 4
    assert lib.benes_switch_words(1, 1) == 1
    assert lib.benes_switch_words(5, 2) == 2 * 9
    assert lib.benes_switch_words(26, 1) == 51 * (1 << 20)
    assert lib.benes_switch_words(0, 1) == 0 and lib.benes_switch_words(31, 1) == 0
    assert lib.benes_switch_words(8, 0) == 0
    m = lib.benes_fused_log2m()
    assert 8 <= m <= 16
    assert lib.benes_route_workspace_bytes(m, 4) == 0          # fused path needs no scratch
    assert lib.benes_route_workspace_bytes(20, 1) >= 24 << 20  # P, P', Q, Q' and 64-bit words
    assert lib.benes_apply_workspace_bytes(8, 20, 1) == 8 << 20
    assert lib.benes_apply_workspace_bytes(3, 20, 1) == 0
    assert lib.benes_apply_workspace_bytes(4, 1, 1) == 0


def test_argument_errors_are_reported_on_the_host(lib):
    one = ctypes.c_void_p(256)   # never dereferenced: checks fail first
    assert lib.benes_route(None, 10, 1, one, None) == binding.BENES_ERR_BADARG
    assert lib.benes_route(one, 10, 1, None, None) == binding.BENES_ERR_BADARG
    assert lib.benes_route(one, 0, 1, one, None) == binding.BENES_ERR_BADARG
    assert lib.benes_route(one, 31, 1, one, None) == binding.BENES_ERR_BADARG
    assert lib.benes_route(one, 10, 0, one, None) == binding.BENES_ERR_BADARG
    assert lib.benes_apply(None, one, one, 10, 1, None) == binding.BENES_ERR_BADARG
    assert lib.benes_apply_ex(one, one, ctypes.c_void_p(512), 3, 10, 1, None) == binding.BENES_ERR_BADARG
    assert lib.benes_apply_ex(one, one, one, 4, 10, 1, None) == binding.BENES_ERR_BADARG  # in == out
    assert lib.benes_validate_perm(None, 10, 1, None) == binding.BENES_ERR_BADARG
    assert lib.benes_route_host(None, 10, 1, one, None) == binding.BENES_ERR_BADARG
    assert lib.benes_apply_host(one, one, one, 5, 10, 1, None) == binding.BENES_ERR_BADARG
    assert lib.benes_set_workspace(ctypes.c_void_p(256), 0) == binding.BENES_ERR_BADARG
    assert lib.benes_set_workspace(ctypes.c_void_p(100), 1024) == binding.BENES_ERR_BADARG  # alignment


def test_options_are_validated(lib):
    k0 = lib.benes_get_option(binding.OPT_SAMPLE_LOG2K)
    c0 = lib.benes_get_option(binding.OPT_WALK_CAP)
    assert 2 <= k0 <= 8 and c0 >= 1
    for bad in (1, 9, -1):
        assert lib.benes_set_option(binding.OPT_SAMPLE_LOG2K, bad) == binding.BENES_ERR_BADARG
    assert lib.benes_set_option(binding.OPT_WALK_CAP, 0) == binding.BENES_ERR_BADARG
    assert lib.benes_set_option(99, 1) == binding.BENES_ERR_BADARG
    assert lib.benes_get_option(99) == binding.BENES_ERR_BADARG
    assert lib.benes_set_option(binding.OPT_SAMPLE_LOG2K, 0) == binding.BENES_OK
    assert lib.benes_get_option(binding.OPT_SAMPLE_LOG2K) == 0
    assert lib.benes_set_option(binding.OPT_SAMPLE_LOG2K, k0) == binding.BENES_OK
    assert lib.benes_get_option(binding.OPT_SAMPLE_LOG2K) == k0 and lib.benes_get_option(binding.OPT_WALK_CAP) == c0


def test_padded_size(lib):
    assert [lib.benes_padded_log2n(v) for v in (1, 2, 3, 4, 5, 1024, 1025, 1 << 30)] == [1, 1, 2, 2, 3, 10, 11, 30]
    assert lib.benes_padded_log2n(0) == 0 and lib.benes_padded_log2n((1 << 30) + 1) == 0
    one = ctypes.c_void_p(256)
    assert lib.benes_route_padded(one, 0, 1, one, None) == binding.BENES_ERR_BADARG
    assert lib.benes_apply_padded(one, one, ctypes.c_void_p(512), 3, 100, 1, None) == binding.BENES_ERR_BADARG


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    seen = {binding.status_string(s) for s in (0, -1, -2, -3, -4)}
    assert len(seen) == 5
    assert binding.status_string(-99) == "unknown status"


def test_binding_rejects_host_tensors_for_device_arguments():
    import torch
    with pytest.raises(TypeError):
        binding.benes_route(torch.zeros(4, dtype=torch.int32), 2, 1, torch.zeros(3, dtype=torch.int32), stream=0)
