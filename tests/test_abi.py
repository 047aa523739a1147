"""The C-ABI library loads, exports every symbol the public header declares, and rejects bad
arguments on the host before touching a device (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2605_26266_b200 import build
    build.build_library()
    from paper_2605_26266_b200 import binding as b
    return b


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "kvq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvq_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_exported(binding):
    syms = declared_symbols()
    assert {"kvq_quantize_append", "kvq_attn_corrected", "kvq_cache_bytes", "kvq_unpack_codes",
            "kvq_attn_workspace_bytes", "kvq_attn_kernel_launches", "kvq_status_string", "kvq_last_cuda_error", "kvq_version"} <= set(syms)
    for s in syms:
        assert hasattr(binding.lib, s), s


def test_version_and_status_strings(binding):
    assert binding.kvq_version() == 1
    for code in range(0, -8, -1):
        assert binding.lib.kvq_status_string(code)
    assert binding.lib.kvq_status_string(-99) == b"unknown status"


def test_cache_bytes_accounting(binding):
    d = binding.kvq_cache_desc(2, 32, 128, 2, 32, 0, 4096)
    sizes = binding.kvq_cache_bytes(d)
    tok = 2 * 32 * 4096
    assert sizes == [tok * 32, tok * 32, tok * 4, tok * 4, tok * 8, tok * 8]
    # effective bits per element: 2 + 24/32
    assert 8 * (sizes[0] + sizes[2] + sizes[4]) / (tok * 128) == 2.75


def test_argument_errors_without_gpu(binding):
    b = binding
    sizes = (C.c_size_t * 6)()
    bad = b.kvq_cache_desc(1, 2, 96, 2, 32, 0, 128)
    assert b.lib.kvq_cache_bytes(C.byref(bad), sizes) == b.KVQ_ERR_UNSUPPORTED
    bad = b.kvq_cache_desc(1, 2, 128, 2, 48, 0, 128)
    assert b.lib.kvq_cache_bytes(C.byref(bad), sizes) == b.KVQ_ERR_INVALID_ARG
    bad = b.kvq_cache_desc(1, 2, 128, 3, 32, 0, 128)
    assert b.lib.kvq_cache_bytes(C.byref(bad), sizes) == b.KVQ_ERR_UNSUPPORTED
    bad = b.kvq_cache_desc(2048, 32, 128, 2, 32, 0, 128)        # batch * heads is a grid dimension: at most 65535
    assert b.lib.kvq_cache_bytes(C.byref(bad), sizes) == b.KVQ_ERR_UNSUPPORTED
    ok = b.kvq_cache_desc(2047, 32, 128, 2, 32, 0, 128)
    assert b.lib.kvq_cache_bytes(C.byref(ok), sizes) == b.KVQ_OK
    bad = b.kvq_cache_desc(1, 2, 128, 2, 32, 0, 100)
    assert b.lib.kvq_cache_bytes(C.byref(bad), sizes) == b.KVQ_ERR_INVALID_ARG
    assert b.lib.kvq_cache_bytes(None, sizes) == b.KVQ_ERR_INVALID_ARG
    ok = b.kvq_cache_desc(1, 2, 128, 2, 32, b.KVQ_ROTATE_K, 256)
    s = b.kvq_strides(2 * 256 * 128, 256 * 128, 128)
    # null cache buffers
    assert b.lib.kvq_quantize_append(C.byref(ok), 0, 0x1000, 0x1000, s, 16, None) == b.KVQ_ERR_INVALID_ARG
    for f in ("k_codes", "v_codes", "k_scale", "v_scale", "k_zero", "v_zero"):
        setattr(ok, f, 0x10000)
    assert b.lib.kvq_quantize_append(C.byref(ok), 250, 0x1000, 0x1000, s, 16, None) == b.KVQ_ERR_CAPACITY
    assert b.lib.kvq_quantize_append(C.byref(ok), 0, 0x1004, 0x1000, s, 16, None) == b.KVQ_ERR_ALIGNMENT
    assert b.lib.kvq_quantize_append(C.byref(ok), 0, None, 0x1000, s, 16, None) == b.KVQ_ERR_INVALID_ARG
    s_bad = b.kvq_strides(2 * 256 * 128, 256 * 128, 100)
    assert b.lib.kvq_quantize_append(C.byref(ok), 0, 0x1000, 0x1000, s_bad, 16, None) == b.KVQ_ERR_ALIGNMENT
    assert b.lib.kvq_quantize_append(C.byref(ok), 0, 0x1000, 0x1000, s, 0, None) == b.KVQ_OK      # no-op
    args = lambda begin, n_cache, m, n_cur, flags: b.lib.kvq_attn_corrected(
        C.byref(ok), begin, n_cache, 0x1000, s, 0x1000, 0x1000, s, m, n_cur, 0x1000, s, 0.088, flags,
        None, None, None, 0, None, None)
    assert args(0, 300, 16, 16, 1) == b.KVQ_ERR_CAPACITY
    assert args(8, 16, 16, 16, 1) == b.KVQ_ERR_ALIGNMENT
    assert args(0, 16, 16, 0, 1) == b.KVQ_ERR_INVALID_ARG
    assert args(0, 16, 16, 16, 1 << 20) == b.KVQ_ERR_INVALID_ARG
    assert args(0, 16, 0, 16, 1 | b.KVQ_KERNEL_MMA_SYNC) == b.KVQ_OK                             # m = 0: no-op
    assert b.lib.kvq_unpack_codes(C.byref(ok), 2, 0, 4, 0x1000, None) == b.KVQ_ERR_INVALID_ARG
    assert b.lib.kvq_unpack_codes(C.byref(ok), 0, 250, 16, 0x1000, None) == b.KVQ_ERR_CAPACITY


def test_ring_cache_argument_rules_without_gpu(binding):
    b = binding
    ring = b.kvq_cache_desc(1, 2, 128, 2, 32, b.KVQ_ROTATE_K | b.KVQ_RING, 256)
    for f in ("k_codes", "v_codes", "k_scale", "v_scale", "k_zero", "v_zero"):
        setattr(ring, f, 0x10000)
    s = b.kvq_strides(2 * 256 * 128, 256 * 128, 128)
    # positions are unbounded, but one append and one window hold at most `capacity` tokens
    assert b.lib.kvq_quantize_append(C.byref(ring), 10 ** 9, 0x1000, 0x1000, s, 0, None) == b.KVQ_OK
    assert b.lib.kvq_quantize_append(C.byref(ring), 250, 0x1000, 0x1000, s, 257, None) == b.KVQ_ERR_CAPACITY
    args = lambda begin, n_cache, m: b.lib.kvq_attn_corrected(
        C.byref(ring), begin, n_cache, 0x1000, s, 0x1000, 0x1000, s, m, 16, 0x1000, s, 0.088, 1,
        None, None, None, 0, None, None)
    assert args(1024, 256, 0) == b.KVQ_OK            # m = 0: checks only
    assert args(1024, 257, 0) == b.KVQ_ERR_CAPACITY
    assert args(1000, 16, 0) == b.KVQ_ERR_ALIGNMENT
    assert b.lib.kvq_unpack_codes(C.byref(ring), 0, 250, 257, 0x1000, None) == b.KVQ_ERR_CAPACITY
    unknown = b.kvq_cache_desc(1, 2, 128, 2, 32, 16, 256)
    sizes = (C.c_size_t * 6)()
    assert b.lib.kvq_cache_bytes(C.byref(unknown), sizes) == b.KVQ_ERR_INVALID_ARG


def test_wait_budget_argument_and_status_word_mapping(binding):
    b = binding
    assert b.lib.kvq_set_wait_budget_cycles(0xFFFF0001) == b.KVQ_ERR_INVALID_ARG
    assert b.lib.kvq_set_wait_budget_cycles(0) == b.KVQ_OK
    assert b.kvq_status_word_result(0) == b.KVQ_OK
    for word in (100, 204, 301, 404, -1):
        assert b.kvq_status_word_result(word) == b.KVQ_ERR_TIMEOUT
