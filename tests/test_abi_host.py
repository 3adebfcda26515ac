"""Host-only checks of the C ABI: the library loads without a GPU, exports every function the
public header declares, and validates arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2405_06219_b200 import binding as B
from paper_2405_06219_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return B.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "skvq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(skvq_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == names


def cfg(**kw):
    base = dict(batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, k_bits=2, v_bits=2, group_size=128, window=128,
                max_tokens=4096)
    base.update(kw)
    return B.SkvqConfig(**base)


def test_version_and_strerror(lib):
    assert B.skvq_version() >= 100
    assert B.skvq_strerror(0) == "ok"
    for code in range(-6, 0):
        assert B.skvq_strerror(code) not in ("ok", "unknown error code")
    assert B.skvq_strerror(-99) == "unknown error code"


@pytest.mark.parametrize("kw,code", [
    (dict(head_dim=64), B.SKVQ_ERR_UNSUPPORTED), (dict(k_bits=3), B.SKVQ_OK), (dict(k_bits=1), B.SKVQ_ERR_UNSUPPORTED), (dict(v_bits=5), B.SKVQ_ERR_UNSUPPORTED),
    (dict(v_bits=8), B.SKVQ_ERR_UNSUPPORTED), (dict(group_size=16), B.SKVQ_ERR_UNSUPPORTED),
    (dict(n_q_heads=7), B.SKVQ_ERR_UNSUPPORTED), (dict(n_q_heads=32, n_kv_heads=2), B.SKVQ_ERR_UNSUPPORTED),
    (dict(batch=0), B.SKVQ_ERR_INVALID_ARG), (dict(window=-1), B.SKVQ_ERR_INVALID_ARG),
    (dict(max_tokens=0), B.SKVQ_ERR_INVALID_ARG), (dict(), B.SKVQ_OK), (dict(n_sink=5), B.SKVQ_OK), (dict(meta_fp8=1), B.SKVQ_OK), (dict(meta_fp8=2), B.SKVQ_ERR_INVALID_ARG),
    (dict(n_sink=-1), B.SKVQ_ERR_INVALID_ARG), (dict(n_sink=65), B.SKVQ_ERR_UNSUPPORTED), (dict(window=0, k_bits=4, group_size=32), B.SKVQ_OK),
])
def test_config_validation(lib, kw, code):
    assert B.skvq_check_config(cfg(**kw)) == code


def test_sizes_follow_the_documented_layout(lib):
    c = cfg(max_tokens=4096 + 5, group_size=32, k_bits=4)
    cap = B.skvq_quant_capacity(c)
    assert cap == 4032 and cap % B.SKVQ_TOKEN_ALIGN == 0          # round_up(4101 - 128, 64)
    sizes = B.skvq_cache_sizes(c)
    rows = 2 * 2 * cap
    assert sizes == [rows * 64, rows * 32, rows * 4 * 4, rows * 4 * 4, 2 * 2 * 128 * 128 * 2, 2 * 2 * 128 * 128 * 2]
    assert B.skvq_quant_capacity(cfg(max_tokens=10)) == B.SKVQ_TOKEN_ALIGN
    # stored bits per element of the quantized segment: 4 + 32/32 and 2 + 32/32 (N + 2*16/G)
    assert (sizes[0] + sizes[2]) * 8 / (rows * 128) == 5.0 and (sizes[1] + sizes[3]) * 8 / (rows * 128) == 3.0


def test_workspace_size_grows_with_splits(lib):
    """Workspace = [B][Hq][s_max] partials of 132 floats, where the flat partition has n_slots = n_splits * B * Hkv
    slots and a pair can spread over at most n_slots // Hkv + 2 of them (never over more than its 256-token
    units); batches above 32 put a header in front: 4 ints + prefix [B+1] + first sequence per slot [n_slots],
    padded to 64 ints."""
    def expect(batch, n_splits, hint):
        units = max(-(-(hint - 128) // 256), 1)
        n_slots = min(n_splits * batch * 2, units * batch * 2)
        s_max = min(n_slots // 2 + 2, units)
        hdr = 0 if batch <= 32 else (4 + batch + 1 + n_slots + 63) // 64 * 64
        return (hdr + batch * 8 * s_max * 132) * 4

    c = cfg()                                                 # B 2, Hq 8, Hkv 2, W 128
    one = B.skvq_workspace_size(c, 4096, 1)
    four = B.skvq_workspace_size(c, 4096, 4)
    assert one == expect(2, 1, 4096) and four == expect(2, 4, 4096) and four > one
    assert B.skvq_workspace_size(c, 4096, 1000) == expect(2, 1000, 4096)      # capped by the units that exist
    assert B.skvq_workspace_size(c, 300, 7) == expect(2, 7, 300)
    assert B.skvq_workspace_size(cfg(batch=40), 4096, 3) == expect(40, 3, 4096)
    assert B.skvq_workspace_size(c, 4096, 0) >= one
    assert B.skvq_workspace_size(cfg(head_dim=64), 4096, 0) == 0
    assert B.skvq_step_staging_size(c) == 2 * (2 * 2 * 128 * 2) + 2 * (2 * 8 * 128 * 2)


def test_calls_reject_bad_arguments_before_any_launch(lib):
    c = cfg()
    empty = B.SkvqCacheStruct()
    before = B.skvq_launch_count()
    rc = lib.skvq_quantize_append(ctypes.byref(c), ctypes.byref(empty), None, None, None, 1, None)
    assert rc == B.SKVQ_ERR_INVALID_ARG
    args = B.SkvqAttnArgs(0.1, 4096, 0, None, 0, None, None)
    assert lib.skvq_decode_attention(ctypes.byref(c), ctypes.byref(empty), None, None, ctypes.byref(args), None) \
        == B.SKVQ_ERR_INVALID_ARG
    # fake (never dereferenced) pointers: alignment, capacity and workspace checks are host-side
    fake = B.SkvqCacheStruct(*([0x1000] * 11), None, None, None)
    assert lib.skvq_quantize_append(ctypes.byref(c), ctypes.byref(fake), 0x1008, 0x1000, None, 1, None) \
        == B.SKVQ_ERR_MISALIGNED
    assert lib.skvq_quantize_append(ctypes.byref(c), ctypes.byref(fake), 0x1000, 0x1000, None, 5000, None) \
        == B.SKVQ_ERR_CAPACITY
    assert lib.skvq_quantize_append(ctypes.byref(c), ctypes.byref(fake), 0x1000, 0x1000, None, -1, None) \
        == B.SKVQ_ERR_INVALID_ARG
    misal = B.SkvqCacheStruct(0x1004, *([0x1000] * 10), None, None, None)
    nosink = cfg(n_sink=4)
    assert lib.skvq_quantize_append(ctypes.byref(nosink), ctypes.byref(fake), 0x1000, 0x1000, None, 1, None) \
        == B.SKVQ_ERR_INVALID_ARG                                  # sinks asked for, no sink buffers
    assert B.skvq_sink_bytes(nosink) == 2 * 2 * 4 * 128 * 2 and B.skvq_sink_bytes(cfg()) == 0
    assert lib.skvq_quantize_append(ctypes.byref(c), ctypes.byref(misal), 0x1000, 0x1000, None, 1, None) \
        == B.SKVQ_ERR_MISALIGNED
    assert lib.skvq_decode_attention(ctypes.byref(c), ctypes.byref(fake), 0x1000, 0x1000, ctypes.byref(args), None) \
        == B.SKVQ_ERR_WORKSPACE
    small = B.SkvqAttnArgs(0.1, 4096, 4, 0x1000, 64, None, None)
    assert lib.skvq_decode_attention(ctypes.byref(c), ctypes.byref(fake), 0x1000, 0x1000, ctypes.byref(small), None) \
        == B.SKVQ_ERR_WORKSPACE
    toolong = B.SkvqAttnArgs(0.1, 5000, 0, 0x1000, 1 << 30, None, None)
    assert lib.skvq_decode_attention(ctypes.byref(c), ctypes.byref(fake), 0x1000, 0x1000, ctypes.byref(toolong), None) \
        == B.SKVQ_ERR_CAPACITY
    assert B.skvq_launch_count() == before


def test_three_bit_rows_are_48_bytes(lib):
    sizes = B.skvq_cache_sizes(cfg(k_bits=3, v_bits=2, group_size=64))
    cap = B.skvq_quant_capacity(cfg(k_bits=3, v_bits=2, group_size=64))
    assert sizes[0] == 2 * 2 * cap * 48 and sizes[1] == 2 * 2 * cap * 32      # 128 three-bit fields = 48 bytes


def test_three_level_value_rows_are_26_bytes_and_keys_stay_binary(lib):
    c = cfg(k_bits=2, v_bits=B.SKVQ_BITS_TERNARY, group_size=64)
    assert B.skvq_check_config(c) == B.SKVQ_OK
    sizes, cap = B.skvq_cache_sizes(c), B.skvq_quant_capacity(c)
    assert sizes[0] == 2 * 2 * cap * 32 and sizes[1] == 2 * 2 * cap * 26      # five base-3 digits per byte: ceil(128 / 5)
    assert B.skvq_check_config(cfg(k_bits=B.SKVQ_BITS_TERNARY, v_bits=2)) == B.SKVQ_ERR_UNSUPPORTED
    for v in (5, 8, 14, 16):
        assert B.skvq_check_config(cfg(v_bits=v)) == B.SKVQ_ERR_UNSUPPORTED


def test_group_bounds_are_validated_on_the_host(lib):
    import numpy as np
    c = cfg(group_size=64)                                   # two groups per row, two KV heads
    ok = np.array([[0, 32, 128], [0, 96, 128]], np.int32)
    assert B.skvq_check_group_bounds(c, ok) == B.SKVQ_OK
    for bad in ([[0, 32, 128], [0, 48, 128]],                # not a multiple of the 32-channel granule
                [[0, 128, 128], [0, 64, 128]],               # an empty group
                [[32, 64, 128], [0, 64, 128]],               # does not start at 0
                [[0, 64, 96], [0, 64, 128]]):                # does not end at head_dim
        assert B.skvq_check_group_bounds(c, np.array(bad, np.int32)) == B.SKVQ_ERR_INVALID_ARG
    assert lib.skvq_check_group_bounds(ctypes.byref(c), None) == B.SKVQ_ERR_INVALID_ARG
    assert B.SKVQ_GROUP_GRANULE == 32
