"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol
the header declares, answers the size queries, and rejects bad arguments before touching
a device."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def w4a8():
    entry.build()
    import paper_2311_05161_b200 as mod
    return mod


def test_library_exports_every_declared_symbol(w4a8):
    header = open(os.path.join(ROOT, "include", "w4a8.h")).read()
    declared = set(re.findall(r"\b(w4a8_[a-z0-9_]+)\s*\(", header))
    assert declared == set(w4a8.EXPORTS)
    raw = ctypes.CDLL(w4a8.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name
    assert "sm_100a" in w4a8.version()


def test_size_queries(w4a8):
    # header + FP32 steps + u8 zero-points (each 256-aligned) + 8 KiB per 128x128 tile
    assert w4a8.packed_bytes(768, 768, 0) == 256 + 3072 + 768 + 36 * 8192
    assert w4a8.packed_bytes(768, 768, 128) == 256 + 6 * 3072 + 6 * 768 + 36 * 8192
    assert w4a8.packed_bytes(200, 256, 0) == 256 + 1024 + 256 + 2 * 2 * 8192   # N padded to 256
    assert w4a8.packed_bytes(768, 700, 0) == 0          # K % 128
    assert w4a8.packed_bytes(7, 768, 0) == 0            # N % 8
    assert w4a8.packed_bytes(768, 768, 64) == 0         # group size
    assert w4a8.packed_bytes(768, 1 << 19, 0) == 0      # K too large for INT32 sums
    assert w4a8.linear_workspace_bytes(16, 768, 768, 0) >= 256
    assert w4a8.linear_workspace_bytes(0, 768, 768, 0) == 0
    o = w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=3, tok_tile=16)
    need = w4a8.linear_workspace_bytes(16, 768, 768, 0, o)
    assert need >= 256 + 3 * 16 * 768 * 4
    assert w4a8.linear_workspace_bytes(16, 768, 768, 0, w4a8.make_opts(tok_tile=48)) == 0
    assert w4a8.linear_workspace_bytes(16, 768, 768, 128, w4a8.make_opts(tok_tile=256)) == 0
    assert w4a8.linear_workspace_bytes(16, 768, 768, 0, w4a8.make_opts(split_k=7)) == 0


def test_dint4_table_matches_eq6(w4a8):
    for z in range(14):
        assert w4a8.dint4_table(z) == [2 * (c - z) for c in range(14)] + [1, -1]


def test_argument_validation_needs_no_device(w4a8):
    lib = w4a8.lib
    p = ctypes.c_void_p
    good = 0x10000          # never dereferenced: validation fails first
    # NULL
    assert lib.w4a8_pack_weights(None, None, 768, 768, 0, 1.0, p(good), 1 << 30, None) == 1
    assert lib.w4a8_quantize_act(p(good), None, 16, 768, None, p(good), None) == 1
    assert lib.w4a8_linear(p(good), p(good), p(good), None, 16, 768, 768, 0, None, p(good), 1 << 20, None) == 1
    assert lib.w4a8_linear(p(good), p(good), p(good), None, 16, 768, 768, 0, p(good), None, 1 << 20, None) == 1
    # shape
    assert lib.w4a8_pack_weights(p(good), None, 768, 700, 0, 1.0, p(good), 1 << 30, None) == 2
    assert lib.w4a8_pack_weights(p(good), None, 768, 768, 32, 1.0, p(good), 1 << 30, None) == 2
    assert lib.w4a8_pack_weights(p(good), None, 768, 768, 0, 0.0, p(good), 1 << 30, None) == 2
    assert lib.w4a8_pack_weights(p(good), None, 768, 768, 0, 1.5, p(good), 1 << 30, None) == 2
    assert lib.w4a8_quantize_act(p(good), None, 0, 768, p(good), p(good), None) == 2
    assert lib.w4a8_linear(p(good), p(good), p(good), None, 16, 770, 768, 0, p(good), p(good), 1 << 20, None) == 2
    # alignment
    assert lib.w4a8_pack_weights(p(good + 2), None, 768, 768, 0, 1.0, p(good), 1 << 30, None) == 3
    assert lib.w4a8_pack_weights(p(good), None, 768, 768, 0, 1.0, p(good + 16), 1 << 30, None) == 3
    assert lib.w4a8_quantize_act(p(good), p(good + 4), 16, 768, p(good), p(good), None) == 3
    assert lib.w4a8_linear(p(good + 8), p(good), p(good), None, 16, 768, 768, 0, p(good), p(good), 1 << 20, None) == 3
    assert lib.w4a8_linear(p(good), p(good), p(good), None, 16, 768, 768, 0, p(good), p(good + 128), 1 << 20, None) == 3
    # buffers too small
    assert lib.w4a8_pack_weights(p(good), None, 768, 768, 0, 1.0, p(good), 1000, None) == 4
    assert lib.w4a8_linear(p(good), p(good), p(good), None, 16, 768, 768, 0, p(good), p(good), 100, None) == 4
    # options
    o = w4a8.make_opts(path=9)
    assert lib.w4a8_linear_ex(p(good), p(good), p(good), None, 16, 768, 768, 0, p(good), p(good), 1 << 20, None, ctypes.byref(o)) == 2
