"""Pins for the oracle's dINT format routines against what Eq. 5 / Eq. 6 fix.

Nothing here compares the oracle with itself only: expected values are read off
the paper's inequalities (golden file), enumerated from Eq. 6 by hand, or come
from numpy / torch conversion routines.
"""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_level_count_matches_section_4_2():
    # "the quantization range represents integers from 0 to 2^b - 3"
    assert oracle.dint_p(4) == 13
    assert oracle.dint_p(3) == 5
    assert oracle.dint_p(8) == 253


def test_half_conversion_against_numpy_all_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(b)) for b in bits], dtype=np.float32)
    finite = np.isfinite(want)
    assert np.array_equal(got[finite].view(np.uint32), want[finite].view(np.uint32))
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(np.isinf(got), np.isinf(want))


def test_bf16_rounding_against_torch():
    rng = np.random.default_rng(1)
    vals = rng.standard_normal(20000).astype(np.float32) * np.float32(37.0)
    # exact ties and their neighbours: low 16 bits 0x8000 with even / odd keep bit
    ties = np.array([0x3F808000, 0x3F818000, 0x3F808001, 0x3F807FFF, 0xBF808000,
                     0xBF818000, 0x00000000, 0x80000000, 0x7F7FFFFF, 0x00008000,
                     0x00018000], dtype=np.uint32).view(np.float32)
    vals = np.concatenate([vals, ties])
    want = torch.from_numpy(vals).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.float_to_bf16(float(v)) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, want)


def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "dint4_eq5_probes.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            ratio, z, code = line.split()[:3]
            rows.append((float.fromhex(ratio), int(z), int(code), line))
    return rows


def test_eq5_threshold_and_tie_probes_from_golden_file():
    s = np.float32(2.0 ** -6)
    rows = _golden_rows()
    assert len(rows) >= 25
    for ratio, z, code, line in rows:
        r32 = np.float32(ratio)
        assert float(r32) == ratio, "probe must be exact in binary32: " + line
        x = np.float32(r32 * s)
        assert oracle.dint_quantize(float(x), float(s), z) == code, line


@pytest.mark.parametrize("b", [3, 4])
def test_eq6_levels_written_out(b):
    # Eq. 6 enumerated by hand: integer levels (code - z) s, then +s/2, -s/2.
    p = (1 << b) - 3
    s = 0.375
    for z in range(p + 1):
        levels = [(c - z) * s for c in range(p + 1)] + [s / 2, -s / 2]
        got = [oracle.dint_dequantize(c, s, z, b) for c in range(p + 3)]
        assert got == levels
        assert len(set(levels)) == (1 << b)          # all 2^b codes are distinct values
        t2 = oracle.dint_table2(z, b)
        assert list(t2) == [2 * (c - z) for c in range(p + 1)] + [1, -1]
        # the doubled table times s/2 is the dequantized value, exactly
        assert [float(t) * (s / 2) for t in t2] == levels


@pytest.mark.parametrize("b", [3, 4])
@pytest.mark.parametrize("s", [2.0 ** -6, 0.1, 3.7e-3, 1.0])
def test_round_trip_of_every_code(b, s):
    # Q(DQ(code)) = code for every code and every zero-point (Eq. 5 inverts Eq. 6).
    p = (1 << b) - 3
    for z in range(p + 1):
        for code in range(p + 3):
            x = oracle.dint_dequantize(code, s, z, b)
            assert oracle.dint_quantize(x, s, z, b) == code, (b, s, z, code)


def test_special_codes_are_the_two_above_p():
    s = 0.25
    for z in (0, 6, 13):
        assert oracle.dint_quantize(0.5 * s, s, z) == 14      # c1 = +s/2
        assert oracle.dint_quantize(-0.5 * s, s, z) == 15     # c2 = -s/2
        assert oracle.dint_dequantize(14, s, z) == 0.5 * s
        assert oracle.dint_dequantize(15, s, z) == -0.5 * s


def _sweep(s, z, n=4001):
    lo, hi = -z * s, (13 - z) * s
    xs = np.linspace(lo - s, hi + s, n).astype(np.float32)
    codes = np.array([oracle.dint_quantize(float(x), s, z) for x in xs])
    deq = np.array([oracle.dint_dequantize(int(c), s, z) for c in codes], dtype=np.float64)
    return xs.astype(np.float64), codes, deq, lo, hi


@pytest.mark.parametrize("z", [0, 1, 5, 12, 13])
@pytest.mark.parametrize("s", [2.0 ** -5, 0.013])
def test_quantizer_invariants(z, s):
    xs, codes, deq, lo, hi = _sweep(s, z)
    s32 = float(np.float32(s))
    # idempotent
    again = np.array([oracle.dint_quantize(float(np.float32(d)), s, z) for d in deq])
    assert np.array_equal(again, codes)
    # monotone in value, apart from the clamp edge the literal Eq. 5 leaves (z = 13 / z = 0:
    # a positive / negative value clamps to the zero level although s/2 exists)
    inside = (xs >= lo) & (xs <= hi)
    assert np.all(np.diff(deq[inside]) >= -1e-12)
    # error bounds inside the range: s/2 everywhere, s/4 within one step of zero
    err = np.abs(xs - deq)
    assert np.all(err[inside] <= s32 / 2 * (1 + 1e-6))
    near = inside & (np.abs(xs) <= s32)
    assert np.all(err[near] <= s32 / 4 * (1 + 1e-6))
    # the zero bin is exactly |x| <= s/4 (INT4's would be s/2)
    zero_bin = inside & (codes == z)
    assert np.all(np.abs(xs[zero_bin]) <= s32 / 4 * (1 + 1e-6))
    inner = inside & (np.abs(xs) < s32 / 4 * (1 - 1e-6))
    assert np.all(codes[inner] == z)


def test_all_16_codes_are_reachable_and_only_those():
    s, z = 2.0 ** -4, 6
    xs, codes, _, _, _ = _sweep(s, z, n=8001)
    assert set(codes.tolist()) == set(range(16))
