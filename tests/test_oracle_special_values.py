"""Pins for the oracle's dINT variants with the special value c = step / 2^shift (Section 4.2:
"half of the chosen step size, which is a power of two"; App. A.5 sweeps c / step = 0.5, 0.25,
0.125).  shift = 1 must be Eq. 5 / Eq. 6 themselves; for the others the format is pinned by
what defines it: the level set, round trips, nearest-level behaviour and brute force.
"""
import numpy as np
import pytest

import oracle


def unpack(codes):
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


def test_shift_one_is_eq5_and_eq6():
    rng = np.random.default_rng(3)
    for s in (2.0 ** -6, 0.013, 1.0):
        for z in (0, 4, 13):
            xs = (rng.standard_normal(400) * 3 * s).astype(np.float32)
            xs = np.concatenate([xs, np.float32(s) * np.array([0.25, -0.25, 0.75, -0.75, 0.5, 0], np.float32)])
            for x in xs:
                assert oracle.dint_quantize_fmt(float(x), s, z, 1) == oracle.dint_quantize(float(x), s, z)
            for code in range(16):
                assert oracle.dint_dequantize_fmt(code, s, z, 1) == oracle.dint_dequantize(code, s, z)
            assert np.array_equal(oracle.dint_table_fmt(z, 1), oracle.dint_table2(z))


@pytest.mark.parametrize("shift", [1, 2, 3])
def test_level_set_written_out(shift):
    s = 0.375
    c = s / 2 ** shift
    for z in range(14):
        levels = [(code - z) * s for code in range(14)] + [c, -c]
        got = [oracle.dint_dequantize_fmt(code, s, z, shift) for code in range(16)]
        assert got == levels
        assert len(set(levels)) == 16
        t = oracle.dint_table_fmt(z, shift)
        assert list(t) == [(code - z) * 2 ** shift for code in range(14)] + [1, -1]
        assert [float(v) * c for v in t] == levels          # table times the unit is the value
        assert np.abs(t.astype(int)).max() <= 13 * 2 ** shift <= 127


@pytest.mark.parametrize("shift", [1, 2, 3])
@pytest.mark.parametrize("s", [2.0 ** -6, 0.1, 3.7e-3])
def test_round_trip_of_every_code(shift, s):
    for z in range(14):
        for code in range(16):
            x = oracle.dint_dequantize_fmt(code, s, z, shift)
            assert oracle.dint_quantize_fmt(x, s, z, shift) == code


@pytest.mark.parametrize("shift", [2, 3])
def test_nearest_level_away_from_boundaries(shift):
    """Inside the range every value goes to the nearest of the 16 levels (that is what puts the
    special thresholds at the midpoints c/2 and (c + s)/2)."""
    s, z = 2.0 ** -5, 6
    c = s / 2 ** shift
    levels = np.array([(code - z) * s for code in range(14)] + [c, -c])
    xs = np.linspace(-z * s, (13 - z) * s, 5001).astype(np.float32)
    for x in xs:
        d = np.abs(levels - float(x))
        order = np.argsort(d)
        if d[order[1]] - d[order[0]] < 1e-3 * s:
            continue                                           # too close to a boundary
        assert oracle.dint_quantize_fmt(float(x), s, z, shift) == order[0]


@pytest.mark.parametrize("shift", [2, 3])
def test_threshold_strictness_follows_eq5(shift):
    s, z = 2.0 ** -4, 5
    c = s / 2 ** shift
    lower, upper = c / 2, (c + s) / 2                         # exact in binary32
    assert oracle.dint_quantize_fmt(lower, s, z, shift) == z          # x = c/2 is not special
    assert oracle.dint_quantize_fmt(np.nextafter(np.float32(lower), np.float32(1)), s, z, shift) == 14
    assert oracle.dint_quantize_fmt(upper, s, z, shift) == 14         # x = (c+s)/2 is
    assert oracle.dint_quantize_fmt(np.nextafter(np.float32(upper), np.float32(1)), s, z, shift) == z + 1
    assert oracle.dint_quantize_fmt(-upper, s, z, shift) == 15
    assert oracle.dint_quantize_fmt(-lower, s, z, shift) == z


@pytest.mark.parametrize("shift", [2, 3])
@pytest.mark.parametrize("group", [0, 128])
def test_pack_and_layer(shift, group):
    rng = np.random.default_rng(10 + shift)
    M, N, K = 5, 24, 256
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    X = rng.standard_normal((M, K)).astype(np.float16)
    bias = (rng.standard_normal(N) * 0.1).astype(np.float32)
    codes, scales, zeros = oracle.pack_weights_fmt(W, None, group, shift)
    # step sizes and zero-points do not depend on the special value; codes differ only where
    # a value lies in one of the special bands of either format
    c1, s1, z1 = oracle.pack_weights(W, None, group)
    assert np.array_equal(scales, s1) and np.array_equal(zeros, z1)
    glen = group or K
    sfull = np.repeat(scales.T, glen, axis=1).astype(np.float64)
    zfull = np.repeat(zeros.T, glen, axis=1).astype(np.int64)
    c = unpack(codes).astype(np.int64)
    unit = sfull / 2 ** shift
    deq = np.where(c == 14, unit, np.where(c == 15, -unit, (c - zfull) * sfull))
    err = np.abs(W.astype(np.float64) - deq)
    assert np.all(err <= sfull / 2 * (1 + 1e-5))
    near = np.abs(W.astype(np.float64)) <= unit                 # around zero the error shrinks with c
    assert np.all(err[near] <= (unit / 2 * (1 + 1e-5) + 1e-12)[near])
    assert (c == 14).any() and (c == 15).any()
    # the layer: brute-force integers, then the real-valued meaning
    Xq, tok = oracle.quantize_act(X)
    acc, Y, wide = oracle.linear_fmt(Xq, tok, codes, scales, zeros, bias, group, shift)
    lv = np.where(c == 14, 1, np.where(c == 15, -1, (c - zfull) * 2 ** shift))
    G = K // glen
    want = np.stack([Xq.astype(np.int64)[:, g * glen:(g + 1) * glen] @ lv[:, g * glen:(g + 1) * glen].T
                     for g in range(G)])
    assert np.array_equal(acc, want)
    real = (want * (scales.astype(np.float64) / 2 ** shift)[:, None, :]).sum(0) * tok.astype(np.float64)[:, None] + bias
    assert np.allclose(wide, real, rtol=1e-12, atol=1e-15)
    got = oracle.bf16_bits_to_float(Y).astype(np.float64)
    assert np.all(np.abs(got - wide) <= np.abs(wide) * 2.0 ** -8 + 1e-6)
    # equals "dequantize, then multiply"
    assert np.allclose(real, (Xq.astype(np.float64) * tok[:, None]) @ deq.T + bias, rtol=1e-9, atol=1e-12)
