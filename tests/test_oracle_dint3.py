"""Pins for the oracle's 3-bit dINT (Section 4.2 with b = 3: p = 2^3 - 3 = 5 uniform steps,
integer codes 0..5 and the two special codes 6 = +c, 7 = -c; the paper's 3-bit results are
Tables 10-11).  The scalar Eq. 5 / Eq. 6 routines are pinned for b = 3 in
test_oracle_format.py; here the row / group quantizer and the layer built on them."""
import numpy as np
import pytest

import oracle


def unpack(codes):
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


def test_level_set_and_table_written_out():
    s = 0.75
    for shift in (1, 2, 3):
        c = s / 2 ** shift
        for z in range(6):
            levels = [(code - z) * s for code in range(6)] + [c, -c]
            assert [oracle.dint_dequantize_fmt(code, s, z, shift, b=3) for code in range(8)] == levels
            assert len(set(levels)) == 8
            t = oracle.dint_table_fmt(z, shift, b=3)[:8]
            assert list(t) == [(code - z) * 2 ** shift for code in range(6)] + [1, -1]
            for code in range(8):
                assert oracle.dint_quantize_fmt(levels[code], s, z, shift, b=3) == code


def test_four_bit_entry_points_are_the_general_ones_at_b4():
    rng = np.random.default_rng(1)
    W = (rng.standard_normal((16, 256)) * 0.02).astype(np.float16)
    for group in (0, 128):
        a = oracle.pack_weights_bits(W, None, group, 4, 1)
        b = oracle.pack_weights(W, None, group)
        assert all(np.array_equal(x, y) for x, y in zip(a, b))


@pytest.mark.parametrize("group", [0, 128])
def test_reduces_to_textbook_minmax_with_six_levels(group):
    """Without values in a special band the quantizer is asymmetric Min-Max rounding to 0..5."""
    rng = np.random.default_rng(2)
    N, K = 12, 256
    # values on a coarse grid far from the bands around +-step/2: multiples of the step itself
    W = np.zeros((N, K), dtype=np.float16)
    glen = group or K
    for n in range(N):
        for g in range(K // glen):
            lo_i = -int(rng.integers(0, 6))
            vals = rng.integers(lo_i, lo_i + 6, size=glen)
            vals[0], vals[1] = lo_i, lo_i + 5                 # the range is exactly five steps
            W[n, g * glen:(g + 1) * glen] = vals * 2.0 ** -6
    codes, scales, zeros = oracle.pack_weights_bits(W, None, group, 3)
    c = unpack(codes).astype(np.int64)
    assert c.max() <= 5
    w64 = W.astype(np.float64)
    for n in range(N):
        for g in range(K // glen):
            seg = w64[n, g * glen:(g + 1) * glen]
            lo, hi = min(0.0, seg.min()), max(0.0, seg.max())
            step = (hi - lo) / 5
            z = int(np.clip(np.rint(-lo / step), 0, 5))
            assert scales[g, n] == np.float32(step) and zeros[g, n] == z
            assert np.array_equal(c[n, g * glen:(g + 1) * glen], np.clip(np.rint(seg / step) + z, 0, 5))


@pytest.mark.parametrize("shift", [1, 2])
@pytest.mark.parametrize("group", [0, 128])
def test_pack_and_layer_three_bits(shift, group):
    rng = np.random.default_rng(30 + shift)
    M, N, K = 5, 24, 256
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    X = rng.standard_normal((M, K)).astype(np.float16)
    bias = (rng.standard_normal(N) * 0.1).astype(np.float32)
    codes, scales, zeros = oracle.pack_weights_bits(W, None, group, 3, shift)
    glen = group or K
    sfull = np.repeat(scales.T, glen, axis=1).astype(np.float64)
    zfull = np.repeat(zeros.T, glen, axis=1).astype(np.int64)
    c = unpack(codes).astype(np.int64)
    assert c.max() <= 7 and zeros.max() <= 5
    unit = sfull / 2 ** shift
    deq = np.where(c == 6, unit, np.where(c == 7, -unit, (c - zfull) * sfull))
    err = np.abs(W.astype(np.float64) - deq)
    assert np.all(err <= sfull / 2 * (1 + 1e-5))              # never worse than plain rounding
    near = np.abs(W.astype(np.float64)) <= unit
    assert np.all(err[near] <= (unit / 2 * (1 + 1e-5) + 1e-12)[near])
    assert (c == 6).any() and (c == 7).any() and (c == 0).any() and (c == 5).any()
    Xq, tok = oracle.quantize_act(X)
    acc, Y, wide = oracle.linear_bits(Xq, tok, codes, scales, zeros, bias, group, 3, shift)
    lv = np.where(c == 6, 1, np.where(c == 7, -1, (c - zfull) * 2 ** shift))
    G = K // glen
    want = np.stack([Xq.astype(np.int64)[:, g * glen:(g + 1) * glen] @ lv[:, g * glen:(g + 1) * glen].T
                     for g in range(G)])
    assert np.array_equal(acc, want)
    # one entry by a Python triple loop (a transposed operand or a wrong table cannot pass)
    tot = 0
    for k in range(glen):
        tot += int(Xq[3, k]) * int(lv[7, k])
    assert acc[0, 3, 7] == tot
    real = (want * (scales.astype(np.float64) / 2 ** shift)[:, None, :]).sum(0) * tok.astype(np.float64)[:, None] + bias
    assert np.allclose(wide, real, rtol=1e-12, atol=1e-15)
    got = oracle.bf16_bits_to_float(Y).astype(np.float64)
    assert np.all(np.abs(got - wide) <= np.abs(wide) * 2.0 ** -8 + 1e-6)
    assert np.allclose(real, (Xq.astype(np.float64) * tok[:, None]) @ deq.T + bias, rtol=1e-9, atol=1e-12)


def test_exact_grid_recovery_three_bits():
    # weights drawn on a 3-bit dINT grid with codes 0 and 5 in every row: packing returns them
    rng = np.random.default_rng(9)
    N, K, s = 16, 128, 2.0 ** -5
    z = rng.integers(1, 5, size=N)        # (with z = 0 or 5 a special value would widen the range)
    c = rng.integers(0, 8, size=(N, K))
    c[:, 0], c[:, 1] = 0, 5
    val = np.where(c == 6, s / 2, np.where(c == 7, -s / 2, (c - z[:, None]) * s))
    codes, scales, zeros = oracle.pack_weights_bits(val.astype(np.float16), None, 0, 3)
    assert np.array_equal(zeros[0], z) and np.all(scales == np.float32(s))
    assert np.array_equal(unpack(codes), c)
