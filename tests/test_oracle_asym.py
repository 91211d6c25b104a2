"""Pins for the oracle's asymmetric token-wise activation path (App. A.1: Min-Max asymmetric
quantization of activations per token) and the linear layer built on it.

Expected values come from closed forms, from a float64 numpy restatement of textbook
asymmetric quantization, from exact grids, from Python-integer brute force and from the
algebraic identity that links the path to the symmetric contraction; none is the oracle's
own output.
"""
import numpy as np
import pytest

import oracle


def rand_x(M, K, seed, shift=0.0):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K)).astype(np.float32) + np.float32(shift)
    x[:, :3] *= 30
    return x.astype(np.float16)


def unpack(codes):
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


def test_range_ends_zero_and_step():
    M, K = 11, 512
    X = rand_x(M, K, 41, shift=0.7)
    Q, step, zx = oracle.quantize_act_asym(X)
    Xf = X.astype(np.float64)
    lo = np.minimum(Xf.min(1), 0)
    hi = np.maximum(Xf.max(1), 0)
    # the token's minimum maps to code 0 and its maximum to 255; the step is the range / 255
    assert np.all(Q[np.arange(M), Xf.argmin(1)] == 0)
    assert np.all(Q[np.arange(M), Xf.argmax(1)] == 255)
    assert np.array_equal(step, ((hi - lo).astype(np.float32) / np.float32(255)))
    # zero is exactly representable: a zero activation gets the zero-point as its code
    X0 = X.copy()
    X0[:, 7] = 0
    Q0, _, z0 = oracle.quantize_act_asym(X0)
    assert np.array_equal(Q0[:, 7].astype(np.int32), z0)
    # the zero-point is where the range says it is, within rounding
    assert np.all(np.abs(zx - (-lo) / (hi - lo) * 255) <= 0.5 + 1e-3)
    assert zx.min() >= 0 and zx.max() <= 255


def test_reduces_to_textbook_asymmetric_quantization():
    """Float64 numpy restatement: q = clip(rint(x / step) + z, 0, 255); compared wherever the
    real ratio is not within binary32 noise of a rounding tie."""
    M, K = 16, 768
    X = rand_x(M, K, 43, shift=-0.4)
    Q, step, zx = oracle.quantize_act_asym(X)
    Xf = X.astype(np.float64)
    lo = np.minimum(Xf.min(1), 0)
    hi = np.maximum(Xf.max(1), 0)
    a = (hi - lo) / 255.0
    z = np.clip(np.rint(-lo / a), 0, 255)
    ratio = Xf / a[:, None]
    want = np.clip(np.rint(ratio) + z[:, None], 0, 255)
    safe = np.abs(ratio - np.floor(ratio) - 0.5) > 1e-3
    zsafe = np.abs((-lo / a) - np.floor(-lo / a) - 0.5) > 1e-3
    assert safe.mean() > 0.99 and zsafe.all()
    assert np.array_equal(zx, z.astype(np.int32))
    assert np.array_equal(Q[safe], want[safe].astype(np.uint8))
    # reconstruction error: half a step everywhere
    err = np.abs(Xf - step.astype(np.float64)[:, None] * (Q.astype(np.float64) - zx[:, None]))
    assert np.all(err <= step.astype(np.float64)[:, None] * 0.5 * (1 + 1e-3))


def test_exact_grid_is_recovered():
    rng = np.random.default_rng(47)
    M, K = 9, 256
    a = 2.0 ** -4
    z = rng.integers(0, 256, M)
    z[0], z[1] = 0, 255                      # one-sided tokens
    q = rng.integers(0, 256, (M, K))
    q[:, 0], q[:, 1] = 0, 255                # both range ends present
    X = ((q - z[:, None]) * a).astype(np.float16)
    assert np.array_equal(X.astype(np.float64), (q - z[:, None]) * a)
    Q, step, zx = oracle.quantize_act_asym(X)
    assert np.array_equal(Q, q.astype(np.uint8))
    assert np.array_equal(zx, z.astype(np.int32))
    assert np.all(step == np.float32(a))


def test_one_sided_and_zero_tokens():
    K = 128
    X = np.zeros((3, K), dtype=np.float16)
    X[1] = np.linspace(0, 4, K).astype(np.float16)        # no negative value: zero-point 0
    X[2] = -np.linspace(0, 4, K).astype(np.float16)       # no positive value: zero-point 255
    Q, step, zx = oracle.quantize_act_asym(X)
    assert step[0] == 0 and zx[0] == 0 and np.all(Q[0] == 0)
    assert zx[1] == 0 and Q[1, 0] == 0 and Q[1, -1] == 255
    assert zx[2] == 255 and Q[2, 0] == 255 and Q[2, -1] == 0


def test_scale_folding_with_power_of_two_scales():
    M, K = 6, 384
    X = rand_x(M, K, 53)
    rng = np.random.default_rng(54)
    inv = (2.0 ** rng.integers(0, 5, K)).astype(np.float32)
    Xpre = (X.astype(np.float32) * inv).astype(np.float16)
    assert np.array_equal(Xpre.astype(np.float32), X.astype(np.float32) * inv)
    a = oracle.quantize_act_asym(X, inv)
    b = oracle.quantize_act_asym(Xpre, None)
    for u, v in zip(a, b):
        assert np.array_equal(u, v)
    assert not np.array_equal(oracle.quantize_act_asym(X)[0], a[0])


def test_asymmetric_beats_symmetric_on_shifted_tokens():
    """The reason the paper uses it: a token with an offset wastes half of a symmetric range."""
    X = rand_x(8, 1024, 57, shift=3.0)
    Q, step, zx = oracle.quantize_act_asym(X)
    Xq, tok = oracle.quantize_act(X)
    Xf = X.astype(np.float64)
    e_asym = np.abs(Xf - step[:, None].astype(np.float64) * (Q.astype(np.float64) - zx[:, None])).mean()
    e_sym = np.abs(Xf - tok[:, None].astype(np.float64) * Xq).mean()
    assert e_asym < 0.75 * e_sym


def layer(M, N, K, seed):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    X = rand_x(M, K, seed + 1, shift=0.5)
    bias = (rng.standard_normal(N) * 0.1).astype(np.float32)
    return W, X, bias


def test_contraction_against_python_integers():
    M, N, K = 3, 5, 128
    W, X, _ = layer(M, N, K, 61)
    codes, scales, zeros = oracle.pack_weights(W, None, 0)
    Q, step, zx = oracle.quantize_act_asym(X)
    acc = oracle.linear_asym_acc(Q, zx, codes, zeros)
    c = unpack(codes)
    for m in range(M):
        for n in range(N):
            z = int(zeros[0, n])
            tot = 0
            for k in range(K):
                code = int(c[n, k])
                t2 = 2 * (code - z) if code <= 13 else (1 if code == 14 else -1)
                tot += (int(Q[m, k]) - int(zx[m])) * t2
            assert tot == int(acc[m, n])


def test_identity_with_the_symmetric_contraction_and_row_sums():
    """sum (Q - zx) t2 = sum (Q - 128) t2 - (zx - 128) * sum t2: the shifted INT8 codes go
    through the symmetric integer contraction, the zero-point through the weights' row sums."""
    M, N, K = 7, 48, 512
    W, X, _ = layer(M, N, K, 67)
    codes, scales, zeros = oracle.pack_weights(W, None, 0)
    Q, step, zx = oracle.quantize_act_asym(X)
    acc = oracle.linear_asym_acc(Q, zx, codes, zeros)
    shifted = (Q.astype(np.int16) - 128).astype(np.int8)
    sym = oracle.linear_acc(shifted, codes, zeros, 0, wide=True)[0]
    c = unpack(codes).astype(np.int64)
    z = zeros[0].astype(np.int64)[:, None]
    t2 = np.where(c == 14, 1, np.where(c == 15, -1, 2 * (c - z)))
    rowsum = t2.sum(1)
    assert np.array_equal(acc, sym - (zx.astype(np.int64) - 128)[:, None] * rowsum[None, :])
    # numpy matmul of the dequantized integers
    assert np.array_equal(acc, (Q.astype(np.int64) - zx[:, None]) @ t2.T)
    assert np.abs(acc).max() < 2 ** 31


def test_output_against_float64_and_real_matmul():
    M, N, K = 6, 40, 512
    W, X, bias = layer(M, N, K, 71)
    codes, scales, zeros = oracle.pack_weights(W, None, 0)
    Q, step, zx = oracle.quantize_act_asym(X)
    Y, wide = oracle.linear_asym(Q, step, zx, codes, scales, zeros, bias, wide=True)
    acc = oracle.linear_asym_acc(Q, zx, codes, zeros)
    want = acc * step.astype(np.float64)[:, None] * (0.5 * scales[0].astype(np.float64))[None, :] + bias
    assert np.allclose(wide, want, rtol=1e-12, atol=0)
    got = oracle.bf16_bits_to_float(Y).astype(np.float64)
    assert np.all(np.abs(got - wide) <= np.abs(wide) * 2.0 ** -8 + 1e-30)
    # and it approximates the real layer it stands for
    real = X.astype(np.float64) @ W.astype(np.float64).T + bias
    rel = np.linalg.norm(got - real) / np.linalg.norm(real)
    assert rel < 0.2                                      # 4-bit round-to-nearest weights
    # dropping the zero-point must break it (the term is not optional)
    Y0 = oracle.linear_asym(Q, step, np.zeros_like(zx), codes, scales, zeros, bias)
    got0 = oracle.bf16_bits_to_float(Y0).astype(np.float64)
    assert np.linalg.norm(got0 - real) / np.linalg.norm(real) > 3 * rel


def test_group_wise_weights_with_asymmetric_activations():
    """Group-128 steps: per group the integer sum of (Q - zx) * level by numpy, the real-valued
    meaning "dequantize both operands, multiply", and the one-group case equal to the
    per-channel function."""
    rng = np.random.default_rng(21)
    M, N, K, group = 5, 24, 384, 128
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    X = (rng.standard_normal((M, K)) + 1.5).astype(np.float16)
    bias = (rng.standard_normal(N) * 0.1).astype(np.float32)
    codes, scales, zeros = oracle.pack_weights(W, None, group)
    Q, step, zx = oracle.quantize_act_asym(X)
    acc, Y, wide = oracle.linear_asym_group(Q, step, zx, codes, scales, zeros, bias, group)
    c = np.empty((N, K), dtype=np.int64)
    c[:, 0::2], c[:, 1::2] = codes & 15, codes >> 4
    zf = np.repeat(zeros.T.astype(np.int64), group, axis=1)
    lv = np.where(c == 14, 1, np.where(c == 15, -1, 2 * (c - zf)))
    A = Q.astype(np.int64) - zx.astype(np.int64)[:, None]
    want = np.stack([A[:, g * group:(g + 1) * group] @ lv[:, g * group:(g + 1) * group].T for g in range(K // group)])
    assert np.array_equal(acc, want)
    sf = np.repeat(scales.T.astype(np.float64), group, axis=1)
    deq_w = lv * sf / 2
    deq_x = A * step.astype(np.float64)[:, None]
    assert np.allclose(wide, deq_x @ deq_w.T + bias, rtol=1e-9, atol=1e-12)
    got = oracle.bf16_bits_to_float(Y).astype(np.float64)
    assert np.all(np.abs(got - wide) <= np.abs(wide) * 2.0 ** -8 + 1e-6)
    # one group covering all of K is the per-channel layer (same integer, one scaling order apart)
    c1, s1, z1 = oracle.pack_weights(W[:, :128], None, 128)
    Q1, st1, zx1 = oracle.quantize_act_asym(X[:, :128])
    a1, _, w1 = oracle.linear_asym_group(Q1, st1, zx1, c1, s1, z1, bias, 128)
    assert np.array_equal(a1[0], oracle.linear_asym_acc(Q1, zx1, c1, z1))
    _, w0 = oracle.linear_asym(Q1, st1, zx1, c1, s1, z1, bias, wide=True)
    assert np.allclose(w1, w0, rtol=1e-12)
