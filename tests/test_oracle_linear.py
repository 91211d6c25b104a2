"""Pins for the oracle's integer contraction and output rescale (Eq. 1, Eq. 6)."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle


def unpack(codes):
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


def pack(c):
    return (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)


def table2(z):
    """Eq. 6 doubled, written out independently of the oracle."""
    return [2 * (c - z) for c in range(14)] + [1, -1]


def rand_problem(M, N, K, group, seed):
    rng = np.random.default_rng(seed)
    G = K // group if group else 1
    c = rng.integers(0, 16, (N, K)).astype(np.uint8)
    zeros = rng.integers(0, 14, (G, N)).astype(np.uint8)
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    return Xq, c, zeros


def weights_int(c, zeros, group):
    """[N, K] doubled integer weights from codes, by table lookup in numpy."""
    N, K = c.shape
    glen = group or K
    T = np.array([table2(z) for z in range(14)], dtype=np.int64)      # [z][code]
    zfull = np.repeat(zeros.T.astype(np.int64), glen, axis=1)         # [N, K]
    return T[zfull, c.astype(np.int64)]


@pytest.mark.parametrize("group", [0, 128])
def test_acc_brute_force_triple_loop_tiny(group):
    M, N, K = 3, 5, 256
    Xq, c, zeros = rand_problem(M, N, K, group, 41)
    glen = group or K
    got = oracle.linear_acc(Xq, pack(c), zeros, group)
    for g in range(K // glen):
        for m in range(M):
            for n in range(N):
                t = table2(int(zeros[g, n]))
                want = sum(int(Xq[m, k]) * t[int(c[n, k])] for k in range(g * glen, (g + 1) * glen))
                assert int(got[g, m, n]) == want


@pytest.mark.parametrize("group", [0, 128])
def test_acc_against_numpy_int64_matmul(group):
    M, N, K = 37, 72, 640          # all different: a transposed operand cannot pass
    Xq, c, zeros = rand_problem(M, N, K, group, 43)
    W2 = weights_int(c, zeros, group)
    glen = group or K
    want = np.stack([Xq[:, g * glen:(g + 1) * glen].astype(np.int64)
                     @ W2[:, g * glen:(g + 1) * glen].T for g in range(K // glen)])
    got32 = oracle.linear_acc(Xq, pack(c), zeros, group)
    got64 = oracle.linear_acc(Xq, pack(c), zeros, group, wide=True)
    assert np.array_equal(got64, want)
    assert np.array_equal(got32.astype(np.int64), want)


def test_acc_algebraic_special_cases():
    M, N, K = 6, 8, 256
    rng = np.random.default_rng(45)
    Xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    zeros = rng.integers(0, 14, (1, N)).astype(np.uint8)
    rowsum = Xq.astype(np.int64).sum(1)
    # every weight at the zero-point -> 0
    c = np.repeat(zeros.T, K, axis=1).astype(np.uint8)
    assert np.all(oracle.linear_acc(Xq, pack(c), zeros) == 0)
    # every weight +s/2 -> sum of the token; -s/2 -> minus that
    c14 = np.full((N, K), 14, dtype=np.uint8)
    c15 = np.full((N, K), 15, dtype=np.uint8)
    assert np.array_equal(oracle.linear_acc(Xq, pack(c14), zeros)[0], np.repeat(rowsum[:, None], N, 1))
    assert np.array_equal(oracle.linear_acc(Xq, pack(c15), zeros)[0], -np.repeat(rowsum[:, None], N, 1))
    # one-hot tokens read out single table entries (and the nibble order)
    c = rng.integers(0, 16, (N, K)).astype(np.uint8)
    X1 = np.zeros((K, K), dtype=np.int8)
    np.fill_diagonal(X1, 1)
    acc = oracle.linear_acc(X1, pack(c), zeros)[0]            # [K, N]
    want = weights_int(c, zeros, 0).T
    assert np.array_equal(acc, want)


def test_acc_cannot_overflow_32_bits_at_the_largest_k():
    # worst case |q| = 127, |t2| = 26 over the largest K of the workloads
    K = 36864
    Xq = np.full((1, K), 127, dtype=np.int8)
    c = np.full((2, K), 13, dtype=np.uint8)
    c[1] = 0
    zeros = np.array([[0, 13]], dtype=np.uint8)
    a64 = oracle.linear_acc(Xq, pack(c), zeros, wide=True)
    a32 = oracle.linear_acc(Xq, pack(c), zeros)
    assert a64[0, 0, 0] == K * 127 * 26 and a64[0, 0, 1] == -K * 127 * 26
    assert np.array_equal(a32.astype(np.int64), a64)
    assert K * 127 * 26 < 2 ** 31


def bf16_rne(fr: Fraction) -> float:
    """Nearest-even rounding of an exact rational to 8 significant bits (normal range)."""
    if fr == 0:
        return 0.0
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = 0
    while a >= 2:
        a /= 2
        e += 1
    while a < 1:
        a *= 2
        e -= 1
    scaled = a * 128                       # 1.xxxxxxx -> integer part has 8 bits
    q, r = divmod(scaled.numerator, scaled.denominator)
    twice = 2 * r
    if twice > scaled.denominator or (twice == scaled.denominator and (q & 1)):
        q += 1
    return float(sign * Fraction(q, 128) * Fraction(2) ** e)


@pytest.mark.parametrize("use_scale", [False, True])
def test_whole_pipeline_on_an_exactly_representable_problem(use_scale):
    """Weights on a dINT grid, activations on an INT8 grid, power-of-two channel scales:
    every quantizer is lossless, so the output is W X exactly (Eq. 1 in full precision),
    computed here with Python integers and rounded to BF16 independently."""
    rng = np.random.default_rng(47)
    M, N, K = 5, 16, 256
    sw = Fraction(1, 64)
    z = rng.integers(0, 14, N)
    gen = rng.integers(0, 16, (N, K))
    gen[:, 0], gen[:, 1] = 0, 13
    gen[(z == 0)[:, None] & (gen == 15)] = 14
    gen[(z == 13)[:, None] & (gen == 14)] = 15
    q = rng.integers(-127, 128, (M, K))
    q[np.arange(M), rng.integers(0, K, M)] = 127
    w2 = [[table2(int(z[n]))[int(gen[n, k])] for k in range(K)] for n in range(N)]  # units of s/2
    if use_scale:
        e = rng.integers(0, 3, K)                   # s_k = 2^e, applied to W; 2^-e to X
    else:
        e = np.zeros(K, dtype=np.int64)
    # real tensors handed to the library: W = w_grid / s_k, X = x_grid * s_k
    Wreal = np.array([[float(Fraction(w2[n][k]) * sw / 2 / (2 ** int(e[k]))) for k in range(K)]
                      for n in range(N)])
    Xreal = np.array([[float(Fraction(int(q[m, k]), 8) * (2 ** int(e[k]))) for k in range(K)]
                      for m in range(M)])
    W = Wreal.astype(np.float16)
    X = Xreal.astype(np.float16)
    assert np.array_equal(W.astype(np.float64), Wreal) and np.array_equal(X.astype(np.float64), Xreal)
    s_in = (2.0 ** e).astype(np.float32) if use_scale else None
    inv = (2.0 ** -e.astype(np.float64)).astype(np.float32) if use_scale else None
    bias = (rng.integers(-8, 9, N) / 4.0).astype(np.float32)
    codes, scales, zeros = oracle.pack_weights(W, s_in, 0)
    Xq, tok = oracle.quantize_act(X, inv)
    assert np.array_equal(unpack(codes), gen.astype(np.uint8))
    assert np.array_equal(Xq, q.astype(np.int8)) and np.all(tok == np.float32(0.125))
    Y = oracle.bf16_bits_to_float(oracle.linear(Xq, tok, codes, scales, zeros, bias))
    for m in range(M):
        for n in range(N):
            exact = sum(int(q[m, k]) * w2[n][k] for k in range(K)) * Fraction(1, 8) * sw / 2 \
                + Fraction(float(bias[n]))
            assert float(Y[m, n]) == bf16_rne(exact), (m, n)


@pytest.mark.parametrize("group", [0, 128])
def test_output_rescale_against_float64_and_torch_bf16(group):
    M, N, K = 19, 40, 512
    rng = np.random.default_rng(49)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    X = rng.standard_normal((M, K)).astype(np.float16)
    bias = rng.standard_normal(N).astype(np.float32)
    codes, scales, zeros = oracle.pack_weights(W, None, group)
    Xq, tok = oracle.quantize_act(X)
    acc = oracle.linear_acc(Xq, codes, zeros, group, wide=True)       # [G, M, N]
    want = (acc * (0.5 * scales.astype(np.float64))[:, None, :]).sum(0) * tok.astype(np.float64)[:, None] \
        + bias.astype(np.float64)
    y64 = oracle.linear_f64(Xq, tok, codes, scales, zeros, bias, group)
    assert np.allclose(y64, want, rtol=1e-12, atol=1e-12)
    ybits = oracle.linear(Xq, tok, codes, scales, zeros, bias, group)
    y = oracle.bf16_bits_to_float(ybits).astype(np.float64)
    # within one BF16 step of the binary64 value
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-30))) - 7)
    assert np.all(np.abs(y - want) <= ulp)
    # and close to the full-precision product W X + b: the quantized layer approximates it
    ref = X.astype(np.float64) @ W.astype(np.float64).T + bias
    rel = np.linalg.norm(y - ref) / np.linalg.norm(ref)
    assert rel < 0.1
    if group == 0:
        # binary32 order (acc * tok) * (0.5 s) + bias, BF16 by torch: bit-exact
        t = (acc[0].astype(np.float32) * tok[:, None]) * (np.float32(0.5) * scales[0])[None, :] + bias[None, :]
        tb = torch.from_numpy(t.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(ybits, tb)


def test_error_split_of_eq4_sums_to_the_output_error():
    """Eq. 4: with Delta = Delta_u + Delta_r (weights that quantize to zero vs the rest), the
    output error is E[(Du X)^2] + E[(Dr X)^2] + 2 E[(Du X)(Dr X)].  Informational beside
    it: dINT4 has less underflow error than plain INT4 on the same normal weights."""
    rng = np.random.default_rng(51)
    N, K, T = 64, 512, 96
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    X = rng.standard_normal((K, T))
    codes, scales, zeros = oracle.pack_weights(W, None, 0)
    c = unpack(codes).astype(np.int64)
    s = scales[0].astype(np.float64)[:, None]
    z = zeros[0].astype(np.int64)[:, None]
    Wq = np.where(c == 14, s / 2, np.where(c == 15, -s / 2, (c - z) * s))
    Wd = W.astype(np.float64)
    delta = Wq - Wd
    under = Wq == 0
    du, dr = np.where(under, delta, 0), np.where(under, 0, delta)
    total = np.mean((Wd @ X - Wq @ X) ** 2)
    parts = np.mean((du @ X) ** 2) + np.mean((dr @ X) ** 2) + np.mean(2 * (du @ X) * (dr @ X))
    assert np.isclose(total, parts, rtol=1e-9)
    # plain INT4 (16 integer levels) on the same rows
    lo, hi = np.minimum(Wd.min(1), 0)[:, None], np.maximum(Wd.max(1), 0)[:, None]
    s4 = (hi - lo) / 15
    z4 = np.rint(-lo / s4)
    W4 = (np.clip(np.rint(Wd / s4) + z4, 0, 15) - z4) * s4
    du4 = np.where(W4 == 0, W4 - Wd, 0)
    assert np.mean((du @ X) ** 2) < np.mean((du4 @ X) ** 2)
