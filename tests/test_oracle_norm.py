"""Pins of the oracle's norm-fused activation quantizer (Fig. 1(a), Section 3.1: the Eq. 1
scale lives in the normalisation in front of the matmul; Appendix A.1: token-wise INT8).

Pinned against things other than the oracle itself: torch's layer_norm / rms_norm in float64,
closed forms on inputs whose statistics are exact, invariances of the normalisations, and the
plain quantizer of the already pinned oracle_quantize_act on inputs where the normalisation is
a multiplication by a power of two."""
import numpy as np
import pytest
import torch

import oracle


def rand_x(M, K, seed, scale=1.0, shift=0.0):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((M, K)) * scale + shift).astype(np.float16)


def dequant(Xq, tok):
    return Xq.astype(np.float64) * tok.astype(np.float64)[:, None]


@pytest.mark.parametrize("kind", ["rms", "layer"])
@pytest.mark.parametrize("with_bias", [False, True])
def test_matches_torch_float64_normalisation_within_half_a_step(kind, with_bias):
    M, K, eps = 7, 640, 1e-5
    X = rand_x(M, K, 1, scale=3.0, shift=0.5)
    rng = np.random.default_rng(2)
    w = (1.0 + 0.3 * rng.standard_normal(K)).astype(np.float32)
    b = (0.2 * rng.standard_normal(K)).astype(np.float32) if with_bias else None
    x64 = torch.from_numpy(X.astype(np.float64))
    if kind == "layer":
        ref = torch.nn.functional.layer_norm(x64, (K,), torch.from_numpy(w.astype(np.float64)),
                                             torch.from_numpy(b.astype(np.float64)) if with_bias else None, eps)
    else:
        ref = torch.nn.functional.rms_norm(x64, (K,), torch.from_numpy(w.astype(np.float64)), eps)
        if with_bias:
            ref = ref + torch.from_numpy(b.astype(np.float64))
    ref = ref.numpy()
    Xq, tok = oracle.norm_quantize_act(X, w, b, kind, eps)
    # the step is absmax / 127 of the normalised token, the codes are its rounding
    amax = np.abs(ref).max(axis=1)
    assert np.allclose(tok, amax / 127.0, rtol=1e-5)
    assert np.all(np.abs(dequant(Xq, tok) - ref) <= 0.5 * tok[:, None] * (1 + 1e-4) + 1e-6 * amax[:, None])
    assert np.all(np.abs(Xq).max(axis=1) == 127)


def test_rms_closed_form_on_an_exact_grid():
    # |x| = 2 everywhere: mean square 4, eps far below one ulp of it, so r = 1/2 exactly;
    # weights are integers with one 127 per token: the codes are sign(x) * w
    K = 256
    rng = np.random.default_rng(3)
    sign = rng.choice([-1.0, 1.0], size=(5, K))
    X = (2.0 * sign).astype(np.float16)
    w = rng.integers(-126, 127, size=K).astype(np.float32)
    w[17] = 127.0
    Xq, tok = oracle.norm_quantize_act(X, w, None, "rms", 1e-30)
    assert np.array_equal(Xq, (sign * w[None, :]).astype(np.int8))
    assert np.array_equal(tok, np.ones(5, dtype=np.float32))


def test_layer_closed_form_on_an_exact_grid():
    # x = 10 +- 4 in equal numbers: mean 10, variance 16, r = 1/4 exactly; bias shifts by integers
    K = 512
    rng = np.random.default_rng(4)
    sign = np.where(np.arange(K) % 2 == 0, 1.0, -1.0)
    X = np.stack([10.0 + 4.0 * np.roll(sign, i) for i in range(4)]).astype(np.float16)
    w = rng.integers(-60, 61, size=K).astype(np.float32)
    b = rng.integers(-60, 61, size=K).astype(np.float32)
    w[0], b[0], w[2], b[2] = 67.0, 60.0, -67.0, 60.0        # some |+-w + b| = 127 whichever the sign
    Xq, tok = oracle.norm_quantize_act(X, w, b, "layer", 1e-30)
    want = np.stack([np.roll(sign, i) * w + b for i in range(4)])
    assert np.all(np.abs(want).max(axis=1) == 127)
    assert np.array_equal(Xq, want.astype(np.int8))
    assert np.array_equal(tok, np.ones(4, dtype=np.float32))


def test_layer_norm_ignores_a_common_offset_and_rms_norm_does_not():
    K = 384
    base = (np.random.default_rng(5).integers(-64, 65, size=(3, K)) / 8.0)
    X0 = base.astype(np.float16)
    X1 = (base + 32.0).astype(np.float16)                 # still exact in binary16
    w = np.ones(K, dtype=np.float32)
    a = oracle.norm_quantize_act(X0, w, None, "layer", 1e-5)
    b = oracle.norm_quantize_act(X1, w, None, "layer", 1e-5)
    # (the mean is rounded to binary32 once, so the invariance holds to rounding, not to the bit)
    assert np.abs(a[0].astype(int) - b[0].astype(int)).max() <= 1
    assert np.mean(a[0] != b[0]) < 0.01 and np.allclose(a[1], b[1], rtol=1e-5)
    c = oracle.norm_quantize_act(X1, w, None, "rms", 1e-5)
    assert not np.array_equal(a[0], c[0])


def test_a_power_of_two_normalisation_reduces_to_the_plain_quantizer():
    # every token has mean square 2^-4 (entries +-1/4): r = 4, an exact scaling, so the result
    # is the plain token-wise quantizer applied to 4 x with the weight as the Eq. 1 factor
    K = 256
    rng = np.random.default_rng(6)
    X = (0.25 * rng.choice([-1.0, 1.0], size=(6, K))).astype(np.float16)
    w = (1.0 + 0.5 * rng.random(K)).astype(np.float32)
    Xq, tok = oracle.norm_quantize_act(X, w, None, "rms", 1e-30)
    Xq2, tok2 = oracle.quantize_act((4.0 * X.astype(np.float32)).astype(np.float16), w)
    assert np.array_equal(Xq, Xq2) and np.array_equal(tok, tok2)


def test_zero_token_and_eps():
    K = 128
    X = np.zeros((2, K), dtype=np.float16)
    X[1, 3] = 1.0
    w = np.ones(K, dtype=np.float32)
    Xq, tok = oracle.norm_quantize_act(X, w, None, "rms", 1e-5)
    assert tok[0] == 0.0 and not Xq[0].any()                 # 0 / sqrt(eps) is still 0
    assert Xq[1, 3] == 127 and np.count_nonzero(Xq[1]) == 1
    # with a bias the all-zero token quantizes the bias alone
    b = np.linspace(-1, 1, K).astype(np.float32)
    Xq, tok = oracle.norm_quantize_act(X[:1], w, b, "layer", 1e-5)
    want, wtok = oracle.quantize_act(np.ones((1, K), dtype=np.float16), b)
    assert np.array_equal(Xq, want) and np.array_equal(tok, wtok)
    # eps matters when the variance is small: a larger eps shrinks the normalised values
    Xs = (1e-3 * np.random.default_rng(7).standard_normal((1, K))).astype(np.float16)
    t_small = oracle.norm_quantize_act(Xs, w, None, "rms", 1e-12)[1]
    t_big = oracle.norm_quantize_act(Xs, w, None, "rms", 1e-2)[1]
    assert t_big[0] < 0.05 * t_small[0]
