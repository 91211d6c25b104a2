"""Pins for the oracle's weight and activation quantizers (Eq. 1, Eq. 5, App. A.1)."""
import numpy as np
import pytest

import oracle


def unpack(codes):
    """[N, K/2] bytes -> [N, K] codes (low nibble first)."""
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


def rand_w(N, K, seed, std=0.02):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((N, K)) * std).astype(np.float16)


# ---------------------------------------------------------------------------
# weights
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("group", [0, 128])
def test_pack_reduces_to_textbook_minmax_when_no_value_is_near_zero(group):
    """With no element inside the two special bands, Eq. 5 is plain asymmetric Min-Max
    integer quantization with 14 levels; that is recomputed here in float64 numpy."""
    N, K = 48, 512
    W = rand_w(N, K, 3).astype(np.float32)
    glen = group or K
    Wg = W.reshape(N, K // glen, glen)
    lo = np.minimum(Wg.min(-1), 0)
    hi = np.maximum(Wg.max(-1), 0)
    s = (hi - lo) / 13
    band = (np.abs(Wg) > 0.24 * s[..., None]) & (np.abs(Wg) < 0.76 * s[..., None])
    Wg = np.where(band, 0, Wg)
    W = Wg.reshape(N, K).astype(np.float16)
    # textbook quantizer, float64
    Wd = W.astype(np.float64).reshape(N, K // glen, glen)
    lo = np.minimum(Wd.min(-1), 0)
    hi = np.maximum(Wd.max(-1), 0)
    s32 = ((hi - lo).astype(np.float32) / np.float32(13)).astype(np.float32)
    z = np.clip(np.rint(-lo / s32), 0, 13)
    ratio = Wd / s32[..., None].astype(np.float64)
    want = np.clip(np.rint(ratio) + z[..., None], 0, 13).reshape(N, K)
    # positions whose ratio is closer to a tie than binary32 can resolve are not compared
    frac = np.abs(ratio - np.floor(ratio) - 0.5).reshape(N, K)
    safe = frac > 1e-5
    codes, scales, zeros = oracle.pack_weights(W, None, group)
    got = unpack(codes)
    assert safe.mean() > 0.999
    assert np.array_equal(got[safe], want[safe].astype(np.uint8))
    assert np.array_equal(zeros.T.astype(np.float64), z)
    assert np.array_equal(scales.T, s32)
    assert got.max() <= 13


def test_pack_codes_dequantize_close_to_the_weights():
    """|w - DQ(Q(w))| <= s/2 for every weight (s/4 near zero): catches a wrong zero-point,
    a wrong nibble order or a transposed scale array."""
    N, K = 40, 384
    W = rand_w(N, K, 5)
    for group in (0, 128):
        codes, scales, zeros = oracle.pack_weights(W, None, group)
        c = unpack(codes).astype(np.int64)
        glen = group or K
        s = np.repeat(scales.T, glen, axis=1).astype(np.float64)
        z = np.repeat(zeros.T, glen, axis=1).astype(np.int64)
        deq = np.where(c == 14, s / 2, np.where(c == 15, -s / 2, (c - z) * s))
        err = np.abs(W.astype(np.float64) - deq)
        assert np.all(err <= s / 2 * (1 + 1e-5))
        small = np.abs(W.astype(np.float64)) <= s
        assert np.all(err[small] <= (s / 4 * (1 + 1e-5))[small])
        # both specials and both range ends occur in every row
        assert np.all((c == 14).any(1)) and np.all((c == 15).any(1))
        assert np.all((c == 0).any(1)) and np.all((c == 13).any(1))


def test_pack_min_and_max_map_to_the_range_ends():
    N, K = 16, 256
    W = rand_w(N, K, 7)
    codes, scales, zeros = oracle.pack_weights(W, None, 0)
    c = unpack(codes)
    for n in range(N):
        assert c[n, np.argmax(W[n])] == 13
        assert c[n, np.argmin(W[n])] == 0


def test_pack_all_zero_row_and_one_sided_rows():
    K = 128
    W = np.zeros((3, K), dtype=np.float16)
    W[1, :] = np.linspace(0, 1, K).astype(np.float16)       # non-negative row: lo = 0 -> z = 0
    W[2, :] = -np.linspace(0, 1, K).astype(np.float16)      # non-positive row: hi = 0 -> z = 13
    codes, scales, zeros = oracle.pack_weights(W, None, 0)
    c = unpack(codes)
    assert scales[0, 0] == 1.0 and zeros[0, 0] == 0 and np.all(c[0] == 0)
    assert zeros[0, 1] == 0 and scales[0, 1] == np.float32(1.0) / np.float32(13)
    assert zeros[0, 2] == 13 and c[2, -1] == 0 and c[1, -1] == 13


def test_pack_scale_folding_with_power_of_two_scales():
    """Eq. 1 weight side: quantizing W diag(s) with s given equals quantizing the
    pre-multiplied matrix, exactly, when s is a power of two."""
    N, K = 24, 256
    W = rand_w(N, K, 11)
    rng = np.random.default_rng(12)
    s_in = (2.0 ** rng.integers(0, 5, K)).astype(np.float32)   # scaling up stays exact in binary16
    Wpre = (W.astype(np.float32) * s_in).astype(np.float16)
    assert np.array_equal(Wpre.astype(np.float32), W.astype(np.float32) * s_in)
    for group in (0, 128):
        a = oracle.pack_weights(W, s_in, group)
        b = oracle.pack_weights(Wpre, None, group)
        for u, v in zip(a, b):
            assert np.array_equal(u, v)
    # and it is not a no-op
    assert not np.array_equal(oracle.pack_weights(W, None, 0)[0], a[0])


def test_pack_clip_ratio_shrinks_the_range():
    W = rand_w(8, 256, 13)
    _, s1, _ = oracle.pack_weights(W, None, 0, 1.0)
    codes, s2, _ = oracle.pack_weights(W, None, 0, 0.5)
    assert np.allclose(s2, s1 * 0.5, rtol=1e-6)
    c = unpack(codes)
    assert c.max() <= 15 and (c == 13).sum() > 8      # clipped values pile up at the ends


def test_exact_grid_weights_are_recovered():
    """Weights placed on a dINT grid (s = 2^-6, every row holding codes 0 and 13) must
    come back as the generating codes with the generating step size and zero-point."""
    rng = np.random.default_rng(17)
    N, K = 32, 256
    s = 2.0 ** -6
    z = rng.integers(0, 14, N)
    gen = rng.integers(0, 16, (N, K))
    gen[:, 0], gen[:, 1] = 0, 13
    # a row whose range ends at zero cannot hold the special value beyond that end
    gen[(z == 0)[:, None] & (gen == 15)] = 14
    gen[(z == 13)[:, None] & (gen == 14)] = 15
    val = np.where(gen == 14, 0.5, np.where(gen == 15, -0.5, gen - z[:, None])) * s
    W = val.astype(np.float16)
    assert np.array_equal(W.astype(np.float64), val)
    codes, scales, zeros = oracle.pack_weights(W, None, 0)
    assert np.array_equal(unpack(codes), gen.astype(np.uint8))
    assert np.all(scales == np.float32(s)) and np.array_equal(zeros[0], z.astype(np.uint8))


# ---------------------------------------------------------------------------
# activations
# ---------------------------------------------------------------------------

def rand_x(M, K, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K)).astype(np.float32)
    x[:, :3] *= 40
    return x.astype(np.float16)


def test_act_quant_closed_forms():
    M, K = 12, 640
    X = rand_x(M, K, 21)
    Xq, tok = oracle.quantize_act(X)
    Xf = X.astype(np.float64)
    amax = np.abs(Xf).max(1)
    # the largest element of a token maps to +-127 and fixes the step size
    idx = np.abs(Xf).argmax(1)
    assert np.array_equal(np.abs(Xq[np.arange(M), idx].astype(int)), np.full(M, 127))
    assert np.array_equal(np.sign(Xq[np.arange(M), idx]), np.sign(Xf[np.arange(M), idx]))
    assert np.array_equal(tok, (amax.astype(np.float32) / np.float32(127)))
    # nearest: within half a step of the real ratio, with binary32 slack
    ratio = Xf * (127.0 / amax)[:, None]
    assert np.all(np.abs(Xq - ratio) <= 0.5 + 1e-4)
    assert np.abs(Xq.astype(int)).max() == 127
    # sign symmetry
    Xn, tokn = oracle.quantize_act((-X).astype(np.float16))
    assert np.array_equal(Xn, -Xq) and np.array_equal(tokn, tok)
    # monotone per token
    for m in range(M):
        order = np.argsort(Xf[m], kind="stable")
        assert np.all(np.diff(Xq[m, order].astype(int)) >= 0)


def test_act_quant_exact_integer_grid_and_idempotence():
    rng = np.random.default_rng(23)
    M, K = 9, 256
    q = rng.integers(-127, 128, (M, K))
    q[np.arange(M), rng.integers(0, K, M)] = 127 * rng.choice([-1, 1], M)
    X = (q * 2.0 ** -3).astype(np.float16)
    assert np.array_equal(X.astype(np.float64), q * 2.0 ** -3)
    Xq, tok = oracle.quantize_act(X)
    assert np.array_equal(Xq, q.astype(np.int8))
    assert np.all(tok == np.float32(2.0 ** -3))
    # idempotence on a general tensor: requantizing q * step returns q
    X2 = rand_x(M, K, 24)
    q2, t2 = oracle.quantize_act(X2)
    back = (q2.astype(np.float32) * t2[:, None])
    # q * step is not a binary16 value in general; feed the nearest binary16 of a
    # power-of-two-step case instead
    assert np.abs(back - X2.astype(np.float32)).max() <= t2.max() * 0.5 * (1 + 1e-5)


def test_act_quant_zero_token_and_ties():
    X = np.zeros((3, 128), dtype=np.float16)
    X[1, 5] = 127.0
    X[1, 6] = 0.5      # tie -> 0 (even)
    X[1, 7] = 1.5      # tie -> 2
    X[1, 8] = 2.5      # tie -> 2
    X[1, 9] = -3.5     # tie -> -4
    X[2, 0] = -1.0
    Xq, tok = oracle.quantize_act(X)
    assert np.all(Xq[0] == 0) and tok[0] == 0.0
    assert list(Xq[1, 5:10]) == [127, 0, 2, 2, -4] and tok[1] == 1.0
    assert Xq[2, 0] == -127 and np.all(Xq[2, 1:] == 0)


def test_act_quant_scale_folding_with_power_of_two_scales():
    """Eq. 1 activation side: multiplying by 1/s inside the quantizer equals quantizing
    the pre-divided tensor, exactly, for power-of-two s."""
    M, K = 10, 384
    X = rand_x(M, K, 29)
    rng = np.random.default_rng(30)
    inv = (2.0 ** rng.integers(0, 5, K)).astype(np.float32)   # scaling up stays exact in binary16
    Xpre = (X.astype(np.float32) * inv).astype(np.float16)
    assert np.array_equal(Xpre.astype(np.float32), X.astype(np.float32) * inv)
    a = oracle.quantize_act(X, inv)
    b = oracle.quantize_act(Xpre, None)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert not np.array_equal(oracle.quantize_act(X)[0], a[0])
