"""Pins of the oracle's attention value path ("W4A8V4": channel-wise 4-bit values, Appendix A.1;
the attention map is an 8-bit token-wise activation).  The pieces (row quantizer, token
quantizer, layer) are pinned elsewhere; here their composition per head: which axis is the
channel, which the reduction, and that the result is the attention output up to the two
quantization errors."""
import numpy as np

import oracle


def softmax_rows(x):
    e = np.exp(x - x.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def unpack(codes):
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


def problem(H, T, S, D, seed):
    rng = np.random.default_rng(seed)
    P = softmax_rows(rng.standard_normal((H, T, S)) * 2.0).astype(np.float16)
    V = (rng.standard_normal((S, H, D)) * (1.0 + rng.random((1, H, D)))).astype(np.float16)
    return P, V


def test_channels_are_head_dim_columns_and_the_range_runs_over_the_sequence():
    P, V = problem(2, 3, 128, 8, 0)
    codes, scales, zeros = oracle.pack_value(V)
    assert codes.shape == (16, 64) and scales.shape == (1, 16)
    v = V.astype(np.float64)
    for h in range(2):
        for d in range(8):
            col = v[:, h, d]
            lo, hi = min(0.0, col.min()), max(0.0, col.max())
            assert scales[0, h * 8 + d] == np.float32(np.float32(hi - lo) / np.float32(13))
    # dequantized values stay within half a step of V
    c = unpack(codes).astype(np.int64)
    s = scales[0].astype(np.float64)[:, None]
    z = zeros[0].astype(np.int64)[:, None]
    deq = np.where(c == 14, s / 2, np.where(c == 15, -s / 2, (c - z) * s))
    assert np.all(np.abs(deq - v.reshape(128, 16).T) <= s / 2 * (1 + 1e-5))


def test_integer_sums_by_brute_force_and_output_close_to_float_attention():
    H, T, S, D = 2, 5, 256, 8
    P, V = problem(H, T, S, D, 1)
    codes, scales, zeros = oracle.pack_value(V)
    Pq, ps = oracle.quantize_act(P.reshape(H * T, S))
    Pq, ps = Pq.reshape(H, T, S), ps.reshape(H, T)
    O = oracle.bf16_bits_to_float(oracle.attn_pv(Pq, ps, codes, scales, zeros, D)).astype(np.float64)
    c = unpack(codes).astype(np.int64)
    lv = np.where(c == 14, 1, np.where(c == 15, -1, 2 * (c - zeros[0].astype(np.int64)[:, None])))
    for h in range(H):
        for t in (0, T - 1):
            for d in (0, D - 1):
                tot = 0
                for s_ in range(S):
                    tot += int(Pq[h, t, s_]) * int(lv[h * D + d, s_])
                want = np.float32(np.float32(tot) * ps[h, t]) * np.float32(0.5 * scales[0, h * D + d])
                assert abs(O[t, h, d] - float(want)) <= abs(float(want)) * 2.0 ** -8 + 1e-30
    ref = np.einsum("hts,shd->thd", P.astype(np.float64), V.astype(np.float64))
    # error bound from the two quantizers: every value is off by at most half its channel's step,
    # every attention entry by at most half its token's step
    p64, v64 = P.astype(np.float64), V.astype(np.float64)
    step = scales[0].astype(np.float64).reshape(H, D)
    bound = (np.einsum("hts->th", p64)[:, :, None] * step[None] / 2
             + (ps.astype(np.float64).T / 2)[:, :, None] * np.abs(v64).sum(axis=0)[None]
             + 2.0 ** -7 * np.abs(ref) + 1e-6)
    assert np.all(np.abs(O - ref) <= bound)
    assert np.corrcoef(O.ravel(), ref.ravel())[0, 1] > 0.98


def test_one_hot_attention_returns_the_dequantized_values():
    H, T, S, D = 1, 4, 128, 8
    _, V = problem(H, T, S, D, 2)
    codes, scales, zeros = oracle.pack_value(V)
    pos = [0, 5, 77, 127]
    P = np.zeros((H, T, S), dtype=np.float16)
    for t, p in enumerate(pos):
        P[0, t, p] = 1.0
    Pq, ps = oracle.quantize_act(P.reshape(H * T, S))
    O = oracle.bf16_bits_to_float(oracle.attn_pv(Pq.reshape(H, T, S), ps.reshape(H, T), codes, scales, zeros, D))
    c = unpack(codes).astype(np.int64)
    s = scales[0].astype(np.float64)[:, None]
    deq = np.where(c == 14, s / 2, np.where(c == 15, -s / 2, (c - zeros[0].astype(np.int64)[:, None]) * s))
    for t, p in enumerate(pos):
        assert np.allclose(O[t, 0], deq[:, p], rtol=2.0 ** -7, atol=1e-30)
