"""Pins of the oracle's gated-unit layer (gate and up projections, h = silu(g) * u): the FP32
values it starts from are those of the pinned oracle_linear, the unit is torch's silu in
float64, and the row pairing is checked on a hand-made case."""
import numpy as np
import torch

import oracle


def problem(M, F, K, group, seed):
    rng = np.random.default_rng(seed)
    Wg = (rng.standard_normal((F, K)) * 0.05).astype(np.float16)
    Wu = (rng.standard_normal((F, K)) * 0.05).astype(np.float16)
    W = np.stack((Wg, Wu), axis=1).reshape(2 * F, K)
    X = rng.standard_normal((M, K)).astype(np.float16)
    bias = (rng.standard_normal(2 * F) * 0.1).astype(np.float32)
    return Wg, Wu, np.ascontiguousarray(W), X, bias


def test_fp32_values_are_those_of_the_plain_layer_and_unit_is_silu_times_up():
    for group in (0, 128):
        Wg, Wu, W, X, bias = problem(6, 20, 256, group, 1)
        codes, scales, zeros = oracle.pack_weights(W, None, group)
        Xq, tok = oracle.quantize_act(X)
        H, T = oracle.linear_swiglu(Xq, tok, codes, scales, zeros, bias, group)
        # T rounds to the BF16 output of the plain layer
        Y = oracle.linear(Xq, tok, codes, scales, zeros, bias, group)
        assert np.array_equal(torch.from_numpy(T).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16), Y)
        g = torch.from_numpy(T[:, 0::2].astype(np.float64))
        u = torch.from_numpy(T[:, 1::2].astype(np.float64))
        want = (torch.nn.functional.silu(g) * u).numpy()
        assert np.allclose(H, want, rtol=1e-14, atol=0)
        # and the rows pair up as gate / up of the same feature: packing the two projections
        # separately gives the same g and u
        cg, sg, zg = oracle.pack_weights(Wg, None, group)
        cu, su, zu = oracle.pack_weights(Wu, None, group)
        Tg = np.empty((6, 20), np.float32)
        Yg = oracle.linear_f64(Xq, tok, cg, sg, zg, bias[0::2], group)
        Yu = oracle.linear_f64(Xq, tok, cu, su, zu, bias[1::2], group)
        assert np.allclose(T[:, 0::2], Yg, rtol=1e-5, atol=1e-6) and np.allclose(T[:, 1::2], Yu, rtol=1e-5, atol=1e-6)


def test_limits_of_the_unit():
    # weights on an exact grid so that g is exactly 0, large positive, large negative
    K, F = 128, 2
    W = np.zeros((2 * F, K), dtype=np.float16)
    W[0, 0], W[0, 1] = 13.0, 0.0          # gate 0: x0 * 13
    W[1, 0], W[1, 1] = 0.0, 13.0          # up 0:   x1 * 13
    W[2, 0], W[2, 1] = -13.0, 0.0         # gate 1: -x0 * 13
    W[3, 0], W[3, 1] = 0.0, 13.0
    X = np.zeros((2, K), dtype=np.float16)
    X[0, 0], X[0, 1] = 127.0, 1.0          # g = 1651 (unit passes it), u = 13
    X[1, 0], X[1, 1] = 0.0, 127.0          # g = 0 -> h = 0 whatever u
    codes, scales, zeros = oracle.pack_weights(W, None, 0)
    Xq, tok = oracle.quantize_act(X)
    H, T = oracle.linear_swiglu(Xq, tok, codes, scales, zeros, None, 0)
    assert T[0, 0] == 1651.0 and T[0, 1] == 13.0 and T[0, 2] == -1651.0
    assert H[0, 0] == 1651.0 * 13.0            # silu(g) = g for large g
    assert H[0, 1] == 0.0 or abs(H[0, 1]) < 1e-300   # silu(-1651) = -0
    assert H[1, 0] == 0.0 and H[1, 1] == 0.0
