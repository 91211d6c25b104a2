"""GPU parity of the norm-fused activation quantizer (w4a8_norm_quantize_act) against the CPU
oracle, through the C ABI: INT8 codes and token steps bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from util import Guarded, to_dev

pytestmark = pytest.mark.gpu


def run(M, K, kind, with_bias, seed, dist="normal", eps=1e-5, mutate=None):
    rng = np.random.default_rng(seed)
    from paper_2311_05161_b200 import synth
    X = synth.make_activations(M, K, seed, dist, 0.01, 20.0)
    X = (X.astype(np.float32) + np.float32(0.75)).astype(np.float16)        # a mean to remove
    if mutate is not None:
        mutate(X)
    # weight = gamma / s with a seeded per-channel scale s in [1/16, 16] (Eq. 1), bias likewise
    s = np.exp2(rng.uniform(-4, 4, K)).astype(np.float32)
    w = ((1.0 + 0.2 * rng.standard_normal(K)).astype(np.float32) / s).astype(np.float32)
    b = ((0.1 * rng.standard_normal(K)).astype(np.float32) / s).astype(np.float32) if with_bias else None
    want_q, want_t = oracle.norm_quantize_act(X, w, b, kind, eps)
    gq, gt = Guarded((M, K), torch.int8), Guarded((M,), torch.float32)
    code = w4a8.NORM_LAYER if kind == "layer" else w4a8.NORM_RMS
    Xq, tok = w4a8.norm_quantize_act(to_dev(X), to_dev(w), to_dev(b), code, eps, out=(gq.t, gt.t))
    torch.cuda.synchronize()
    gq.check("Xq")
    gt.check("tok_scale")
    got_t = tok.cpu().numpy()
    assert np.array_equal(got_t.view(np.uint32), want_t.view(np.uint32)), "token steps differ"
    bad = np.argwhere(Xq.cpu().numpy() != want_q)
    assert bad.size == 0, f"{len(bad)} codes differ, first at {bad[0]}"


@pytest.mark.parametrize("kind", ["rms", "layer"])
@pytest.mark.parametrize("with_bias", [False, True])
@pytest.mark.parametrize("M,K", [(16, 768), (37, 128), (300, 4096), (5, 16384), (70, 1152), (1, 9216)])
def test_norm_quantize_matches_oracle(M, K, kind, with_bias):
    run(M, K, kind, with_bias, seed=1000 + M + K)


@pytest.mark.parametrize("kind", ["rms", "layer"])
def test_laplace_tokens_zero_token_and_constant_token(kind):
    def mutate(X):
        X[1] = 0                 # all-zero token: step 0 without a bias
        X[2] = 3.0               # constant token: zero variance, eps alone under the root
    run(9, 2048, kind, False, seed=77, dist="laplace", mutate=mutate)
    run(9, 2048, kind, True, seed=78, dist="laplace", mutate=mutate, eps=1e-6)


def test_more_tokens_than_resident_ctas():
    run(2048, 4096, "rms", False, seed=5)
    run(1500, 1024, "layer", True, seed=6)


def test_validation():
    lib = w4a8.lib
    import ctypes
    p = ctypes.c_void_p
    good = 0x10000
    assert lib.w4a8_norm_quantize_act(p(good), None, None, 0, 1e-5, 4, 256, p(good), p(good), None) == 1
    assert lib.w4a8_norm_quantize_act(p(good), p(good), None, 2, 1e-5, 4, 256, p(good), p(good), None) == 2
    assert lib.w4a8_norm_quantize_act(p(good), p(good), None, 0, 0.0, 4, 256, p(good), p(good), None) == 2
    assert lib.w4a8_norm_quantize_act(p(good), p(good), None, 0, 1e-5, 4, 16512, p(good), p(good), None) == 2
    assert lib.w4a8_norm_quantize_act(p(good), p(good + 4), None, 0, 1e-5, 4, 256, p(good), p(good), None) == 3
