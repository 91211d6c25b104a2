"""GPU parity of w4a8_linear_swiglu against the oracle through the C ABI: the binary16 output
within one binary16 step of the binary64 evaluation of silu(g) * u on the layer's FP32 values
(the kernel's exponential is the fast one; group-128 weights add their FP32 reordering
allowance), and equal to the unfused route (two w4a8_linear calls) up to BF16 rounding."""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from paper_2311_05161_b200 import synth
from util import Guarded, guarded_workspace, to_dev

pytestmark = pytest.mark.gpu


def half_ulp_of(x64):
    """Spacing of binary16 numbers at |x| (11 significant bits; subnormal step 2^-24)."""
    e = np.floor(np.log2(np.maximum(np.abs(x64), 2.0 ** -14)))
    return 2.0 ** (e - 10)


def run(M, F, K, group, seed, with_bias=True):
    rng = np.random.default_rng(seed)
    Wg = synth.make_weights(F, K, seed)
    Wu = synth.make_weights(F, K, seed + 1)
    W = np.ascontiguousarray(np.stack((Wg, Wu), axis=1).reshape(2 * F, K))
    X = synth.make_activations(M, K, seed, "laplace", 0.01, 20.0)
    s, inv = synth.make_channel_scales(X, W)
    bias = (rng.standard_normal(2 * F) * 0.2).astype(np.float32) if with_bias else None
    codes, scales, zeros = oracle.pack_weights(W, s, group)
    oXq, otok = oracle.quantize_act(X, inv)
    H64, T = oracle.linear_swiglu(oXq, otok, codes, scales, zeros, bias, group)
    Wd = w4a8.interleave_gate_up(to_dev(Wg), to_dev(Wu))
    assert np.array_equal(Wd.cpu().numpy().view(np.uint16), W.view(np.uint16))
    packed = w4a8.pack_weights(Wd, to_dev(s), group)
    Xq, tok = w4a8.quantize_act(to_dev(X), to_dev(inv))
    gH = Guarded((M, F), torch.float16)
    gws = guarded_workspace(int(w4a8.lib.w4a8_linear_swiglu_workspace_bytes(M, F, K, group)))
    for _ in range(2):
        Hd = w4a8.linear_swiglu(Xq, tok, packed, to_dev(bias), F, group, gws.t, out=gH.t)
        w4a8.check_status(gws.t)
        gH.check("H")
        gws.check("workspace")
        got = Hd.cpu().numpy().astype(np.float64)
        tol = half_ulp_of(H64) * 1.0 + 1e-30
        if group:
            # the FP32 group sums may be added in another order: allow that on g and u
            # (|dh| <= |dg| * |u| * 1.1 + |du| * |silu(g)|)
            g64, u64 = T[:, 0::2].astype(np.float64), T[:, 1::2].astype(np.float64)
            slack = 2.0 ** -19 * (np.abs(g64) * np.abs(u64) * 2.2 + np.abs(u64) * 1e-3)
            tol = tol + slack + 2.0 ** -18 * np.abs(u64)
        bad = np.argwhere(np.abs(got - H64) > tol)
        assert bad.size == 0, f"{len(bad)} outputs beyond one binary16 step, first at {bad[0]}: {got[tuple(bad[0])]} vs {H64[tuple(bad[0])]}"
    # the unfused route: two plain layers, the unit on their BF16 outputs
    ws = w4a8.new_workspace(M, 2 * F, K, group)
    Y = w4a8.linear(Xq, tok, packed, to_dev(bias), 2 * F, group, ws).float().cpu().numpy().astype(np.float64)
    ref = Y[:, 0::2] / (1 + np.exp(-Y[:, 0::2])) * Y[:, 1::2]
    assert np.all(np.abs(got - ref) <= 2.0 ** -6 * (np.abs(ref) + np.abs(Y[:, 1::2])) + 1e-3)


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("M,F,K", [(16, 384, 768), (37, 104, 1024), (300, 1376, 512), (1, 2752, 1024), (520, 64, 256)])
def test_linear_swiglu_matches_oracle(M, F, K, group):
    run(M, F, K, group, seed=7000 + M + F + K + group)


def test_without_bias_and_many_tiles_per_cta():
    run(130, 64 * 170, 256, 0, seed=12, with_bias=False)


def test_validation():
    assert w4a8.lib.w4a8_linear_swiglu_workspace_bytes(16, 12, 256, 0) == 0         # F % 8
    assert w4a8.lib.w4a8_linear_swiglu_workspace_bytes(16, 64, 200, 0) == 0         # K % 128
    assert w4a8.lib.w4a8_linear_swiglu_workspace_bytes(16, 64, 256, 0) >= 256
