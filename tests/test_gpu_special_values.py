"""GPU parity of the dINT variants with the special value step / 2^shift (App. A.5: c / step =
0.25 and 0.125 beside the paper's 0.5) against the CPU oracle: packed codes and INT32 sums bit
for bit, BF16 outputs bit for bit with per-channel weights and within 1 BF16 ulp (+ the FP32
reordering allowance) with group-128 weights, on every kernel path."""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from paper_2311_05161_b200 import synth
from util import bf16_bits, bf16_ulp, to_dev

pytestmark = pytest.mark.gpu


def run(K, N, M, group, shift, opts_kw, seed):
    lay = synth.make_layer(K, N, M, seed, "laplace", 0.01, 20.0, True, True)
    d = {k: to_dev(v) for k, v in lay.items()}
    packed = w4a8.pack_weights(d["W"], d["s"], group, level_shift=shift)
    gcodes, gscales, gzeros = w4a8.unpack_codes(packed, N, K, group)
    codes, scales, zeros = oracle.pack_weights_fmt(lay["W"], lay["s"], group, shift)
    assert np.array_equal(gcodes.cpu().numpy(), codes)
    assert np.array_equal(gzeros.cpu().numpy(), zeros)
    assert np.array_equal(gscales.cpu().numpy().view(np.uint32), scales.view(np.uint32))
    opts = w4a8.make_opts(level_shift=shift, **opts_kw)
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    ws = w4a8.new_workspace(M, N, K, group, opts)
    Y = w4a8.linear(Xq, tok, packed, d["bias"], N, group, ws, opts)
    acc = w4a8.linear_acc_i32(Xq, packed, N, group, ws, opts)
    w4a8.check_status(ws)
    oXq, otok = oracle.quantize_act(lay["X"], lay["inv_s"])
    want_acc, want_Y, wide = oracle.linear_fmt(oXq, otok, codes, scales, zeros, lay["bias"], group, shift)
    assert np.abs(want_acc).max() < 2 ** 31
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), want_acc)
    got = bf16_bits(Y)
    if group == 0:
        bad = np.argwhere(got != want_Y)
        assert bad.size == 0, f"{len(bad)} BF16 outputs differ, first at {bad[0]}"
    else:
        mag = (np.abs(want_acc) * (scales.astype(np.float64) / 2 ** shift)[:, None, :]).sum(0)
        tol = bf16_ulp(wide) + 2.0 ** -20 * otok.astype(np.float64)[:, None] * mag
        err = np.abs(oracle.bf16_bits_to_float(got).astype(np.float64) - wide)
        assert np.all(err <= tol)
    return packed, lay, d


@pytest.mark.parametrize("shift", [2, 3])
@pytest.mark.parametrize("group", [0, 128])
def test_simple_path(shift, group):
    run(768, 768, 16, group, shift, dict(path=w4a8.PATH_SIMPLE), seed=shift)


@pytest.mark.parametrize("shift", [2, 3])
@pytest.mark.parametrize("group,tok_tile", [(0, 16), (0, 128), (0, 256), (128, 16), (128, 128)])
def test_tcgen05_paths(shift, group, tok_tile):
    run(1024, 200, tok_tile * 2 + 5, group, shift, dict(path=w4a8.PATH_TCGEN05, tok_tile=tok_tile),
        seed=10 * shift + tok_tile)


@pytest.mark.parametrize("shift", [2, 3])
@pytest.mark.parametrize("group", [0, 128])
def test_split_k_and_gemv(shift, group):
    run(1024, 384, 16, group, shift, dict(path=w4a8.PATH_TCGEN05, split_k=4), seed=50 + shift)
    run(2048, 520, 2, group, shift, dict(path=w4a8.PATH_GEMV), seed=60 + shift)
    run(1024, 640, 300, group, shift, {}, seed=70 + shift)          # automatic plan


def test_mismatched_shift_is_reported_and_depth_limit():
    K, N, M = 256, 128, 4
    lay = synth.make_layer(K, N, M, 5, "normal", 4, 50.0, True, True)
    d = {k: to_dev(v) for k, v in lay.items()}
    packed = w4a8.pack_weights(d["W"], d["s"], 0, level_shift=3)
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    ws = w4a8.new_workspace(M, N, K, 0)
    w4a8.linear(Xq, tok, packed, d["bias"], N, 0, ws)               # options say shift 1
    torch.cuda.synchronize()
    assert w4a8.poll_status(ws) == 8                                 # W4A8_ERR_BAD_BLOB
    # K * 127 * 13 * 8 must stay below 2^31
    with pytest.raises(w4a8.W4A8Error) as e:
        big = torch.zeros((8, 163840), dtype=torch.float16, device="cuda")
        w4a8.pack_weights(big, None, 0, level_shift=3)
    assert e.value.status == 2                                       # W4A8_ERR_SHAPE


@pytest.mark.parametrize("shift", [2, 3])
def test_asymmetric_activations_with_other_special_values(shift):
    K, N, M = 1024, 256, 40
    lay = synth.make_layer(K, N, M, 80 + shift, "normal", 4, 30.0, True, True)
    d = {k: to_dev(v) for k, v in lay.items()}
    packed = w4a8.pack_weights(d["W"], d["s"], 0, level_shift=shift)
    rowsum = w4a8.weight_rowsum(packed, N, K, 0)
    Xq, tok, tz = w4a8.quantize_act_asym(d["X"], d["inv_s"])
    opts = w4a8.make_opts(level_shift=shift)
    ws = w4a8.new_workspace(M, N, K, 0, opts)
    Y, acc = w4a8.linear_asym(Xq, tok, tz, packed, rowsum[0], d["bias"], N, ws, opts, want_acc=True)
    w4a8.check_status(ws)
    codes, scales, zeros = oracle.pack_weights_fmt(lay["W"], lay["s"], 0, shift)
    Q, step, zx = oracle.quantize_act_asym(lay["X"], lay["inv_s"])
    # definition: levels in units of step / 2^shift times (Q - zx), then the FP32 rescale
    c = np.empty((N, K), dtype=np.int64)
    c[:, 0::2] = codes & 15
    c[:, 1::2] = codes >> 4
    lv = np.where(c == 14, 1, np.where(c == 15, -1, (c - zeros[0].astype(np.int64)[:, None]) * 2 ** shift))
    want_acc = (Q.astype(np.int64) - zx[:, None]) @ lv.T
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), want_acc)
    h = (scales[0] * np.float32(2.0 ** -shift)).astype(np.float32)
    t = (want_acc.astype(np.float32) * step[:, None]).astype(np.float32) * h[None, :]
    t = (t + lay["bias"][None, :]).astype(np.float32)
    want = torch.from_numpy(t).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bf16_bits(Y), want)


@pytest.mark.parametrize("shift", [1, 2, 3])
@pytest.mark.parametrize("N,M", [(200, 1), (200, 3), (3080, 1), (3080, 2), (3080, 4)])
def test_weight_streaming_kernels_every_zero_point(shift, N, M):
    """Rows built so that output row n gets zero-point n mod 14: both weight-streaming kernels
    (K-sliced for N = 200, row slabs for N = 3080) expand every code under every zero-point,
    with the offset tables (step/2, step/4) and with the plain ones (step/8)."""
    K = 1280
    rng = np.random.default_rng(900 + shift + N + M)
    z = np.arange(N) % 14
    W = rng.integers(0, 14, size=(N, K)) - z[:, None]                 # integer levels -z .. 13-z
    W = W + rng.choice([0.0, 0.5, -0.5, 0.3, -0.3], size=(N, K)) * (np.abs(W) < 1)   # near zero: specials
    W[:, 0] = -z
    W[:, 1] = 13 - z
    W = (W * 2.0 ** -6).astype(np.float16)
    X = rng.standard_normal((M, K)).astype(np.float16)
    codes, scales, zeros = oracle.pack_weights_fmt(W, None, 0, shift)
    assert np.array_equal(zeros[0], z)
    assert len(np.unique(codes & 15)) == 16
    d = {"W": to_dev(W), "X": to_dev(X)}
    packed = w4a8.pack_weights(d["W"], None, 0, level_shift=shift)
    opts = w4a8.make_opts(w4a8.PATH_GEMV, level_shift=shift)
    Xq, tok = w4a8.quantize_act(d["X"], None)
    ws = w4a8.new_workspace(M, N, K, 0, opts)
    Y = w4a8.linear(Xq, tok, packed, None, N, 0, ws, opts)
    acc = w4a8.linear_acc_i32(Xq, packed, N, 0, ws, opts)
    w4a8.check_status(ws)
    oXq, otok = oracle.quantize_act(X, None)
    want_acc, want_Y, _ = oracle.linear_fmt(oXq, otok, codes, scales, zeros, None, 0, shift)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), want_acc)
    assert np.array_equal(bf16_bits(Y), want_Y)
