"""GPU parity, bit-exact: weight packing (Eq. 1 weight side, Eq. 5) and the token-wise
activation quantizer (Eq. 1 activation side) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from paper_2311_05161_b200 import synth
from util import to_dev

pytestmark = pytest.mark.gpu


def pack_and_compare(W, s_in, group, clip=1.0):
    N, K = W.shape
    packed = w4a8.pack_weights(to_dev(W), to_dev(s_in), group, clip)
    codes, scales, zeros = w4a8.unpack_codes(packed, N, K, group)
    torch.cuda.synchronize()
    ocodes, oscales, ozeros = oracle.pack_weights(W, s_in, group, clip)
    assert np.array_equal(zeros.cpu().numpy(), ozeros)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), oscales.view(np.uint32))
    assert np.array_equal(codes.cpu().numpy(), ocodes)
    return packed


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("N,K", [(768, 768), (200, 256), (8, 128), (384, 4096), (136, 11008)])
def test_pack_matches_oracle(N, K, group):
    lay = synth.make_layer(K, N, 64, seed=N + K + group, outliers=0.01, mult=20.0)
    pack_and_compare(lay["W"], lay["s"], group)
    pack_and_compare(lay["W"], None, group)


@pytest.mark.parametrize("group", [0, 128])
def test_pack_edge_rows_and_clip(group):
    rng = np.random.default_rng(5)
    N, K = 64, 512
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    W[0] = 0                                   # all-zero row: step 1, zero-point 0
    W[1] = np.abs(W[1])                        # one-sided rows
    W[2] = -np.abs(W[2])
    W[3, :128] = 0                             # an all-zero group
    W[4] = np.float16(6e-8)                    # binary16 subnormals
    W[5, ::2] = 60000.0                        # near the binary16 maximum
    s_in = (2.0 ** rng.integers(-4, 5, K)).astype(np.float32)
    pack_and_compare(W, None, group)
    pack_and_compare(W, s_in, group)
    pack_and_compare(W, s_in, group, clip=0.75)


def test_pack_exact_grid_and_header_blob_reuse():
    rng = np.random.default_rng(17)
    N, K = 128, 256
    z = rng.integers(0, 14, N)
    gen = rng.integers(0, 16, (N, K))
    gen[:, 0], gen[:, 1] = 0, 13
    gen[(z == 0)[:, None] & (gen == 15)] = 14
    gen[(z == 13)[:, None] & (gen == 14)] = 15
    W = (np.where(gen == 14, 0.5, np.where(gen == 15, -0.5, gen - z[:, None])) * 2.0 ** -6).astype(np.float16)
    packed = pack_and_compare(W, None, 0)
    codes, _, zeros = w4a8.unpack_codes(packed, N, K, 0)
    c = codes.cpu().numpy()
    got = np.empty((N, K), dtype=np.uint8)
    got[:, 0::2], got[:, 1::2] = c & 15, c >> 4
    assert np.array_equal(got, gen.astype(np.uint8))
    assert np.array_equal(zeros.cpu().numpy()[0], z.astype(np.uint8))
    # the blob is position independent: a byte copy unpacks to the same codes
    copy = packed.clone()
    c2, _, _ = w4a8.unpack_codes(copy, N, K, 0)
    assert torch.equal(c2, codes)


@pytest.mark.parametrize("M,K", [(16, 768), (1, 128), (33, 4096), (7, 11008), (5, 16384),
                                 (3, 22016), (2, 36864)])
@pytest.mark.parametrize("scaled", [False, True])
def test_quantize_act_matches_oracle(M, K, scaled):
    lay = synth.make_layer(K, 8, M, seed=M * 31 + K, dist="laplace", outliers=0.01, mult=20.0,
                           scaled=scaled)
    Xq, tok = w4a8.quantize_act(to_dev(lay["X"]), to_dev(lay["inv_s"]))
    torch.cuda.synchronize()
    oXq, otok = oracle.quantize_act(lay["X"], lay["inv_s"])
    assert np.array_equal(tok.cpu().numpy().view(np.uint32), otok.view(np.uint32))
    assert np.array_equal(Xq.cpu().numpy(), oXq)


def test_quantize_act_zero_token_ties_and_extremes():
    K = 256
    X = np.zeros((5, K), dtype=np.float16)
    X[1, 5], X[1, 6], X[1, 7], X[1, 8], X[1, 9] = 127.0, 0.5, 1.5, 2.5, -3.5
    X[2, 0] = -1.0
    X[3, :] = 6e-8                              # subnormal token
    X[4, 3], X[4, 4] = 65504.0, -65504.0
    Xq, tok = w4a8.quantize_act(to_dev(X))
    oXq, otok = oracle.quantize_act(X)
    assert np.array_equal(Xq.cpu().numpy(), oXq)
    assert np.array_equal(tok.cpu().numpy().view(np.uint32), otok.view(np.uint32))
    assert list(oXq[1, 5:10]) == [127, 0, 2, 2, -4] and otok[0] == 0.0


def test_config1_quantizers():
    lay = synth.workload_layer(1, 0, 16)
    pack_and_compare(lay["W"], lay["s"], 0)
    Xq, tok = w4a8.quantize_act(to_dev(lay["X"]), to_dev(lay["inv_s"]))
    oXq, otok = oracle.quantize_act(lay["X"], lay["inv_s"])
    assert np.array_equal(Xq.cpu().numpy(), oXq)
    assert np.array_equal(tok.cpu().numpy(), otok)
