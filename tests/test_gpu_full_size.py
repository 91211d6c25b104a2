"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration
the bench uses (automatic plan), on sampled outputs.

The CPU oracle is far too slow for a whole 2048 x 36864 x 9216 layer, but every output element
depends only on its own token (activation quantizer is per token) and its own weight row (weight
quantizer is per output row), so a seeded sample of tokens x rows can be recomputed exactly:
the oracle packs only the sampled rows and quantizes only the sampled tokens.  Sampled sets always
include the first and last token and row, and rows on both sides of a 128-row tile edge.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from paper_2311_05161_b200 import synth
from util import bf16_bits, bf16_ulp, to_dev

pytestmark = pytest.mark.gpu

N_ROWS, N_TOKENS = 96, 48


def sample(total, count, seed, edges):
    rng = np.random.Generator(np.random.PCG64([seed, 99]))
    picked = set(int(v) for v in edges if 0 <= v < total)
    picked.update(int(v) for v in rng.choice(total, size=min(count, total), replace=False))
    return np.array(sorted(picked))


def check_shape(config, shape_index, tokens, acc_for_M=None):
    wl = synth.WORKLOADS[config]
    K, N, label = wl.shapes[shape_index]
    seed = wl.seed(shape_index)
    group = wl.group
    W = synth.make_weights(N, K, seed)
    rows = sample(N, N_ROWS, seed, [0, 1, 127, 128, 129, N - 129, N - 128, N - 1])
    Wd = to_dev(W)
    packed = None
    for M in tokens:
        X = synth.make_activations(M, K, seed, wl.act_dist, wl.outlier_channels, wl.outlier_mult)
        s, inv = synth.make_channel_scales(X, W)
        bias = synth.make_bias(N, seed)
        Xd, sd, invd, biasd = to_dev(X), to_dev(s), to_dev(inv), to_dev(bias)
        # the channel scale depends on the activations, so the weights are packed per M
        packed = w4a8.pack_weights(Wd, sd, group, out=packed)
        Xq, tok = w4a8.quantize_act(Xd, invd)
        ws = w4a8.new_workspace(M, N, K, group)
        Y = w4a8.linear(Xq, tok, packed, biasd, N, group, ws)
        w4a8.check_status(ws)
        toks = sample(M, N_TOKENS, seed + M, [0, 1, 15, 16, 127, 128, 255, 256, M - 2, M - 1])
        # oracle on the sample
        ocodes, oscales, ozeros = oracle.pack_weights(np.ascontiguousarray(W[rows]), s, group)
        oXq, otok = oracle.quantize_act(np.ascontiguousarray(X[toks]), inv)
        gcodes, gscales, gzeros = w4a8.unpack_codes(packed, N, K, group)
        rows_t = torch.from_numpy(rows).cuda()
        toks_t = torch.from_numpy(toks).cuda()
        assert np.array_equal(gcodes[rows_t].cpu().numpy(), ocodes), (label, M, "codes")
        assert np.array_equal(gzeros[:, rows_t].cpu().numpy(), ozeros), (label, M, "zero-points")
        assert np.array_equal(gscales[:, rows_t].cpu().numpy().view(np.uint32),
                              oscales.view(np.uint32)), (label, M, "steps")
        assert np.array_equal(Xq[toks_t].cpu().numpy(), oXq), (label, M, "Xq")
        assert np.array_equal(tok[toks_t].cpu().numpy().view(np.uint32), otok.view(np.uint32))
        if acc_for_M == M:
            # the INT32 accumulators of the same launch configuration, on the same sample
            acc = w4a8.linear_acc_i32(Xq, packed, N, group, ws)
            w4a8.check_status(ws)
            G = acc.shape[0]
            got_acc = acc[:, toks_t][:, :, rows_t].cpu().numpy()
            want_acc = oracle.linear_acc(oXq, ocodes, ozeros, group).reshape(G, len(toks), len(rows))
            assert np.array_equal(got_acc, want_acc), (label, M, "INT32 accumulators")
            del acc
        got = bf16_bits(Y[toks_t][:, rows_t].contiguous())
        want = oracle.linear(oXq, otok, ocodes, oscales, ozeros, bias[rows], group)
        plan_splits = w4a8.linear_workspace_bytes(M, N, K, group) > 4096 + 4 * 4096
        if group == 0:
            # per-channel: one FP32 evaluation order whatever the K split (integer partials)
            bad = np.argwhere(got != want)
            assert bad.size == 0, (label, M, len(bad), bad[:4].tolist())
        else:
            y64 = oracle.linear_f64(oXq, otok, ocodes, oscales, ozeros, bias[rows], group)
            acc = oracle.linear_acc(oXq, ocodes, ozeros, group, wide=True)
            mag = (np.abs(acc) * (0.5 * oscales.astype(np.float64))[:, None, :]).sum(0)
            tol = bf16_ulp(y64) + 2.0 ** -20 * otok.astype(np.float64)[:, None] * mag
            err = np.abs(oracle.bf16_bits_to_float(got).astype(np.float64) - y64)
            bad = np.argwhere(err > tol)
            assert bad.size == 0, (label, M, len(bad), bad[:4].tolist(), plan_splits)
        del Xd, Xq, Y, ws
    del Wd, packed
    torch.cuda.empty_cache()


@pytest.mark.parametrize("shape_index", [0, 1, 2, 3])
def test_config2_opt_6_7b_block(shape_index):
    check_shape(2, shape_index, (2048, 1))


@pytest.mark.parametrize("shape_index", [0, 2, 3])
def test_config3_llama_7b_block_group128(shape_index):
    check_shape(3, shape_index, (1, 8, 512, 2048))


@pytest.mark.parametrize("shape_index", [0, 1, 2, 3, 4, 5, 6, 7])
def test_config4_large_linears(shape_index):
    # (the first shape, 9216 -> 36864, also compares the INT32 accumulators at 2048 tokens)
    check_shape(4, shape_index, (2048, 16), acc_for_M=2048 if shape_index == 0 else None)


def test_config5_token_sweep_group128():
    check_shape(5, 0, (1, 2, 4, 16, 64, 256, 1024, 4096, 16384))
