"""GPU parity of the 3-bit dINT path (Section 4.2 with b = 3; Tables 10-11) through the C ABI:
codes, steps and zero-points of the packer bit for bit against the oracle, INT32 sums bit for
bit, BF16 outputs bit for bit (per channel) or within the group tolerance, on the simple and
the tensor-core kernel, at the shapes of the first two benchmark configurations too."""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from paper_2311_05161_b200 import synth
from util import Guarded, bf16_bits, bf16_ulp, guarded_workspace, to_dev

pytestmark = pytest.mark.gpu


def run(K, N, M, group, shift, opt_kw, seed, dist="laplace"):
    lay = synth.make_layer(K, N, M, seed, dist, 0.01, 20.0)
    d = {k: to_dev(v) for k, v in lay.items()}
    packed = w4a8.pack_weights(d["W"], d["s"], group, level_shift=shift, bits=3)
    assert packed.numel() == w4a8.packed_bytes(N, K, group, 3)
    codes, scales, zeros = oracle.pack_weights_bits(lay["W"], lay["s"], group, 3, shift)
    gc, gs, gz = w4a8.unpack_codes(packed, N, K, group, bits=3)
    assert np.array_equal(gc.cpu().numpy(), codes), "codes"
    assert np.array_equal(gz.cpu().numpy(), zeros), "zero-points"
    assert np.array_equal(gs.cpu().numpy().view(np.uint32), scales.view(np.uint32)), "steps"
    oXq, otok = oracle.quantize_act(lay["X"], lay["inv_s"])
    acc_w, y_w, wide = oracle.linear_bits(oXq, otok, codes, scales, zeros, lay["bias"], group, 3, shift)
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    opts = w4a8.make_opts(level_shift=shift, bits=3, **opt_kw)
    G = K // group if group else 1
    gY, gacc = Guarded((M, N), torch.bfloat16), Guarded((G, M, N), torch.int32)
    gws = guarded_workspace(w4a8.linear_workspace_bytes(M, N, K, group, opts))
    for _ in range(2):
        Y = w4a8.linear(Xq, tok, packed, d["bias"], N, group, gws.t, opts, out=gY.t)
        acc = w4a8.linear_acc_i32(Xq, packed, N, group, gws.t, opts, out=gacc.t)
        w4a8.check_status(gws.t)
        for g, what in ((gY, "Y"), (gacc, "acc"), (gws, "workspace")):
            g.check(what)
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_w), "INT32 sums"
        got = bf16_bits(Y)
        if group == 0:
            bad = np.argwhere(got != y_w)
            assert bad.size == 0, f"{len(bad)} BF16 outputs differ, first at {bad[0]}"
        else:
            mag = (np.abs(acc_w) * (scales.astype(np.float64) / 2 ** shift)[:, None, :]).sum(0)
            tol = bf16_ulp(wide) + 2.0 ** -20 * otok.astype(np.float64)[:, None] * mag
            err = np.abs(oracle.bf16_bits_to_float(got).astype(np.float64) - wide)
            assert np.all(err <= tol)


def test_table_matches_eq6_for_three_bits():
    for shift in (1, 2, 3):
        for z in range(6):
            assert w4a8.dint_table(z, 3, shift) == [(c - z) * 2 ** shift for c in range(6)] + [1, -1]
            assert w4a8.dint_table(z, 3, shift) == list(oracle.dint_table_fmt(z, shift, b=3)[:8])
    assert w4a8.packed_bytes(768, 768, 0, 3) == 256 + 3072 + 768 + 36 * 6144


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("shift", [1, 2])
def test_simple_path_config1(group, shift):
    run(768, 768, 16, group, shift, dict(path=w4a8.PATH_SIMPLE), seed=shift, dist="normal")


@pytest.mark.parametrize("tok_tile,group", [(t, g) for g in (0, 128) for t in (16, 32, 64, 128, 192, 256)
                                            if not (g and t > 128)])
def test_tcgen05_token_tiles_and_ragged_edges(tok_tile, group):
    run(1024, 200, tok_tile * 2 + 5, group, 1, dict(path=w4a8.PATH_TCGEN05, tok_tile=tok_tile),
        seed=40 + tok_tile + group)


@pytest.mark.parametrize("group", [0, 128])
def test_split_k_automatic_plan_and_single_token(group):
    run(1024, 384, 16, group, 1, dict(path=w4a8.PATH_TCGEN05, split_k=4), seed=50 + group)
    run(1024, 640, 300, group, 2, {}, seed=60 + group)          # automatic plan
    run(2048, 520, 1, group, 1, {}, seed=70 + group)            # one token: the tensor-core kernel too
    run(768, 128 * 40, 130, group, 1, dict(path=w4a8.PATH_TCGEN05, tok_tile=16), seed=80 + group)  # many tiles per CTA


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("M", [1, 2])
def test_weight_streaming_kernel_reads_three_bit_tiles(M, group):
    """One and two tokens on layers wide enough for row slabs: the weight-streaming kernel with
    the 3-bit tile layout and the 8-entry table (automatic plan and 8 / 16 warps on request)."""
    K, N = 1280, 3072 + 128
    assert w4a8.linear_plan(M, N, K, group, w4a8.make_opts(bits=3))["kernel"] == "weight-streaming"
    run(K, N, M, group, 1, {}, seed=90 + M + group)
    run(K, N, M, group, 2, dict(path=w4a8.PATH_GEMV, decode_warps=16), seed=95 + M + group)
    run(K, N - 24, M, group, 1, dict(path=w4a8.PATH_GEMV, decode_warps=8), seed=99 + M + group)   # rows past N


def test_unsupported_combinations_are_refused():
    # narrow layers have no row slabs, and the K-sliced weight-streaming kernel reads 4-bit tiles
    assert w4a8.linear_workspace_bytes(2, 256, 256, 0, w4a8.make_opts(w4a8.PATH_GEMV, bits=3)) == 0
    assert w4a8.linear_workspace_bytes(4, 4096, 1024, 0, w4a8.make_opts(w4a8.PATH_GEMV, bits=3)) == 0
    assert w4a8.linear_workspace_bytes(300, 256, 256, 0, w4a8.make_opts(tok_tile=128, cluster=2, bits=3)) == 0
    assert w4a8.linear_workspace_bytes(300, 256, 256, 0, w4a8.make_opts(bits=5)) == 0
    assert w4a8.linear_plan(1, 1024, 4096, 0, w4a8.make_opts(bits=3))["kernel"] == "tcgen05"
    assert w4a8.linear_plan(1, 4096, 4096, 0, w4a8.make_opts(bits=3))["kernel"] == "weight-streaming"
    assert w4a8.linear_plan(4, 4096, 4096, 0, w4a8.make_opts(bits=3))["kernel"] == "tcgen05"


@pytest.mark.parametrize("shape_index", [0, 3])
def test_config2_shapes_on_sampled_rows(shape_index):
    """OPT-6.7B-shaped linears at full size (M = 2048 and M = 1), automatic plan, sampled outputs."""
    wl = synth.WORKLOADS[2]
    K, N, _ = wl.shapes[shape_index]
    seed = wl.seed(shape_index)
    W = synth.make_weights(N, K, seed)
    rng = np.random.Generator(np.random.PCG64([seed, 3]))
    rows = np.array(sorted({0, 127, 128, N - 1, *map(int, rng.choice(N, 60, replace=False))}))
    Wd = to_dev(W)
    for M in (2048, 1):
        X = synth.make_activations(M, K, seed, wl.act_dist, wl.outlier_channels, wl.outlier_mult)
        s, inv = synth.make_channel_scales(X, W)
        bias = synth.make_bias(N, seed)
        packed = w4a8.pack_weights(Wd, to_dev(s), 0, bits=3)
        Xq, tok = w4a8.quantize_act(to_dev(X), to_dev(inv))
        opts = w4a8.make_opts(bits=3)
        ws = w4a8.new_workspace(M, N, K, 0, opts)
        Y = w4a8.linear(Xq, tok, packed, to_dev(bias), N, 0, ws, opts)
        w4a8.check_status(ws)
        toks = np.array(sorted({0, M - 1, *map(int, rng.choice(M, min(M, 40), replace=False))}))
        codes, scales, zeros = oracle.pack_weights_bits(np.ascontiguousarray(W[rows]), s, 0, 3)
        gc, gs, gz = w4a8.unpack_codes(packed, N, K, 0, bits=3)
        rows_t, toks_t = torch.from_numpy(rows).cuda(), torch.from_numpy(toks).cuda()
        assert np.array_equal(gc[rows_t].cpu().numpy(), codes)
        oXq, otok = oracle.quantize_act(np.ascontiguousarray(X[toks]), inv)
        _, want, _ = oracle.linear_bits(oXq, otok, codes, scales, zeros, bias[rows], 0, 3)
        got = bf16_bits(Y[toks_t][:, rows_t].contiguous())
        assert np.array_equal(got, want), (K, N, M)
