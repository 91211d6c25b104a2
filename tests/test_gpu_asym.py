"""GPU parity of the asymmetric-activation path (App. A.1 token-wise Min-Max asymmetric
quantizer, per-output-channel dINT4 weights) against the CPU oracle, through the C ABI.

The device stores the unsigned activation code and its zero-point shifted by 128 (INT8 and
INT32); the oracle keeps the paper's unsigned form.  Codes, zero-points, row sums and INT32
accumulators must agree bit for bit, step sizes as FP32 bit patterns, BF16 outputs bit for bit
(the FP32 evaluation order is the oracle's on every kernel path).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from paper_2311_05161_b200 import synth
from util import bf16_bits, to_dev

pytestmark = pytest.mark.gpu


def make(K, N, M, seed, dist="normal", shift=0.5):
    lay = synth.make_layer(K, N, M, seed, dist, 4, 30.0, True, True)
    # an offset per token is what the asymmetric quantizer is for
    rng = np.random.Generator(np.random.PCG64([seed, 7]))
    off = (rng.standard_normal((M, 1)) * shift).astype(np.float32)
    lay["X"] = (lay["X"].astype(np.float32) + off).astype(np.float16)
    return lay


def unpack(codes):
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


def host_rowsum(codes, zeros):
    c = unpack(codes).astype(np.int64)
    z = zeros[0].astype(np.int64)[:, None]
    return np.where(c == 14, 1, np.where(c == 15, -1, 2 * (c - z))).sum(1)


@pytest.mark.parametrize("M,K", [(1, 128), (7, 1024), (33, 4096), (5, 16384), (3, 20480)])
def test_quantizer_matches_oracle(M, K):
    lay = make(K, 128, M, seed=900 + M)
    lay["X"][0, :] = 0 if M > 1 else lay["X"][0, :]          # an all-zero token
    if M > 2:
        lay["X"][1, :] = np.abs(lay["X"][1, :])              # a one-sided token
    for inv in (None, lay["inv_s"]):
        Q, step, zx = oracle.quantize_act_asym(lay["X"], inv)
        Xq, tok, tz = w4a8.quantize_act_asym(to_dev(lay["X"]), to_dev(inv))
        assert np.array_equal(Xq.cpu().numpy().astype(np.int16) + 128, Q.astype(np.int16))
        assert np.array_equal(tz.cpu().numpy() + 128, zx)
        assert np.array_equal(tok.cpu().numpy().view(np.uint32), step.view(np.uint32))


@pytest.mark.parametrize("group", [0, 128])
def test_rowsum_matches_the_codes(group):
    N, K = 200, 1024
    lay = make(K, N, 4, seed=77)
    packed = w4a8.pack_weights(to_dev(lay["W"]), to_dev(lay["s"]), group)
    got = w4a8.weight_rowsum(packed, N, K, group).cpu().numpy()
    codes, scales, zeros = oracle.pack_weights(lay["W"], lay["s"], group)
    c = unpack(codes).astype(np.int64)
    G = zeros.shape[0]
    z = np.repeat(zeros.T.astype(np.int64), K // G, axis=1)
    t2 = np.where(c == 14, 1, np.where(c == 15, -1, 2 * (c - z)))
    want = t2.reshape(N, G, K // G).sum(2).T
    assert np.array_equal(got, want)


def run(lay, K, N, M, opts):
    d = {k: to_dev(v) for k, v in lay.items()}
    packed = w4a8.pack_weights(d["W"], d["s"], 0)
    rowsum = w4a8.weight_rowsum(packed, N, K, 0)
    Xq, tok, tz = w4a8.quantize_act_asym(d["X"], d["inv_s"])
    ws = w4a8.new_workspace(M, N, K, 0, opts)
    Y, acc = w4a8.linear_asym(Xq, tok, tz, packed, rowsum[0], d["bias"], N, ws, opts, want_acc=True)
    w4a8.check_status(ws)
    return bf16_bits(Y), acc.cpu().numpy()


def check(lay, Y, acc, rows=None, toks=None):
    W = lay["W"] if rows is None else lay["W"][rows]
    X = lay["X"] if toks is None else lay["X"][toks]
    bias = lay["bias"] if rows is None else lay["bias"][rows]
    codes, scales, zeros = oracle.pack_weights(np.ascontiguousarray(W), lay["s"], 0)
    Q, step, zx = oracle.quantize_act_asym(np.ascontiguousarray(X), lay["inv_s"])
    want_acc = oracle.linear_asym_acc(Q, zx, codes, zeros)
    assert np.abs(want_acc).max() < 2 ** 31
    assert np.array_equal(acc.astype(np.int64), want_acc)
    want = oracle.linear_asym(Q, step, zx, codes, scales, zeros, bias)
    bad = np.argwhere(Y != want)
    assert bad.size == 0, f"{len(bad)} BF16 outputs differ, first at {bad[0]}"


def test_simple_path():
    K, N, M = 768, 768, 16
    lay = make(K, N, M, seed=0)
    Y, acc = run(lay, K, N, M, w4a8.make_opts(w4a8.PATH_SIMPLE))
    check(lay, Y, acc)


@pytest.mark.parametrize("tok_tile", [16, 32, 64, 128, 192, 256])
def test_tcgen05_token_tiles_and_ragged_edges(tok_tile):
    K, N, M = 1024, 200, tok_tile * 2 + 5
    lay = make(K, N, M, seed=tok_tile, dist="laplace")
    Y, acc = run(lay, K, N, M, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=tok_tile))
    check(lay, Y, acc)


@pytest.mark.parametrize("M,split", [(1, 2), (5, 3), (16, 8), (40, 5)])
def test_tcgen05_split_k(M, split):
    K, N = 1024, 384
    lay = make(K, N, M, seed=M + split)
    Y, acc = run(lay, K, N, M, w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=split))
    check(lay, Y, acc)


@pytest.mark.parametrize("M", [1, 2, 4])
def test_gemv_path(M):
    K, N = 2048, 520
    lay = make(K, N, M, seed=40 + M)
    Y, acc = run(lay, K, N, M, w4a8.make_opts(w4a8.PATH_GEMV))
    check(lay, Y, acc)


@pytest.mark.parametrize("M", [1, 2])
def test_gemv_row_slab_kernel(M):
    K, N = 2560, 3080
    lay = make(K, N, M, seed=45 + M)
    Y, acc = run(lay, K, N, M, w4a8.make_opts(w4a8.PATH_GEMV))
    check(lay, Y, acc)


@pytest.mark.parametrize("M", [1, 3, 16, 100, 300])
def test_automatic_plan(M):
    K, N = 1024, 640
    lay = make(K, N, M, seed=60 + M)
    Y, acc = run(lay, K, N, M, None)
    check(lay, Y, acc)


def test_argument_checks():
    K, N, M = 256, 128, 4
    lay = make(K, N, M, seed=3)
    d = {k: to_dev(v) for k, v in lay.items()}
    packed = w4a8.pack_weights(d["W"], d["s"], 0)
    rowsum = w4a8.weight_rowsum(packed, N, K, 0)
    Xq, tok, tz = w4a8.quantize_act_asym(d["X"], d["inv_s"])
    ws = w4a8.new_workspace(M, N, K, 0)
    with pytest.raises(w4a8.W4A8Error) as e:
        w4a8.linear_asym(Xq, tok, None, packed, rowsum[0], None, N, ws)
    assert e.value.status == 1            # W4A8_ERR_NULL
    with pytest.raises(w4a8.W4A8Error) as e:
        w4a8.linear_asym(Xq, tok, tz, packed, None, None, N, ws)
    assert e.value.status == 1


@pytest.mark.parametrize("shape_index,M", [(1, 2048), (2, 2048), (3, 1)])
def test_full_size_opt_6_7b_shapes_sampled(shape_index, M):
    """The block's shapes at full size in the automatic plan; the oracle recomputes a seeded
    sample of rows and tokens (weights quantize per row, activations per token)."""
    wl = synth.WORKLOADS[2]
    K, N, label = wl.shapes[shape_index]
    seed = wl.seed(shape_index) + 5
    rng = np.random.Generator(np.random.PCG64([seed, 99]))
    W = synth.make_weights(N, K, seed)
    X = synth.make_activations(M, K, seed, wl.act_dist, wl.outlier_channels, wl.outlier_mult)
    X = (X.astype(np.float32) + (rng.standard_normal((M, 1)) * 0.5).astype(np.float32)).astype(np.float16)
    s, inv = synth.make_channel_scales(X, W)
    lay = {"W": W, "X": X, "s": s, "inv_s": inv, "bias": synth.make_bias(N, seed)}
    Y, acc = run(lay, K, N, M, None)
    rows = np.unique(np.concatenate([[0, 127, 128, N - 1], rng.choice(N, 60, replace=False)]))
    toks = np.unique(np.concatenate([[0, M - 1], rng.choice(M, min(M, 24), replace=False)]))
    check(lay, Y[np.ix_(toks, rows)], acc[np.ix_(toks, rows)], rows=rows, toks=toks)


@pytest.mark.parametrize("cluster", [2, 3, 4])
@pytest.mark.parametrize("offset_tables", [0, 1])
def test_cluster_forms_with_zero_points(cluster, offset_tables):
    """The zero-point term (and the offset term of the offset tables) in every cluster form of the
    tensor-core kernel: ragged token tile, rows past N in the last tile."""
    K, N, M = 512, 128 * 6 - 24, 2 * 256 + 37
    lay = make(K, N, M, seed=80 + cluster)
    Y, acc = run(lay, K, N, M, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=256, cluster=cluster,
                                              offset_tables=offset_tables))
    check(lay, Y, acc)


def test_large_layer_in_the_mma_pair_with_offset_tables_sampled():
    """A layer large enough for the automatic MMA pair with offset tables (8192 x 8192, more than
    1024 tokens): the zero-point term and the offset term leave the accumulator together."""
    K, N, M = 8192, 8192, 1024 + 53
    assert w4a8.linear_plan(M, N, K, 0)["cluster"] == 3
    seed = 4711
    rng = np.random.Generator(np.random.PCG64([seed, 99]))
    W = synth.make_weights(N, K, seed)
    X = synth.make_activations(M, K, seed, "normal", 8, 60.0)
    X = (X.astype(np.float32) + (rng.standard_normal((M, 1)) * 0.5).astype(np.float32)).astype(np.float16)
    s, inv = synth.make_channel_scales(X, W)
    lay = {"W": W, "X": X, "s": s, "inv_s": inv, "bias": synth.make_bias(N, seed)}
    Y, acc = run(lay, K, N, M, None)
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, N - 1], rng.choice(N, 40, replace=False)]))
    toks = np.unique(np.concatenate([[0, 255, 256, M - 1], rng.choice(M, 24, replace=False)]))
    check(lay, Y[np.ix_(toks, rows)], acc[np.ix_(toks, rows)], rows=rows, toks=toks)


# ---- group-128 weight steps with asymmetric activations ----
def run_group(K, N, M, opts, seed):
    lay = make(K, N, M, seed=seed, dist="laplace")
    d = {k: to_dev(v) for k, v in lay.items()}
    packed = w4a8.pack_weights(d["W"], d["s"], 128)
    rowsum = w4a8.weight_rowsum(packed, N, K, 128).contiguous()
    Xq, tok, tz = w4a8.quantize_act_asym(d["X"], d["inv_s"])
    ws = w4a8.new_workspace(M, N, K, 128, opts)
    codes, scales, zeros = oracle.pack_weights(lay["W"], lay["s"], 128)
    Q, step, zx = oracle.quantize_act_asym(lay["X"], lay["inv_s"])
    acc_w, y_w, wide = oracle.linear_asym_group(Q, step, zx, codes, scales, zeros, lay["bias"], 128)
    from util import bf16_ulp
    for _ in range(2):
        Y, acc = w4a8.linear_asym_group(Xq, tok, tz, packed, rowsum, d["bias"], N, 128, ws, opts, want_acc=True)
        w4a8.check_status(ws)
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_w), "group sums"
        mag = (np.abs(acc_w) * (0.5 * scales.astype(np.float64))[:, None, :]).sum(0)
        tol = bf16_ulp(wide) + 2.0 ** -20 * step.astype(np.float64)[:, None] * mag
        got = oracle.bf16_bits_to_float(bf16_bits(Y)).astype(np.float64)
        assert np.all(np.abs(got - wide) <= tol)


def test_group_weights_simple_path():
    run_group(768, 768, 16, w4a8.make_opts(w4a8.PATH_SIMPLE), seed=1300)


@pytest.mark.parametrize("tok_tile", [16, 64, 128])
def test_group_weights_tensor_core_path(tok_tile):
    run_group(1024, 200, 2 * tok_tile + 5, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=tok_tile), seed=1310 + tok_tile)


def test_group_weights_split_k_and_automatic_plan():
    run_group(1024, 384, 16, w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=4), seed=1320)
    run_group(2048, 640, 300, None, seed=1321)


@pytest.mark.parametrize("M,N", [(1, 200), (2, 200), (3, 200), (1, 3080), (4, 3080)])
def test_group_weights_weight_streaming_kernels(M, N):
    run_group(1280, N, M, w4a8.make_opts(w4a8.PATH_GEMV), seed=1330 + M + N)
