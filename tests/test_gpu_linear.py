"""GPU parity of the quantized linear layer against the CPU oracle, through the C ABI:
INT32 accumulators bit-exact; BF16 outputs bit-exact for per-channel weights and within
1 BF16 ulp (+ the FP32 reordering allowance) for group-128 weights and split-K."""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from util import Guarded, Problem, bf16_bits, check_y, guarded_workspace

pytestmark = pytest.mark.gpu


def run_linear(prob, opts=None, packed=None, want_acc=True):
    d = prob.dev
    if packed is None:
        packed = w4a8.pack_weights(d["W"], d["s"], prob.group)
    # every output and the workspace sit between patterned margins that must stay untouched
    G = prob.K // prob.group if prob.group else 1
    gXq, gtok = Guarded((prob.M, prob.K), torch.int8), Guarded((prob.M,), torch.float32)
    gY, gacc = Guarded((prob.M, prob.N), torch.bfloat16), Guarded((G, prob.M, prob.N), torch.int32)
    gws = guarded_workspace(w4a8.linear_workspace_bytes(prob.M, prob.N, prob.K, prob.group, opts))
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"], out=(gXq.t, gtok.t))
    Y = w4a8.linear(Xq, tok, packed, d["bias"], prob.N, prob.group, gws.t, opts, out=gY.t)
    acc = w4a8.linear_acc_i32(Xq, packed, prob.N, prob.group, gws.t, opts, out=gacc.t) if want_acc else None
    w4a8.check_status(gws.t)
    for g, what in ((gXq, "Xq"), (gtok, "tok_scale"), (gY, "Y"), (gacc, "acc"), (gws, "workspace")):
        g.check(what)
    return bf16_bits(Y), (acc.cpu().numpy() if want_acc else None)


@pytest.mark.parametrize("group", [0, 128])
def test_simple_path_config1(group):
    prob = Problem(768, 768, 16, group, seed=0)
    Y, acc = run_linear(prob, w4a8.make_opts(w4a8.PATH_SIMPLE))
    assert np.array_equal(acc, prob.oracle_acc())
    check_y(prob, Y, exact=True)      # same FP32 order as the oracle in both modes


@pytest.mark.parametrize("group", [0, 128])
def test_tcgen05_config1(group):
    prob = Problem(768, 768, 16, group, seed=0)
    Y, acc = run_linear(prob, w4a8.make_opts(w4a8.PATH_TCGEN05))
    assert np.array_equal(acc, prob.oracle_acc())
    check_y(prob, Y, exact=(group == 0))


@pytest.mark.parametrize("tok_tile,group", [(t, g) for g in (0, 128) for t in (16, 32, 64, 128, 192, 256)
                                            if not (g and t > 128)])   # group mode tiles at most 128 tokens
def test_tcgen05_token_tiles_and_ragged_edges(tok_tile, group):
    # M spans several token tiles with a ragged tail; N = 200 is not a multiple of 128
    M = tok_tile * 2 + 5
    prob = Problem(1024, 200, M, group, seed=tok_tile + group, dist="laplace", outliers=0.01,
                   mult=20.0)
    Y, acc = run_linear(prob, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=tok_tile))
    assert np.array_equal(acc, prob.oracle_acc())
    check_y(prob, Y, exact=(group == 0))


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("M,split", [(1, 2), (5, 3), (16, 8), (40, 5)])
def test_tcgen05_split_k(M, split, group):
    prob = Problem(1024, 384, M, group, seed=M + split + group)
    opts = w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=split)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], group)
    for _ in range(2):                       # second call reuses the self-cleaned workspace
        Y, acc = run_linear(prob, opts, packed)
        assert np.array_equal(acc, prob.oracle_acc())
        check_y(prob, Y, exact=(group == 0))


@pytest.mark.parametrize("group", [0, 128])
def test_auto_path_matches_simple_path_and_oracle(group):
    prob = Problem(2048, 1536, 300, group, seed=77, dist="laplace", outliers=0.01, mult=20.0)
    Y, acc = run_linear(prob)
    Ys, accs = run_linear(prob, w4a8.make_opts(w4a8.PATH_SIMPLE))
    assert np.array_equal(acc, accs)
    assert np.array_equal(acc, prob.oracle_acc())
    check_y(prob, Y, exact=(group == 0))
    check_y(prob, Ys, exact=True)


def test_no_bias_no_scale_and_persistent_many_tiles():
    # more tiles than SMs, so every CTA walks several tiles and both accumulator buffers
    prob = Problem(512, 128 * 40, 130, 0, seed=9, scaled=False, with_bias=False)
    Y, acc = run_linear(prob, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=16))
    assert np.array_equal(acc, prob.oracle_acc())
    check_y(prob, Y, exact=True)


def test_worst_case_magnitudes_do_not_overflow():
    K, N, M = 36864, 128, 4
    W = np.zeros((N, K), dtype=np.float16)
    W[:, :] = 1.0
    W[:, 0] = 0.0                      # lo = 0, hi = 1 -> z = 0, every other code 13 (t2 = 26)
    W[1::2] *= -1                      # negative rows: z = 13, codes 0 (t2 = -26)
    X = np.full((M, K), 3.0, dtype=np.float16)
    X[1] = -3.0
    prob = Problem.__new__(Problem)
    prob.K, prob.N, prob.M, prob.group, prob.rows = K, N, M, 0, None
    prob.host = {"W": W, "X": X, "s": None, "inv_s": None, "bias": None}
    prob.dev = {k: (torch.from_numpy(v).cuda() if v is not None else None) for k, v in prob.host.items()}
    prob.codes, prob.scales, prob.zeros = oracle.pack_weights(W, None, 0)
    prob.Xq, prob.tok = oracle.quantize_act(X, None)
    prob.bias_sel = None
    Y, acc = run_linear(prob)
    want = prob.oracle_acc()
    assert np.abs(want).max() == 127 * 26 * (K - 1)
    assert np.array_equal(acc, want)
    check_y(prob, Y, exact=True)


def test_wrong_blob_is_reported_not_computed():
    prob = Problem(768, 768, 16, 0, seed=0)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], 128)      # packed for group mode
    Xq, tok = w4a8.quantize_act(prob.dev["X"], prob.dev["inv_s"])
    for path in (w4a8.PATH_SIMPLE, w4a8.PATH_TCGEN05):
        ws = w4a8.new_workspace(16, 768, 768, 0)
        buf = torch.zeros(max(packed.numel(), w4a8.packed_bytes(768, 768, 0)), dtype=torch.uint8, device="cuda")
        buf[:packed.numel()] = packed
        w4a8.linear(Xq, tok, buf, None, 768, 0, ws, w4a8.make_opts(path))
        assert w4a8.poll_status(ws) == 8          # W4A8_ERR_BAD_BLOB
        assert w4a8.poll_status(ws) == 0          # cleared by the poll


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("M", [1, 2, 3, 4])
def test_gemv_path_small_token_counts(M, group):
    # K = 1280 is ten k-blocks: K slices of 2 k-blocks; N = 200 is not a multiple of the row tile
    prob = Problem(1280, 200, M, group, seed=50 + M + group, dist="laplace", outliers=0.01, mult=20.0)
    opts = w4a8.make_opts(w4a8.PATH_GEMV)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], group)
    for _ in range(2):                       # the second call reuses the self-cleaned workspace
        Y, acc = run_linear(prob, opts, packed)
        assert np.array_equal(acc, prob.oracle_acc())
        check_y(prob, Y, exact=(group == 0))
    # the automatic choice (this kernel or the tensor-core one) meets the same bar
    Ya, acca = run_linear(prob, None, packed)
    assert np.array_equal(acca, prob.oracle_acc())
    check_y(prob, Ya, exact=(group == 0))


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("M,K", [(1, 512), (2, 2560), (4, 4224), (1, 4224), (3, 1024)])
def test_gemv_row_slab_kernel(M, K, group):
    """Wide layers take the variant in which a CTA owns 32 rows over all of K (4, 8 or 16 warps
    split the k-blocks): N = 3080 gives 100 slabs and a ragged last tile."""
    prob = Problem(K, 3080, M, group, seed=300 + M + K + group, dist="laplace", outliers=0.01, mult=20.0)
    opts = w4a8.make_opts(w4a8.PATH_GEMV)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], group)
    for _ in range(2):
        Y, acc = run_linear(prob, opts, packed)
        assert np.array_equal(acc, prob.oracle_acc())
        check_y(prob, Y, exact=(group == 0))


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("warps", [4, 8, 16, 32])
def test_gemv_row_slab_kernel_with_requested_warps(warps, group):
    """Naming the warps of a row-slab CTA selects that kernel whatever the shape: ten k-blocks,
    so CTAs of 16 and 32 warps have warps without work; N = 200 leaves a ragged last tile."""
    M = 2 if warps == 32 else 3
    prob = Problem(1280, 200, M, group, seed=400 + warps + group, dist="laplace", outliers=0.01, mult=20.0)
    opts = w4a8.make_opts(w4a8.PATH_GEMV, decode_warps=warps)
    Y, acc = run_linear(prob, opts)
    assert np.array_equal(acc, prob.oracle_acc())
    check_y(prob, Y, exact=(group == 0))


def test_gemv_path_rejects_more_than_four_tokens():
    assert w4a8.linear_workspace_bytes(5, 256, 256, 0, w4a8.make_opts(w4a8.PATH_GEMV)) == 0


@pytest.mark.parametrize("tok_tile", [128, 192, 256])
def test_tcgen05_two_cta_clusters(tok_tile):
    """Two CTAs of a cluster share the expansion of every code tile (each writes half of the rows
    into both CTAs' stages).  Three token tiles: the last one is paired with an empty tile; N = 200
    leaves a ragged row tile.  The one-CTA form of the same plan gives the same bits."""
    M = tok_tile * 2 + 5
    prob = Problem(1024, 200, M, 0, seed=700 + tok_tile, dist="laplace", outliers=0.01, mult=20.0)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], 0)
    Y2, acc2 = run_linear(prob, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=tok_tile, cluster=2), packed)
    Y1, acc1 = run_linear(prob, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=tok_tile, cluster=1), packed)
    assert np.array_equal(acc2, prob.oracle_acc())
    assert np.array_equal(acc1, acc2) and np.array_equal(Y1, Y2)
    check_y(prob, Y2, exact=True)


def test_tcgen05_two_cta_clusters_many_units_and_split_k():
    # more units than clusters (every cluster walks several units, stages and accumulators wrap),
    # then a K split on top (partial tiles, last-arriver reduction, an empty partner tile)
    prob = Problem(1536, 128 * 44, 300, 0, seed=711)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], 0)
    want = prob.oracle_acc()
    for split in (1, 3):
        opts = w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=split, tok_tile=128, cluster=2)
        for _ in range(2):
            Y, acc = run_linear(prob, opts, packed)
            assert np.array_equal(acc, want)
            check_y(prob, Y, exact=True)


def test_cluster_option_is_validated():
    assert w4a8.linear_workspace_bytes(300, 256, 256, 0, w4a8.make_opts(tok_tile=64, cluster=2)) == 0
    assert w4a8.linear_workspace_bytes(300, 256, 256, 0, w4a8.make_opts(tok_tile=128, cluster=3)) == 0
    assert w4a8.linear_plan(2048, 8192, 8192, 0)["cluster"] == 3         # automatic: the MMA pair
    assert w4a8.linear_plan(2048, 4096, 4096, 0)["cluster"] == 1         # small layers: one CTA
    assert w4a8.linear_plan(512, 8192, 8192, 0)["cluster"] == 1
    assert w4a8.linear_plan(2048, 4096, 4096, 0, w4a8.make_opts(tok_tile=256, cluster=2))["cluster"] == 2


@pytest.mark.parametrize("tok_tile,split", [(16, 1), (16, 4), (128, 1), (256, 1)])
def test_tcgen05_offset_tables(tok_tile, split):
    """Level tables stored with an offset (cheaper expansion) and taken out again with the tokens'
    sums: the same INT32 sums and BF16 bits, every zero-point and both special codes in play."""
    M = 2 * tok_tile + 5 if tok_tile > 16 else 13
    prob = Problem(1024, 200, M, 0, seed=800 + tok_tile + split, dist="laplace", outliers=0.01, mult=20.0)
    opts = w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=split, tok_tile=tok_tile, offset_tables=1)
    for _ in range(2):
        Y, acc = run_linear(prob, opts)
        assert np.array_equal(acc, prob.oracle_acc())
        check_y(prob, Y, exact=True)
    assert len(np.unique(prob.zeros)) >= 4                      # several zero-points among the rows
    assert w4a8.linear_workspace_bytes(16, 256, 256, 128, w4a8.make_opts(offset_tables=1)) == 0


def test_tcgen05_offset_tables_every_zero_point():
    """Rows whose ranges are built to give every zero-point 0..13, values in both special bands."""
    K, N, M = 512, 168, 40
    rng = np.random.default_rng(5)
    W = np.empty((N, K), dtype=np.float16)
    for n in range(N):
        z = n % 14
        vals = rng.uniform(-z, 13 - z, size=K)
        vals[0], vals[1], vals[2], vals[3] = -z, 13 - z, 0.5, -0.5
        W[n] = (vals * 0.01).astype(np.float16)
    prob = Problem.__new__(Problem)
    X = (rng.standard_normal((M, K)) * 2).astype(np.float16)
    prob.K, prob.N, prob.M, prob.group, prob.rows = K, N, M, 0, None
    prob.host = {"W": W, "X": X, "s": None, "inv_s": None, "bias": None}
    prob.dev = {k: (torch.from_numpy(v).cuda() if v is not None else None) for k, v in prob.host.items()}
    prob.codes, prob.scales, prob.zeros = oracle.pack_weights(W, None, 0)
    prob.Xq, prob.tok = oracle.quantize_act(X, None)
    prob.bias_sel = None
    assert set(np.unique(prob.zeros)) == set(range(14))
    for tok_tile in (16, 64):
        Y, acc = run_linear(prob, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=tok_tile, offset_tables=1))
        assert np.array_equal(acc, prob.oracle_acc())
        check_y(prob, Y, exact=True)


def test_tcgen05_mma_pair():
    """Two CTAs as one MMA pair (cta_group::2): two row tiles per instruction, each CTA loads half
    of the 256-token tile; the leader's barriers collect both CTAs' arrivals.  Ragged token tile,
    several units per cluster, a K split; same bits as the one-CTA form."""
    prob = Problem(1536, 128 * 44, 2 * 256 + 37, 0, seed=721)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], 0)
    want = prob.oracle_acc()
    for split, dw in ((1, 16), (1, 8), (3, 16)):
        opts = w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=split, tok_tile=256, decode_warps=dw, cluster=3)
        for _ in range(2):
            Y, acc = run_linear(prob, opts, packed)
            assert np.array_equal(acc, want)
            check_y(prob, Y, exact=True)
    # the same pair with three k-blocks per barrier round (k-block counts that are multiples of three)
    for split in (1, 2):
        opts = w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=split, tok_tile=256, cluster=5)
        for _ in range(2):
            Y, acc = run_linear(prob, opts, packed)
            assert np.array_equal(acc, want)
            check_y(prob, Y, exact=True)
    assert w4a8.linear_workspace_bytes(300, 512, 1024, 0, w4a8.make_opts(tok_tile=256, cluster=5)) == 0  # 8 k-blocks
    assert w4a8.linear_workspace_bytes(300, 384, 256, 0, w4a8.make_opts(tok_tile=256, cluster=3)) == 0   # odd row tiles
    assert w4a8.linear_workspace_bytes(300, 512, 256, 0, w4a8.make_opts(tok_tile=128, cluster=3)) == 0
    assert w4a8.linear_workspace_bytes(300, 512, 256, 128, w4a8.make_opts(tok_tile=256, cluster=3)) == 0


def test_tcgen05_two_row_tiles_per_cta():
    """One CTA on two row tiles and one token tile (cluster form 4): both tiles' MMAs read the same
    token buffer, the weight ring is numbered by (k-block, tile) items, the two accumulators are
    handed back one after the other.  Ragged token tile, rows past N in the last tile, several units
    per CTA (more units than SMs), a K split, asymmetric-free path; same bits as the one-CTA form."""
    prob = Problem(1536, 128 * 44 - 24, 3 * 256 + 37, 0, seed=722)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], 0)
    want = prob.oracle_acc()
    for split in (1, 3):
        opts = w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=split, tok_tile=256, decode_warps=16, cluster=4)
        for _ in range(2):
            Y, acc = run_linear(prob, opts, packed)
            assert np.array_equal(acc, want)
            check_y(prob, Y, exact=True)
    # one k-block only (fewer items than weight buffers), and many k-blocks on few units
    for K, N, M in ((128, 256, 40), (4096, 512, 300)):
        small = Problem(K, N, M, 0, seed=723 + K)
        Y, acc = run_linear(small, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=256, cluster=4))
        assert np.array_equal(acc, small.oracle_acc())
        check_y(small, Y, exact=True)
    assert w4a8.linear_workspace_bytes(300, 384, 256, 0, w4a8.make_opts(tok_tile=256, cluster=4)) == 0   # odd row tiles
    assert w4a8.linear_workspace_bytes(300, 512, 256, 0, w4a8.make_opts(tok_tile=128, cluster=4)) == 0
    assert w4a8.linear_workspace_bytes(300, 512, 256, 0, w4a8.make_opts(tok_tile=256, decode_warps=8, cluster=4)) == 0
    assert w4a8.linear_workspace_bytes(300, 512, 256, 128, w4a8.make_opts(tok_tile=256, cluster=4)) == 0


def test_automatic_plan_takes_the_mma_pair_for_many_tokens():
    """From 1024 tokens on, on layers of at least 8192 x 8192, the library's own plan is the MMA
    pair with offset tables (per-channel 4-bit weights, even numbers of row tiles and k-blocks); the
    bits do not depend on the plan.  The oracle recomputes a sample of rows (every output element
    depends only on its own weight row and token)."""
    K, N, M = 8192, 8192, 1024 + 77
    assert w4a8.linear_plan(M, N, K, 0)["cluster"] == 3
    assert w4a8.linear_plan(1000, N, K, 0)["cluster"] == 1            # fewer tokens
    assert w4a8.linear_plan(M, N - 128, K, 0)["cluster"] == 1         # odd row tiles
    assert w4a8.linear_plan(M, N, K + 128, 0)["cluster"] == 1         # odd k-blocks
    assert w4a8.linear_plan(M, N, K, 128)["cluster"] == 1             # group steps
    assert w4a8.linear_plan(M, 4096, K, 0)["cluster"] == 1            # a narrow layer
    rows = np.array([0, 1, 127, 128, 129, 255, 256, 4095, 4096, N - 129, N - 128, N - 1])
    prob = Problem(K, N, M, 0, seed=731, rows=rows)
    d = prob.dev
    packed = w4a8.pack_weights(d["W"], d["s"], 0)
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    outs = []
    for opts in (None, w4a8.make_opts(w4a8.PATH_TCGEN05, cluster=1)):
        ws = w4a8.new_workspace(M, N, K, 0, opts)
        Y = w4a8.linear(Xq, tok, packed, d["bias"], N, 0, ws, opts)
        acc = w4a8.linear_acc_i32(Xq, packed, N, 0, ws, opts)
        w4a8.check_status(ws)
        outs.append((bf16_bits(Y), acc.cpu().numpy().reshape(M, N)))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    assert np.array_equal(outs[0][1][:, rows], prob.oracle_acc().reshape(M, len(rows)))
    assert np.array_equal(outs[0][0][:, rows], prob.oracle_y_bits())


def test_unit_order_runs_of_token_tiles():
    """The order in which CTAs take (token tile, row tile) units - runs of tok_run token tiles,
    token tile fastest inside a run - changes no bit: every run length, a ragged last run, with a
    K split, in the cluster forms."""
    prob = Problem(512, 128 * 6, 5 * 128 + 9, 0, seed=741)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], 0)
    want = prob.oracle_acc()
    for run in (1, 2, 3, 6, 50):
        for split in (1, 2):
            Y, acc = run_linear(prob, w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=split, tok_tile=128, tok_run=run), packed)
            assert np.array_equal(acc, want)
            check_y(prob, Y, exact=True)
    big = Problem(256, 128 * 6, 5 * 256 + 9, 0, seed=742)
    packed = w4a8.pack_weights(big.dev["W"], big.dev["s"], 0)
    want = big.oracle_acc()
    for cluster, tok_tile in ((2, 128), (3, 256), (4, 256)):
        for run in (2, 4):
            Y, acc = run_linear(big, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=tok_tile, cluster=cluster, tok_run=run), packed)
            assert np.array_equal(acc, want)
            check_y(big, Y, exact=True)
    # (group steps, narrow tiles, 3-bit codes: the request is accepted and the order stays one tile per run)
    grp = Problem(512, 128 * 3, 3 * 64 + 5, 128, seed=743)
    Y, acc = run_linear(grp, w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=64, tok_run=2))
    assert np.array_equal(acc, grp.oracle_acc())
    check_y(grp, Y, exact=False)
    assert w4a8.linear_workspace_bytes(300, 256, 256, 0, w4a8.make_opts(w4a8.PATH_GEMV, tok_run=2)) == 0
