"""GPU parity of the one-launch decode form (activation quantizer + linear layer for one to
four tokens) through the C ABI: BF16 outputs against the CPU oracle's quantizer followed by
its linear layer (bit-exact per channel, within the group tolerance for group-128 weights),
and bit for bit against the two-call path on the GPU."""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from paper_2311_05161_b200 import binding
from util import Guarded, Problem, bf16_bits, check_y, guarded_workspace

pytestmark = pytest.mark.gpu


def run_fused(prob, packed, X=None, inv_s=None):
    d = prob.dev
    X = d["X"] if X is None else X
    inv_s = d["inv_s"] if inv_s is None else inv_s
    # workspace (the quantizer may use its tail) and output between patterned margins
    gws = guarded_workspace(binding.quantize_linear_workspace_bytes(prob.M, prob.N, prob.K, prob.group))
    gY = Guarded((prob.M, prob.N), torch.bfloat16)
    ws = gws.t
    out = []
    for _ in range(2):                       # the second call reuses the self-cleaned workspace
        Y = binding.quantize_linear(X, inv_s, packed, d["bias"], prob.N, prob.group, ws, out=gY.t)
        w4a8.check_status(ws)
        gws.check("workspace")
        gY.check("Y")
        out.append(bf16_bits(Y))
    assert np.array_equal(out[0], out[1])
    return out[0]


def run_two_calls(prob, packed):
    d = prob.dev
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    opts = w4a8.make_opts(w4a8.PATH_GEMV)
    ws = w4a8.new_workspace(prob.M, prob.N, prob.K, prob.group, opts)
    Y = w4a8.linear(Xq, tok, packed, d["bias"], prob.N, prob.group, ws, opts)
    w4a8.check_status(ws)
    return bf16_bits(Y)


# N = 3080: 100 row slabs and a ragged last tile -> the row-slab kernel (4, 8 or 16 warps by K);
# N = 200: the two-phase kernel with K slices
@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("M,K,N", [(1, 512, 3080), (2, 2560, 3080), (4, 4224, 3080), (1, 4224, 3080),
                                   (3, 1024, 3080), (1, 1280, 200), (2, 1280, 200), (3, 2176, 200),
                                   (4, 1280, 200), (1, 4352, 136)])
def test_fused_decode_matches_oracle_and_two_call_path(M, K, N, group):
    prob = Problem(K, N, M, group, seed=700 + M + K + N + group, dist="laplace", outliers=0.01,
                   mult=20.0)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], group)
    Y = run_fused(prob, packed)
    check_y(prob, Y, exact=(group == 0))
    assert np.array_equal(Y, run_two_calls(prob, packed))


@pytest.mark.parametrize("N", [200, 3080])
def test_fused_decode_without_scale_and_bias_and_with_a_zero_token(N):
    prob = Problem(1280, N, 3, 0, seed=41 + N, scaled=False, with_bias=False)
    X = prob.host["X"].copy()
    X[1] = 0                                   # an all-zero token: step 0, codes 0, output 0
    prob.host["X"] = X
    prob.dev["X"] = torch.from_numpy(X).cuda()
    prob.Xq, prob.tok = oracle.quantize_act(X, None)
    assert prob.tok[1] == 0.0
    packed = w4a8.pack_weights(prob.dev["W"], None, 0)
    Y = run_fused(prob, packed)
    check_y(prob, Y, exact=True)
    assert not Y[1].any()


def test_fused_decode_full_size_decode_shapes_sampled_rows():
    """The four OPT-6.7B-shaped linears at M = 1, as the bench times them: the oracle computes
    256 seeded output rows of each."""
    rng = np.random.default_rng(5)
    for K, N in [(4096, 12288), (4096, 4096), (4096, 16384), (16384, 4096)]:
        rows = np.sort(rng.choice(N, size=256, replace=False))
        prob = Problem(K, N, 1, 0, seed=K + N, outliers=0.001, mult=60.0, rows=rows)
        packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], 0)
        Y = run_fused(prob, packed)
        check_y(prob, Y[:, rows], exact=True)


def test_fused_decode_quantizer_in_front_on_very_wide_layers():
    """N = 38016 gives 1188 row slabs of four warps: more than are resident at once, so the call
    runs the quantizer as a launch of its own into the tail of the workspace.  Same bits."""
    prob = Problem(256, 38016, 2, 0, seed=77)
    packed = w4a8.pack_weights(prob.dev["W"], prob.dev["s"], 0)
    Y = run_fused(prob, packed)
    check_y(prob, Y, exact=True)
    assert np.array_equal(Y, run_two_calls(prob, packed))


def test_fused_decode_rejects_bad_arguments():
    assert binding.quantize_linear_workspace_bytes(5, 256, 256, 0) == 0
    assert binding.quantize_linear_workspace_bytes(1, 256, 200, 0) == 0
    X = torch.zeros((5, 256), dtype=torch.float16, device="cuda")
    packed = torch.zeros(w4a8.packed_bytes(256, 256, 0), dtype=torch.uint8, device="cuda")
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(w4a8.W4A8Error) as e:
        binding.quantize_linear(X, None, packed, None, 256, 0, ws)
    assert e.value.status == 2          # W4A8_ERR_SHAPE
    ws_small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(w4a8.W4A8Error) as e:
        binding.quantize_linear(X[:1], None, packed, None, 256, 0, ws_small)
    assert e.value.status == 4          # W4A8_ERR_BUFFER_TOO_SMALL
