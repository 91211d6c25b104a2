"""The workspace-free entry point w4a8_linear_static against w4a8_linear.

Some users of the library cannot allocate device memory when they call it (their host
framework owns the whole device, or allocation is forbidden once serving runs), so they
have no workspace to give.  For them the library carries a fixed scratch array.  This test
calls that entry point through the C ABI twice in a row, on a shape whose plan splits K and
therefore really uses the scratch (tile counters and partial tiles), and expects the very
bits w4a8_linear produces.  It sits in the last-collected file so that a run that stops at
the first failure has already gone through every other test.
"""
import numpy as np
import pytest
import torch

import paper_2311_05161_b200 as w4a8
from util import Problem, bf16_bits, check_y

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("group", [0, 128])
def test_static_scratch_entry_point_matches_linear_twice(group):
    prob = Problem(1024, 384, 16, group, seed=123 + group)
    d = prob.dev
    packed = w4a8.pack_weights(d["W"], d["s"], group)
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    # the automatic plan for this shape splits K: more scratch than the status block alone
    assert w4a8.linear_workspace_bytes(16, 384, 1024, group) > 1024
    ws = w4a8.new_workspace(16, 384, 1024, group)
    want = w4a8.linear(Xq, tok, packed, d["bias"], 384, group, ws)
    w4a8.check_status(ws)
    want_bits = bf16_bits(want)
    check_y(prob, want_bits, exact=(group == 0))
    for call in range(2):
        out = torch.full((16, 384), float("nan"), dtype=torch.bfloat16, device="cuda")
        w4a8.linear_static(Xq, tok, packed, d["bias"], 384, group, out)
        torch.cuda.synchronize()
        got = bf16_bits(out)
        assert np.array_equal(got, want_bits), f"call {call}: differs from w4a8_linear"
        check_y(prob, got, exact=(group == 0))


def test_static_scratch_rejects_plans_beyond_its_size():
    # M = 256 tokens on a narrow layer splits K eight ways: 32 MiB of partial tiles
    M, N, K = 256, 4096, 4096
    assert w4a8.linear_workspace_bytes(M, N, K, 0) > (8 << 20)
    Xq = torch.zeros((M, K), dtype=torch.int8, device="cuda")
    tok = torch.zeros((M,), dtype=torch.float32, device="cuda")
    packed = torch.zeros(w4a8.packed_bytes(N, K, 0), dtype=torch.uint8, device="cuda")
    out = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(w4a8.W4A8Error) as e:
        w4a8.linear_static(Xq, tok, packed, None, N, 0, out)
    assert e.value.status == 4          # W4A8_ERR_BUFFER_TOO_SMALL
