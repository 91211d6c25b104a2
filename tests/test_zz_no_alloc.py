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


def first_shape(shapes, group, more_than):
    """First (M, N, K) whose automatic plan needs more workspace than `more_than` bytes."""
    for M, N, K in shapes:
        if w4a8.linear_workspace_bytes(M, N, K, group) > more_than:
            return M, N, K
    raise AssertionError("no candidate shape has the wanted plan")


@pytest.mark.parametrize("group", [0, 128])
def test_static_scratch_entry_point_matches_linear_twice(group):
    # a shape whose automatic plan splits K: more scratch than the status block alone
    M, N, K = first_shape([(16, 384, 1024), (16, 384, 4096), (16, 256, 8192)], group, 1024)
    prob = Problem(K, N, M, group, seed=123 + group)
    d = prob.dev
    packed = w4a8.pack_weights(d["W"], d["s"], group)
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    ws = w4a8.new_workspace(M, N, K, group)
    want = w4a8.linear(Xq, tok, packed, d["bias"], N, group, ws)
    w4a8.check_status(ws)
    want_bits = bf16_bits(want)
    check_y(prob, want_bits, exact=(group == 0))
    for call in range(2):
        out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        free_before, held_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        w4a8.linear_static(Xq, tok, packed, d["bias"], N, group, out)
        torch.cuda.synchronize()
        if call == 1:       # (the first call on a device may load the kernel's code)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call took device memory"
        assert torch.cuda.memory_allocated() == held_before
        assert w4a8.static_poll_status() == 0
        got = bf16_bits(out)
        assert np.array_equal(got, want_bits), f"call {call}: differs from w4a8_linear"
        check_y(prob, got, exact=(group == 0))


def test_static_scratch_entry_point_with_two_tokens():
    # two tokens: w4a8_linear picks the weight-streaming kernel here, the workspace-free call
    # the tensor-core kernel; per-channel results have the same bits either way
    prob = Problem(1024, 384, 2, 0, seed=321)
    d = prob.dev
    packed = w4a8.pack_weights(d["W"], d["s"], 0)
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    ws = w4a8.new_workspace(2, 384, 1024, 0)
    want_bits = bf16_bits(w4a8.linear(Xq, tok, packed, d["bias"], 384, 0, ws))
    w4a8.check_status(ws)
    for call in range(2):
        out = torch.full((2, 384), float("nan"), dtype=torch.bfloat16, device="cuda")
        w4a8.linear_static(Xq, tok, packed, d["bias"], 384, 0, out)
        torch.cuda.synchronize()
        assert np.array_equal(bf16_bits(out), want_bits), f"call {call}"
        check_y(prob, bf16_bits(out), exact=True)


def test_static_scratch_reports_a_blob_that_does_not_match():
    # a blob packed per channel, described to the call as group-128: the kernel touches nothing
    # but the status block, and the status is readable until the next call clears it
    prob = Problem(1024, 384, 16, 0, seed=322)
    d = prob.dev
    packed = w4a8.pack_weights(d["W"], d["s"], 0)
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    room = torch.zeros(w4a8.packed_bytes(384, 1024, 128), dtype=torch.uint8, device="cuda")
    room[:packed.numel()] = packed
    out = torch.zeros((16, 384), dtype=torch.bfloat16, device="cuda")
    w4a8.linear_static(Xq, tok, room, d["bias"], 384, 128, out)
    assert w4a8.static_poll_status() == 8            # W4A8_ERR_BAD_BLOB
    assert torch.count_nonzero(out).item() == 0
    w4a8.linear_static(Xq, tok, packed, d["bias"], 384, 0, out)
    assert w4a8.static_poll_status() == 0
    check_y(prob, bf16_bits(out), exact=True)


def test_static_scratch_rejects_plans_beyond_its_size():
    # a shape whose split-K partial tiles need more than the 8 MiB the library carries
    M, N, K = first_shape([(128, 8192, 22016), (256, 4096, 4096), (128, 16384, 32768)], 0, 8 << 20)
    Xq = torch.zeros((M, K), dtype=torch.int8, device="cuda")
    tok = torch.zeros((M,), dtype=torch.float32, device="cuda")
    packed = torch.zeros(w4a8.packed_bytes(N, K, 0), dtype=torch.uint8, device="cuda")
    out = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(w4a8.W4A8Error) as e:
        w4a8.linear_static(Xq, tok, packed, None, N, 0, out)
    assert e.value.status == 4          # W4A8_ERR_BUFFER_TOO_SMALL
