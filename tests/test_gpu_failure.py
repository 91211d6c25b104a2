"""The failure path of the tensor-core kernel, made on the host side of the fence: a test hook
leaves out one token load, so that the wait for that stage's operands runs out after a few
milliseconds.  Every role of the kernel must then give up and return: the call reports
W4A8_ERR_TIMEOUT with the code of the wait that ran out, comes back well inside a second,
leaves the device usable, and a normal call on the same (re-initialised) workspace gives the
oracle's bits.  Nothing traps and nothing spins without a limit."""
import time

import numpy as np
import pytest
import torch

import paper_2311_05161_b200 as w4a8
from util import Problem, bf16_bits, check_y

pytestmark = pytest.mark.gpu

TIMEOUT = 7                     # W4A8_ERR_TIMEOUT
SITE_OPERANDS = 21              # the MMA thread's wait for a stage's operands


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("N,M,tok_tile,split", [(128, 16, 16, 1), (384, 40, 16, 1), (256, 300, 128, 2)])
def test_a_wait_that_runs_out_is_reported_and_the_kernel_returns(N, M, tok_tile, split, group):
    prob = Problem(1024, N, M, group, seed=900 + N + M + group)
    d = prob.dev
    packed = w4a8.pack_weights(d["W"], d["s"], group)
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    good = w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=split, tok_tile=tok_tile)
    bad = w4a8.make_opts(w4a8.PATH_TCGEN05, split_k=split, tok_tile=tok_tile, debug_wait_ms=5,
                         debug_skip_load=3)
    ws = w4a8.new_workspace(M, N, 1024, group, good)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    w4a8.linear(Xq, tok, packed, d["bias"], N, group, ws, bad)
    status = w4a8.poll_status(ws)                     # synchronizes the stream
    elapsed = time.perf_counter() - t0
    assert status == TIMEOUT
    assert elapsed < 1.0, f"the failing call took {elapsed:.2f} s"
    assert w4a8.poll_status(ws) == 0                  # cleared by the poll
    # the device and the context are still usable: a workspace that saw a failure is
    # re-initialised, then the same layer gives the oracle's bits
    w4a8.workspace_init(ws)
    for _ in range(2):
        Y = w4a8.linear(Xq, tok, packed, d["bias"], N, group, ws, good)
        w4a8.check_status(ws)
        check_y(prob, bf16_bits(Y), exact=(group == 0))


def test_the_site_of_the_wait_is_recorded():
    # two k-blocks only: no decode warp ever has to wait for a weight buffer, so the issuing
    # thread's wait for the operands of k-block 0 is the one wait that runs out first
    prob = Problem(256, 128, 16, 0, seed=931)
    d = prob.dev
    packed = w4a8.pack_weights(d["W"], d["s"], 0)
    Xq, tok = w4a8.quantize_act(d["X"], d["inv_s"])
    bad = w4a8.make_opts(w4a8.PATH_TCGEN05, tok_tile=16, debug_wait_ms=5, debug_skip_load=1)
    ws = w4a8.new_workspace(16, 128, 256, 0, bad)
    w4a8.linear(Xq, tok, packed, d["bias"], 128, 0, ws, bad)
    torch.cuda.synchronize()
    block = ws[:12].cpu().numpy().view(np.int32)      # status, site, reporting CTA
    assert block[0] == TIMEOUT and block[1] == SITE_OPERANDS and block[2] == 0
    assert w4a8.poll_status(ws) == TIMEOUT


def test_the_hooks_are_refused_outside_the_tensor_core_path():
    for path in (w4a8.PATH_AUTO, w4a8.PATH_SIMPLE, w4a8.PATH_GEMV):
        o = w4a8.make_opts(path, debug_wait_ms=5, debug_skip_load=1)
        assert w4a8.linear_workspace_bytes(2, 256, 256, 0, o) == 0
    assert w4a8.linear_workspace_bytes(2, 256, 256, 0, w4a8.make_opts(w4a8.PATH_TCGEN05, debug_wait_ms=5000)) == 0
