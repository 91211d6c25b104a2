"""GPU parity of the attention value path (w4a8_pack_value, w4a8_attn_pv) against the oracle,
through the C ABI: packed value codes, steps and zero-points bit for bit, INT8 attention map
bit for bit, BF16 outputs bit for bit (channel-wise values: one FP32 evaluation order)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from util import Guarded, bf16_bits, guarded_workspace, to_dev

pytestmark = pytest.mark.gpu
D = 128


def softmax_rows(x):
    e = np.exp(x - x.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def run(H, T, S, seed, causal=False):
    rng = np.random.default_rng(seed)
    logits = rng.standard_normal((H, T, S)) * 2.0
    if causal:                      # token t attends to the first S - T + t + 1 positions
        mask = np.arange(S)[None, :] > (S - T + np.arange(T))[:, None]
        logits = np.where(mask[None], -1e9, logits)
    P = softmax_rows(logits).astype(np.float16)
    V = (rng.standard_normal((S, H, D)) * (0.5 + rng.random((1, H, D)))).astype(np.float16)
    packed = w4a8.pack_value(to_dev(V))
    codes, scales, zeros = oracle.pack_value(V)
    gc, gs, gz = w4a8.unpack_codes(packed, H * D, S, 0)
    assert np.array_equal(gc.cpu().numpy(), codes), "value codes"
    assert np.array_equal(gz.cpu().numpy(), zeros) and np.array_equal(gs.cpu().numpy().view(np.uint32), scales.view(np.uint32))
    Pq, ps = w4a8.quantize_act(to_dev(P.reshape(H * T, S)))
    oPq, ops = oracle.quantize_act(P.reshape(H * T, S))
    assert np.array_equal(Pq.cpu().numpy(), oPq) and np.array_equal(ps.cpu().numpy().view(np.uint32), ops.view(np.uint32))
    want = oracle.attn_pv(oPq.reshape(H, T, S), ops.reshape(H, T), codes, scales, zeros, D)
    gO = Guarded((T, H, D), torch.bfloat16)
    gws = guarded_workspace(int(w4a8.lib.w4a8_attn_pv_workspace_bytes(T, S, H, D)))
    for _ in range(2):
        O = w4a8.attn_pv(Pq.view(H, T, S), ps.view(H, T), packed, D, gws.t, out=gO.t)
        w4a8.check_status(gws.t)
        gO.check("O")
        gws.check("workspace")
        got = bf16_bits(O)
        bad = np.argwhere(got != want)
        assert bad.size == 0, f"{len(bad)} outputs differ, first at {bad[0]}"


@pytest.mark.parametrize("H,T,S", [(2, 16, 128), (3, 37, 384), (4, 300, 512), (32, 1, 1024), (8, 5, 2048),
                                   (2, 520, 640)])
def test_attn_pv_matches_oracle(H, T, S):
    run(H, T, S, seed=H + T + S)


def test_causal_prefill_block():
    run(4, 256, 256, seed=11, causal=True)


def test_validation():
    assert w4a8.lib.w4a8_attn_pv_workspace_bytes(16, 128, 2, 64) == 0      # head dimension 128 only
    assert w4a8.lib.w4a8_attn_pv_workspace_bytes(16, 100, 2, 128) == 0     # S % 128
    assert w4a8.lib.w4a8_attn_pv_workspace_bytes(16, 128, 2, 128) >= 256
