"""Helpers shared by the GPU parity tests: host problem -> device tensors -> comparison."""
import numpy as np
import torch

import oracle
import paper_2311_05161_b200 as w4a8
from paper_2311_05161_b200 import synth


def to_dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


def bf16_bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def bf16_ulp(x64):
    """Spacing of BF16 numbers at |x| (8 significant bits), never below the subnormal step."""
    e = np.floor(np.log2(np.maximum(np.abs(x64), 2.0 ** -126)))
    return 2.0 ** (e - 7)


class Problem:
    """One layer on the host with its oracle results, and the same tensors on the device."""

    def __init__(self, K, N, M, group, seed=0, dist="normal", outliers=4, mult=50.0,
                 scaled=True, with_bias=True, rows=None):
        lay = synth.make_layer(K, N, M, seed, dist, outliers, mult, scaled, with_bias)
        self.K, self.N, self.M, self.group = K, N, M, group
        self.host = lay
        self.dev = {k: to_dev(v) for k, v in lay.items()}
        # oracle side (optionally only for a subset of output rows: quantization is per row)
        self.rows = None if rows is None else np.asarray(rows)
        Wsel = lay["W"] if rows is None else lay["W"][self.rows]
        self.codes, self.scales, self.zeros = oracle.pack_weights(Wsel, lay["s"], group)
        self.Xq, self.tok = oracle.quantize_act(lay["X"], lay["inv_s"])
        self.bias_sel = None if lay["bias"] is None else (
            lay["bias"] if rows is None else lay["bias"][self.rows])

    def oracle_acc(self):
        return oracle.linear_acc(self.Xq, self.codes, self.zeros, self.group)

    def oracle_y_bits(self):
        return oracle.linear(self.Xq, self.tok, self.codes, self.scales, self.zeros,
                             self.bias_sel, self.group)

    def oracle_y64(self):
        return oracle.linear_f64(self.Xq, self.tok, self.codes, self.scales, self.zeros,
                                 self.bias_sel, self.group)

    def group_tolerance(self):
        """1 BF16 ulp of the binary64 value plus the FP32 reordering allowance
        2^-20 * tok_scale * sum_g |acc_g * step_g / 2|."""
        acc = oracle.linear_acc(self.Xq, self.codes, self.zeros, self.group, wide=True)
        mag = (np.abs(acc) * (0.5 * self.scales.astype(np.float64))[:, None, :]).sum(0)
        y64 = self.oracle_y64()
        return bf16_ulp(y64) + 2.0 ** -20 * self.tok.astype(np.float64)[:, None] * mag, y64


def check_y(prob, Y, exact):
    """Compare device output bits Y [M, N'] (uint16) against the oracle."""
    want = prob.oracle_y_bits()
    if exact:
        bad = np.argwhere(Y != want)
        assert bad.size == 0, f"{len(bad)} BF16 outputs differ, first at {bad[0]}"
        return
    tol, y64 = prob.group_tolerance()
    got = oracle.bf16_bits_to_float(Y).astype(np.float64)
    err = np.abs(got - y64)
    bad = np.argwhere(err > tol)
    assert bad.size == 0, f"{len(bad)} outputs beyond tolerance, first at {bad[0]}"
    # and never more than one BF16 step from the binary32-order oracle value
    ref = oracle.bf16_bits_to_float(want).astype(np.float64)
    assert np.all(np.abs(got - ref) <= 2 * bf16_ulp(y64) + tol)


class Guarded:
    """A device tensor in the middle of a larger allocation whose margins hold a byte pattern:
    a kernel that writes outside the tensor it was given changes a margin."""
    MARGIN = 8192
    PATTERN = 0xA5

    def __init__(self, shape, dtype):
        shape = tuple(int(x) for x in shape)
        self.nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        body = (self.nbytes + 255) // 256 * 256
        self.raw = torch.full((2 * self.MARGIN + body,), self.PATTERN, dtype=torch.uint8, device="cuda")
        self.t = self.raw[self.MARGIN:self.MARGIN + self.nbytes].view(dtype).view(shape)

    def check(self, what=""):
        lo = self.raw[:self.MARGIN]
        hi = self.raw[self.MARGIN + self.nbytes:]
        assert bool((lo == self.PATTERN).all()), f"{what}: bytes before the buffer were written"
        assert bool((hi == self.PATTERN).all()), f"{what}: bytes behind the buffer were written"


def guarded_workspace(nbytes):
    g = Guarded((nbytes,), torch.uint8)
    w4a8.workspace_init(g.t)
    return g
