"""Seeded synthetic inputs with the shapes and value structure of the paper's workloads.

This module holds no quantizer or matmul arithmetic: it only draws tensors.  The
same host arrays feed the CUDA library and the CPU checker, so that both sides see
identical bytes.

The paper evaluates OPT and LLaMA decoder layers (Section 3.1, Section 5).  Its
models and datasets are replaced here by random tensors of the same layer shapes:
weights are zero-mean normal with standard deviation 0.02; activations are unit
normal or unit Laplace with a small, fixed set of input channels magnified, which
is the outlier structure Section 3.1 describes (OPT: about 0.1 % of channels carry
large values at fixed positions; LLaMA: a broader set).  The per-input-channel
scale of Eq. 1 is not searched for; a closed form in the style of earlier scaling
methods stands in for the search result.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark configuration: a list of (K, N) linear shapes and token counts."""
    config: int
    name: str
    shapes: tuple          # ((K, N, label), ...)
    tokens: tuple          # token counts M
    act_dist: str          # "normal" | "laplace"
    outlier_channels: object   # int count, or float ratio of K
    outlier_mult: float
    group: int             # 0 = one scale per output channel, 128 = per group

    def seed(self, shape_index: int) -> int:
        return 0 if self.config == 1 else 1000 * self.config + shape_index


WORKLOADS = {
    1: Workload(1, "tiny", ((768, 768, "linear"),), (16,), "normal", 4, 50.0, 0),
    2: Workload(2, "opt-6.7b-block",
                ((4096, 12288, "qkv"), (4096, 4096, "out"),
                 (4096, 16384, "fc1"), (16384, 4096, "fc2")),
                (2048, 1), "normal", 0.001, 60.0, 0),
    3: Workload(3, "llama-7b-block",
                ((4096, 11008, "gate"), (4096, 11008, "up"),
                 (11008, 4096, "down"), (4096, 12288, "qkv")),
                (1, 8, 512, 2048), "laplace", 0.01, 20.0, 128),
    4: Workload(4, "opt-66b-llama-65b",
                ((9216, 36864, "opt66b-fc1"), (36864, 9216, "opt66b-fc2"),
                 (9216, 27648, "opt66b-qkv"), (9216, 9216, "opt66b-out"),
                 (8192, 22016, "llama65b-gate"), (22016, 8192, "llama65b-down"),
                 (8192, 24576, "llama65b-qkv"), (8192, 8192, "llama65b-out")),
                (2048, 16), "normal", 0.001, 60.0, 0),
    5: Workload(5, "llama-7b-down-sweep", ((11008, 4096, "down"),),
                (1, 2, 4, 16, 64, 256, 1024, 4096, 16384), "laplace", 0.01, 20.0, 128),
}


def n_outliers(K: int, spec) -> int:
    if isinstance(spec, float):
        return int(math.ceil(spec * K))
    return int(spec)


def outlier_channels(K: int, spec, seed: int) -> np.ndarray:
    """Indices of the magnified input channels: the head of a seeded permutation."""
    rng = np.random.Generator(np.random.PCG64([seed, 7]))
    return np.sort(rng.permutation(K)[: n_outliers(K, spec)])


def make_weights(N: int, K: int, seed: int, n_rows: int | None = None) -> np.ndarray:
    """[N, K] float16, normal with standard deviation 0.02.  With `n_rows` only the first
    n_rows rows are drawn (the same values the full matrix has there)."""
    rng = np.random.Generator(np.random.PCG64([seed, 1]))
    n_out = N if n_rows is None else min(N, n_rows)
    out = np.empty((n_out, K), dtype=np.float16)
    rows = max(1, (1 << 24) // K)
    buf = np.empty((rows, K), dtype=np.float32)
    for r0 in range(0, n_out, rows):
        r1 = min(N, r0 + rows)          # chunk boundaries follow the full matrix
        chunk = buf[: r1 - r0]
        rng.standard_normal(out=chunk, dtype=np.float32)
        np.multiply(chunk, np.float32(0.02), out=chunk)
        keep = min(r1, n_out) - r0
        out[r0:r0 + keep] = chunk[:keep]
    return out


def make_activations(M: int, K: int, seed: int, dist: str = "normal",
                     outliers=4, mult: float = 50.0) -> np.ndarray:
    """[M, K] float16 tokens; `outliers` input channels are multiplied by `mult`."""
    rng = np.random.Generator(np.random.PCG64([seed, 2]))
    ch = outlier_channels(K, outliers, seed)
    out = np.empty((M, K), dtype=np.float16)
    rows = max(1, (1 << 24) // K)
    for r0 in range(0, M, rows):
        r1 = min(M, r0 + rows)
        if dist == "normal":
            x = rng.standard_normal((r1 - r0, K), dtype=np.float32)
        elif dist == "laplace":
            x = rng.laplace(0.0, 1.0, (r1 - r0, K)).astype(np.float32)
        else:
            raise ValueError(dist)
        x[:, ch] *= np.float32(mult)
        out[r0:r1] = x.astype(np.float16)
    return out


def make_bias(N: int, seed: int) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64([seed, 3]))
    return (rng.standard_normal(N, dtype=np.float32) * np.float32(0.1)).astype(np.float32)


def make_channel_scales(X: np.ndarray, W: np.ndarray):
    """Stand-in for the searched per-input-channel scale s of Eq. 1.

    s_k = clamp(sqrt(max_m |X[m,k]| / max_n |W[n,k]|), 2^-4, 2^4); the weight side
    multiplies by s, the activation side by the binary32 reciprocal.
    Returns (s [K] float32, inv_s [K] float32).
    """
    def col_absmax(A):
        m = np.zeros(A.shape[1], dtype=np.float32)
        rows = max(1, (1 << 24) // A.shape[1])
        for r0 in range(0, A.shape[0], rows):
            np.maximum(m, np.abs(A[r0:r0 + rows]).max(axis=0).astype(np.float32), out=m)
        return m

    ax = col_absmax(X)
    aw = col_absmax(W)
    with np.errstate(divide="ignore", invalid="ignore"):
        s = np.sqrt(ax / aw)
    s = np.where(np.isfinite(s), s, 1.0)
    s = np.clip(s, 2.0 ** -4, 2.0 ** 4).astype(np.float32)
    inv = (np.float32(1.0) / s).astype(np.float32)
    return s, inv


def make_layer(K: int, N: int, M: int, seed: int, dist: str = "normal",
               outliers=4, mult: float = 50.0, scaled: bool = True,
               with_bias: bool = True):
    """One linear layer's host inputs: dict with W, X, s, inv_s, bias."""
    W = make_weights(N, K, seed)
    X = make_activations(M, K, seed, dist, outliers, mult)
    s = inv = None
    if scaled:
        s, inv = make_channel_scales(X, W)
    bias = make_bias(N, seed) if with_bias else None
    return {"W": W, "X": X, "s": s, "inv_s": inv, "bias": bias}


def workload_layer(config: int, shape_index: int, M: int, scaled: bool = True,
                   with_bias: bool = True):
    wl = WORKLOADS[config]
    K, N, _ = wl.shapes[shape_index]
    return make_layer(K, N, M, wl.seed(shape_index), wl.act_dist, wl.outlier_channels,
                      wl.outlier_mult, scaled, with_bias)
